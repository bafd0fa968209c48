/*
 * ksa_oracle.c -- plain CPU oracle for Kwai Summary Attention (KSA): forward and gradients.
 *
 * TEST INFRASTRUCTURE ONLY (see ksa_oracle.h).  Plain C, fp64 arithmetic on the
 * exact bf16 input values, explicit mask row per query, no tiling, no skipping of
 * key positions by band arithmetic: every key position of the query's sequence is
 * put through the visibility predicate.
 */
#include "ksa_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 bit pattern -> double (bf16 is the upper half of an IEEE fp32). */
static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int64_t ksa_oracle_aug_len(int64_t n_text, int32_t k, int32_t m)
{
    if (n_text < 0 || k < 1 || m < 0) return -1;
    /* Eq. 1 with one summary per chunk generalised to m; only FULL chunks get summaries. */
    return n_text + (n_text / k) * (int64_t)m;
}

int ksa_oracle_decode_pos(int64_t n_text, int32_t k, int32_t m, int64_t p,
                          int32_t* is_summary, int64_t* index, int32_t* r)
{
    int64_t L = ksa_oracle_aug_len(n_text, k, m);
    if (L < 0 || p < 0 || p >= L) return -1;
    int64_t s = (int64_t)k + m;      /* chunk_j = [t_{jk} .. t_{jk+k-1}, s_j] has k+m entries */
    int64_t J = n_text / k;          /* full chunks */
    if (p < J * s) {
        int64_t j = p / s, o = p % s;
        if (o < k) { *is_summary = 0; *index = j * k + o; *r = 0; }
        else       { *is_summary = 1; *index = j;         *r = (int32_t)(o - k); }
    } else {
        /* trailing partial chunk: text only */
        *is_summary = 0; *index = J * k + (p - J * s); *r = 0;
    }
    return 0;
}

int ksa_oracle_visible(int64_t n_text, int32_t k, int32_t m, int32_t C, uint32_t flags,
                       int64_t pq, int64_t pk)
{
    int32_t q_sum, k_sum, q_r, k_r;
    int64_t q_idx, k_idx;
    if (C < 0) return -1;
    if (ksa_oracle_decode_pos(n_text, k, m, pq, &q_sum, &q_idx, &q_r) != 0) return -1;
    if (ksa_oracle_decode_pos(n_text, k, m, pk, &k_sum, &k_idx, &k_r) != 0) return -1;

    if (!q_sum) {
        /* Eq. 3: text token i, c = floor(i/k). */
        int64_t i = q_idx, c = i / k;
        if (!k_sum) {
            /* sliding chunk text tokens t_{(c-C)k} .. t_i */
            int64_t ip = k_idx;
            return (ip <= i && ip / k >= c - C) ? 1 : 0;
        }
        /* distant summary tokens s_0 .. s_{c-C-1}: every slot r of those chunks */
        return (k_idx <= c - C - 1) ? 1 : 0;
    }
    /* Summary token (j, r): text of its own chunk; by default also the summaries
     * 0..r of its own chunk (itself included); nothing else. */
    {
        int64_t j = q_idx;
        if (!k_sum) return (k_idx / k == j) ? 1 : 0;
        if (flags & KSA_ORACLE_SUMMARY_TEXT_ONLY) return 0;
        return (k_idx == j && k_r <= q_r) ? 1 : 0;
    }
}

int64_t ksa_oracle_mask_row(int64_t n_text, int32_t k, int32_t m, int32_t C, uint32_t flags,
                            int64_t pq, uint8_t* row)
{
    int64_t L = ksa_oracle_aug_len(n_text, k, m);
    if (L < 0 || pq < 0 || pq >= L || C < 0 || !row) return -1;
    for (int64_t pk = 0; pk < L; ++pk)
        row[pk] = (uint8_t)ksa_oracle_visible(n_text, k, m, C, flags, pq, pk);
    return L;
}

int64_t ksa_oracle_visible_count(int64_t n_text, int32_t k, int32_t m, int32_t C,
                                 uint32_t flags, int64_t pq)
{
    int64_t L = ksa_oracle_aug_len(n_text, k, m);
    if (L < 0 || pq < 0 || pq >= L || C < 0) return -1;
    uint8_t* row = (uint8_t*)malloc((size_t)L);
    if (!row) return -1;
    ksa_oracle_mask_row(n_text, k, m, C, flags, pq, row);
    int64_t cnt = 0;
    for (int64_t pk = 0; pk < L; ++pk) cnt += row[pk];
    free(row);
    return cnt;
}

int64_t ksa_oracle_total_pairs(int32_t num_seqs, const int32_t* cu_text_lens, int32_t k,
                               int32_t m, int32_t C, uint32_t flags)
{
    if (num_seqs < 0 || !cu_text_lens || k < 1 || m < 0 || C < 0) return -1;
    int64_t total = 0;
    for (int32_t b = 0; b < num_seqs; ++b) {
        int64_t n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
        int64_t L = ksa_oracle_aug_len(n, k, m);
        int64_t seq_total = 0;
#pragma omp parallel reduction(+ : seq_total)
        {
            uint8_t* row = (uint8_t*)malloc((size_t)(L > 0 ? L : 1));
#pragma omp for schedule(dynamic, 64)
            for (int64_t pq = 0; pq < L; ++pq) {
                ksa_oracle_mask_row(n, k, m, C, flags, pq, row);
                int64_t cnt = 0;
                for (int64_t pk = 0; pk < L; ++pk) cnt += row[pk];
                seq_total += cnt;
            }
            free(row);
        }
        total += seq_total;
    }
    return total;
}

int ksa_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int ksa_oracle_fwd(const uint16_t* q, const uint16_t* kk, const uint16_t* v,
                   int32_t num_seqs, const int32_t* cu_text_lens,
                   int32_t k, int32_t m, int32_t C,
                   int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                   const int64_t* rows, int64_t n_rows,
                   double* out, double* lse, int64_t* count)
{
    if (!q || !kk || !v || !cu_text_lens || !out || !lse) return -1;
    if (num_seqs < 1 || k < 1 || m < 0 || C < 0 || Hq < 1 || Hkv < 1 || D < 1) return -1;
    if (Hq % Hkv != 0) return -1;
    const int32_t G = Hq / Hkv;

    /* augmented offsets of the packed sequences */
    int64_t* aug_off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(num_seqs + 1));
    if (!aug_off) return -1;
    aug_off[0] = 0;
    int64_t max_L = 1;
    for (int32_t b = 0; b < num_seqs; ++b) {
        int64_t n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
        if (n < 0) { free(aug_off); return -1; }
        int64_t L = ksa_oracle_aug_len(n, k, m);
        aug_off[b + 1] = aug_off[b] + L;
        if (L > max_L) max_L = L;
    }
    const int64_t total_aug = aug_off[num_seqs];
    const int64_t R = rows ? n_rows : total_aug;
    int bad = 0;

#pragma omp parallel
    {
        uint8_t* mask = (uint8_t*)malloc((size_t)max_L);
        double* x = (double*)malloc(sizeof(double) * (size_t)max_L);
        double* acc = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 4)
        for (int64_t ri = 0; ri < R; ++ri) {
            const int64_t g = rows ? rows[ri] : ri;   /* global augmented row */
            if (g < 0 || g >= total_aug) { bad = 1; continue; }
            int32_t b = 0;
            while (g >= aug_off[b + 1]) ++b;          /* sequence of this row */
            const int64_t n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
            const int64_t base = aug_off[b];
            const int64_t L = aug_off[b + 1] - base;
            const int64_t pq = g - base;

            /* explicit mask row M_KSA[pq, :] */
            ksa_oracle_mask_row(n, k, m, C, flags, pq, mask);
            int64_t cnt = 0;
            for (int64_t pk = 0; pk < L; ++pk) cnt += mask[pk];
            if (count) count[ri] = cnt;

            for (int32_t h = 0; h < Hq; ++h) {
                const int32_t hk = h / G;
                const uint16_t* qrow = q + ((size_t)g * Hq + h) * (size_t)D;
                /* x_j = scale * <q, k_j> on visible keys, M = max_j x_j */
                double M = -INFINITY;
                for (int64_t pk = 0; pk < L; ++pk) {
                    if (!mask[pk]) continue;
                    const uint16_t* krow = kk + ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
                    double dot = 0.0;
                    for (int32_t d = 0; d < D; ++d)
                        dot += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
                    x[pk] = scale * dot;
                    if (x[pk] > M) M = x[pk];
                }
                /* l = sum_j exp(x_j - M); out = sum_j exp(x_j - M) v_j / l; lse = M + ln l */
                double l = 0.0;
                for (int32_t d = 0; d < D; ++d) acc[d] = 0.0;
                for (int64_t pk = 0; pk < L; ++pk) {
                    if (!mask[pk]) continue;
                    const double w = exp(x[pk] - M);
                    const uint16_t* vrow = v + ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
                    l += w;
                    for (int32_t d = 0; d < D; ++d) acc[d] += w * bf16_to_double(vrow[d]);
                }
                double* orow = out + ((size_t)ri * Hq + h) * (size_t)D;
                for (int32_t d = 0; d < D; ++d) orow[d] = acc[d] / l;
                lse[(size_t)ri * Hq + h] = M + log(l);
            }
        }
        free(mask); free(x); free(acc);
    }
    free(aug_off);
    return bad ? -1 : 0;
}

/* Softmax weights of row pq of a sequence (head h) over its explicit mask row: x[] receives
 * p_j on visible positions (untouched elsewhere), the return value is the row's output o (in acc). */
static void row_weights(const uint16_t* q, const uint16_t* kk, const uint16_t* v, int64_t base, int64_t L,
                        int64_t g, int32_t h, int32_t hk, int32_t Hq, int32_t Hkv, int32_t D, double scale,
                        const uint8_t* mask, double* x, double* acc)
{
    const uint16_t* qrow = q + ((size_t)g * Hq + h) * (size_t)D;
    double M = -INFINITY;
    for (int64_t pk = 0; pk < L; ++pk) {
        if (!mask[pk]) continue;
        const uint16_t* krow = kk + ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
        double dot = 0.0;
        for (int32_t d = 0; d < D; ++d) dot += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
        x[pk] = scale * dot;
        if (x[pk] > M) M = x[pk];
    }
    double l = 0.0;
    for (int64_t pk = 0; pk < L; ++pk)
        if (mask[pk]) { x[pk] = exp(x[pk] - M); l += x[pk]; }
    for (int32_t d = 0; d < D; ++d) acc[d] = 0.0;
    for (int64_t pk = 0; pk < L; ++pk) {
        if (!mask[pk]) continue;
        x[pk] /= l;                                   /* p_j */
        const uint16_t* vrow = v + ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
        for (int32_t d = 0; d < D; ++d) acc[d] += x[pk] * bf16_to_double(vrow[d]);
    }
}

int ksa_oracle_bwd(const uint16_t* q, const uint16_t* kk, const uint16_t* v, const uint16_t* dout,
                   int32_t num_seqs, const int32_t* cu_text_lens,
                   int32_t k, int32_t m, int32_t C,
                   int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                   double* dq, double* dk, double* dv)
{
    if (!q || !kk || !v || !dout || !cu_text_lens || !dq || !dk || !dv) return -1;
    if (num_seqs < 1 || k < 1 || m < 0 || C < 0 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return -1;
    const int32_t G = Hq / Hkv;
    int64_t total_aug = 0, max_L = 1;
    for (int32_t b = 0; b < num_seqs; ++b) {
        int64_t L = ksa_oracle_aug_len((int64_t)cu_text_lens[b + 1] - cu_text_lens[b], k, m);
        if (L < 0) return -1;
        total_aug += L;
        if (L > max_L) max_L = L;
    }
    memset(dq, 0, sizeof(double) * (size_t)total_aug * Hq * D);
    memset(dk, 0, sizeof(double) * (size_t)total_aug * Hkv * D);
    memset(dv, 0, sizeof(double) * (size_t)total_aug * Hkv * D);

    /* One KV head per task: rows are walked in order, so the sums into dk / dv of that head need no
     * locking and always add in the same order. */
#pragma omp parallel
    {
        uint8_t* mask = (uint8_t*)malloc((size_t)max_L);
        double* p = (double*)malloc(sizeof(double) * (size_t)max_L);
        double* o = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int32_t hk = 0; hk < Hkv; ++hk) {
            int64_t base = 0;
            for (int32_t b = 0; b < num_seqs; ++b) {
                const int64_t n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
                const int64_t L = ksa_oracle_aug_len(n, k, m);
                for (int64_t pq = 0; pq < L; ++pq) {
                    ksa_oracle_mask_row(n, k, m, C, flags, pq, mask);
                    const int64_t g = base + pq;
                    for (int32_t h = hk * G; h < (hk + 1) * G; ++h) {
                        row_weights(q, kk, v, base, L, g, h, hk, Hq, Hkv, D, scale, mask, p, o);
                        const uint16_t* qrow = q + ((size_t)g * Hq + h) * (size_t)D;
                        const uint16_t* drow = dout + ((size_t)g * Hq + h) * (size_t)D;
                        double delta = 0.0;                               /* <dO_i, o_i> */
                        for (int32_t d = 0; d < D; ++d) delta += bf16_to_double(drow[d]) * o[d];
                        double* dqrow = dq + ((size_t)g * Hq + h) * (size_t)D;
                        for (int64_t pk = 0; pk < L; ++pk) {
                            if (!mask[pk]) continue;
                            const size_t kvoff = ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
                            double dP = 0.0;                              /* <dO_i, v_j> */
                            for (int32_t d = 0; d < D; ++d) dP += bf16_to_double(drow[d]) * bf16_to_double(v[kvoff + d]);
                            const double dS = p[pk] * (dP - delta);
                            for (int32_t d = 0; d < D; ++d) {
                                dv[kvoff + d] += p[pk] * bf16_to_double(drow[d]);
                                dk[kvoff + d] += scale * dS * bf16_to_double(qrow[d]);
                                dqrow[d] += scale * dS * bf16_to_double(kk[kvoff + d]);
                            }
                        }
                    }
                }
                base += L;
            }
        }
        free(mask); free(p); free(o);
    }
    return 0;
}

/* The same gradients on a SAMPLE of rows, for inputs too long to differentiate in full:
 *   dq of the query rows q_rows[0..nq)   (global augmented rows; dq of a row only involves that row's own weights);
 *   dk, dv of the key rows k_rows[0..nk) (the sums over every query row of the same sequence that sees the key).
 * Same arithmetic as ksa_oracle_bwd, term by term; every query row that sees a sampled key still gets its complete
 * softmax over its explicit mask row.  Outputs: dq [nq, Hq, D], dk and dv [nk, Hkv, D]. */
int ksa_oracle_bwd_rows(const uint16_t* q, const uint16_t* kk, const uint16_t* v, const uint16_t* dout,
                        int32_t num_seqs, const int32_t* cu_text_lens,
                        int32_t k, int32_t m, int32_t C,
                        int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                        const int64_t* q_rows, int64_t nq, double* dq,
                        const int64_t* k_rows, int64_t nk, double* dk, double* dv)
{
    if (!q || !kk || !v || !dout || !cu_text_lens) return -1;
    if ((nq > 0 && (!q_rows || !dq)) || (nk > 0 && (!k_rows || !dk || !dv)) || nq < 0 || nk < 0) return -1;
    if (num_seqs < 1 || k < 1 || m < 0 || C < 0 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return -1;
    const int32_t G = Hq / Hkv;
    int64_t total_aug = 0, max_L = 1;
    for (int32_t b = 0; b < num_seqs; ++b) {
        int64_t L = ksa_oracle_aug_len((int64_t)cu_text_lens[b + 1] - cu_text_lens[b], k, m);
        if (L < 0) return -1;
        total_aug += L;
        if (L > max_L) max_L = L;
    }
    for (int64_t r = 0; r < nq; ++r) if (q_rows[r] < 0 || q_rows[r] >= total_aug) return -1;
    for (int64_t r = 0; r < nk; ++r) if (k_rows[r] < 0 || k_rows[r] >= total_aug) return -1;
    if (nq > 0) memset(dq, 0, sizeof(double) * (size_t)nq * Hq * D);
    if (nk > 0) { memset(dk, 0, sizeof(double) * (size_t)nk * Hkv * D); memset(dv, 0, sizeof(double) * (size_t)nk * Hkv * D); }

    /* ---- dq of the sampled query rows ---- */
#pragma omp parallel
    {
        uint8_t* mask = (uint8_t*)malloc((size_t)max_L);
        double* p = (double*)malloc(sizeof(double) * (size_t)max_L);
        double* o = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < nq; ++r) {
            const int64_t g = q_rows[r];
            int64_t base = 0, n = 0, L = 0;
            for (int32_t b = 0; b < num_seqs; ++b) {              /* the sequence that holds row g */
                n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
                L = ksa_oracle_aug_len(n, k, m);
                if (g < base + L) break;
                base += L;
            }
            ksa_oracle_mask_row(n, k, m, C, flags, g - base, mask);
            for (int32_t h = 0; h < Hq; ++h) {
                const int32_t hk = h / G;
                row_weights(q, kk, v, base, L, g, h, hk, Hq, Hkv, D, scale, mask, p, o);
                const uint16_t* drow = dout + ((size_t)g * Hq + h) * (size_t)D;
                double delta = 0.0;
                for (int32_t d = 0; d < D; ++d) delta += bf16_to_double(drow[d]) * o[d];
                double* dqrow = dq + ((size_t)r * Hq + h) * (size_t)D;
                for (int64_t pk = 0; pk < L; ++pk) {
                    if (!mask[pk]) continue;
                    const size_t kvoff = ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
                    double dP = 0.0;
                    for (int32_t d = 0; d < D; ++d) dP += bf16_to_double(drow[d]) * bf16_to_double(v[kvoff + d]);
                    const double dS = p[pk] * (dP - delta);
                    for (int32_t d = 0; d < D; ++d) dqrow[d] += scale * dS * bf16_to_double(kk[kvoff + d]);
                }
            }
        }
        free(mask); free(p); free(o);
    }
    if (nk == 0) return 0;

    /* ---- dk, dv of the sampled key rows: every query row of the key's sequence is asked whether it sees the key ---- */
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    const size_t acc_len = (size_t)nk * Hkv * D;
    double* part_k = (double*)calloc((size_t)nthreads * acc_len, sizeof(double));
    double* part_v = (double*)calloc((size_t)nthreads * acc_len, sizeof(double));
    if (!part_k || !part_v) { free(part_k); free(part_v); return -2; }
    int64_t base = 0;
    for (int32_t b = 0; b < num_seqs; ++b) {
        const int64_t n = (int64_t)cu_text_lens[b + 1] - cu_text_lens[b];
        const int64_t L = ksa_oracle_aug_len(n, k, m);
        int64_t in_seq = 0;
        for (int64_t r = 0; r < nk; ++r) if (k_rows[r] >= base && k_rows[r] < base + L) ++in_seq;
        if (in_seq > 0) {
#pragma omp parallel
            {
                int tid = 0;
#ifdef _OPENMP
                tid = omp_get_thread_num();
#endif
                double* ak = part_k + (size_t)tid * acc_len;
                double* av = part_v + (size_t)tid * acc_len;
                uint8_t* mask = (uint8_t*)malloc((size_t)max_L);
                double* p = (double*)malloc(sizeof(double) * (size_t)max_L);
                double* o = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 16)
                for (int64_t pq = 0; pq < L; ++pq) {
                    ksa_oracle_mask_row(n, k, m, C, flags, pq, mask);
                    int any = 0;
                    for (int64_t r = 0; r < nk && !any; ++r)
                        if (k_rows[r] >= base && k_rows[r] < base + L && mask[k_rows[r] - base]) any = 1;
                    if (!any) continue;
                    const int64_t g = base + pq;
                    for (int32_t h = 0; h < Hq; ++h) {
                        const int32_t hk = h / G;
                        row_weights(q, kk, v, base, L, g, h, hk, Hq, Hkv, D, scale, mask, p, o);
                        const uint16_t* qrow = q + ((size_t)g * Hq + h) * (size_t)D;
                        const uint16_t* drow = dout + ((size_t)g * Hq + h) * (size_t)D;
                        double delta = 0.0;
                        for (int32_t d = 0; d < D; ++d) delta += bf16_to_double(drow[d]) * o[d];
                        for (int64_t r = 0; r < nk; ++r) {
                            const int64_t pk = k_rows[r] - base;
                            if (pk < 0 || pk >= L || !mask[pk]) continue;
                            const size_t kvoff = ((size_t)(base + pk) * Hkv + hk) * (size_t)D;
                            double dP = 0.0;
                            for (int32_t d = 0; d < D; ++d) dP += bf16_to_double(drow[d]) * bf16_to_double(v[kvoff + d]);
                            const double dS = p[pk] * (dP - delta);
                            double* akr = ak + ((size_t)r * Hkv + hk) * (size_t)D;
                            double* avr = av + ((size_t)r * Hkv + hk) * (size_t)D;
                            for (int32_t d = 0; d < D; ++d) {
                                avr[d] += p[pk] * bf16_to_double(drow[d]);
                                akr[d] += scale * dS * bf16_to_double(qrow[d]);
                            }
                        }
                    }
                }
                free(mask); free(p); free(o);
            }
        }
        base += L;
    }
    for (int t = 0; t < nthreads; ++t)
        for (size_t e = 0; e < acc_len; ++e) { dk[e] += part_k[(size_t)t * acc_len + e]; dv[e] += part_v[(size_t)t * acc_len + e]; }
    free(part_k); free(part_v);
    return 0;
}
