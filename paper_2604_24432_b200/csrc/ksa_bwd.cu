// Backward pass of the KSA attention operator (gradients dQ, dK, dV for a given dO), first
// tensor-core version: mma.sync m16n8k16 on the packed text / summary streams of the forward
// pass, two kernels over the same Eq. 3 tile ranges:
//   dQ kernel   query-stationary: a CTA owns 64 text query rows of one head and walks the key
//               tiles visible to them; S = Q K^T, P = exp(S - lse), dP = dO V^T,
//               dS = P (dP - delta), dQ += dS K.
//   dKV kernel  key-stationary: a CTA owns 64 keys of one KV head and walks the (query tile, query
//               head) pairs that see them; everything is computed transposed (S^T = K Q^T ...) so
//               that each warp keeps dK, dV of its 16 keys in registers; partial sums of the query
//               segments are added to fp32 accumulators with vector atomics.
// Summary query rows (block-diagonal, at most k + m keys) are handled on CUDA cores.
// delta_i = <dO_i, O_i> and the packed dO / lse rows come from a preparation kernel.
#include <cuda_bf16.h>

#include <algorithm>

#include "ksa_bwd.h"

namespace ksa {

__device__ __forceinline__ uint32_t bsm_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void b_cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void b_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void b_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void b_ldsm4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void b_ldsm4t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void b_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t b_pack2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float b_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float b_bf2f(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

constexpr int kBT = 64;          // rows per tile (queries and keys) of the backward kernels

// A 64 x D bf16 tile in shared memory, rows of D*2 bytes, 16-byte chunks XOR-swizzled by (row & 7).
template <int D>
__device__ __forceinline__ void load_tile64(uint32_t sdst, const uint16_t* src /* row 0 of the tile, row stride D */, int tid, int nthreads)
{
    constexpr int kVec = D / 8;
    for (int idx = tid; idx < kBT * kVec; idx += nthreads) {
        const int r = idx / kVec, c16 = idx - r * kVec;
        b_cp_async16(sdst + (uint32_t)(r * D * 2 + ((c16 ^ (r & 7)) << 4)), src + (size_t)r * D + c16 * 8);
    }
}
template <int D>
__device__ __forceinline__ uint32_t tile_addr(uint32_t sbase, int row, int chunk)
{
    return sbase + (uint32_t)(row * D * 2 + ((chunk ^ (row & 7)) << 4));
}

// Eq. 3 in stream coordinates for text row i: first visible text row and number of visible summary rows.
__device__ __forceinline__ int eq3_lo(const BwdArgs& a, int i) { return max(0, i / a.k - a.C) * a.k; }
__device__ __forceinline__ int eq3_cnt(const BwdArgs& a, int i, int n_summ) { return min(n_summ, max(0, i / a.k - a.C) * a.m); }

// =================================================================================================
// dQ kernel.  grid (query tiles of 64 rows (longest first), query heads, sequences), 128 threads.
// =================================================================================================
template <int D>
__global__ void __launch_bounds__(128) ksa_bwd_dq_kernel(BwdArgs a)
{
    extern __shared__ __align__(128) uint8_t bsm[];
    constexpr int kTileB = kBT * D * 2;
    const SeqInfo sq = a.seqs[blockIdx.z];
    const int n_qt = (sq.n_text + kBT - 1) / kBT;
    const int qt = n_qt - 1 - (int)blockIdx.x;                 // longest (last) tiles first
    if (qt < 0) return;
    const int h = blockIdx.y, hk = h / (a.Hq / a.Hkv);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g0 = lane >> 2, c2 = (lane & 3) * 2, mi = lane >> 3, r8 = lane & 7;
    const int i_first = qt * kBT, i_last = min(sq.n_text, i_first + kBT) - 1;
    const int ns = (eq3_cnt(a, i_last, sq.n_summ) + kBT - 1) / kBT;       // summary tiles [0, ns)
    const int blo = eq3_lo(a, i_first) / kBT;                             // text tiles [blo, qt]
    const int T = ns + (qt - blo + 1);
    const uint32_t sK = bsm_u32(bsm), sV = sK + 2 * kTileB;               // two stages each
    const uint32_t sQ = sV + 2 * kTileB, sG = sQ + kTileB;               // Q and dO tiles of this CTA

    const size_t qrow0 = (size_t)h * a.text_rows + sq.text_off + i_first;
    load_tile64<D>(sQ, a.qt + qrow0 * D, threadIdx.x, 128);
    load_tile64<D>(sG, a.dot + qrow0 * D, threadIdx.x, 128);
    auto kv_src = [&](int j, const uint16_t*& kp, const uint16_t*& vp) {
        if (j < ns) {
            const size_t r = (size_t)hk * a.summ_rows + sq.summ_off + (size_t)j * kBT;
            kp = a.ks + r * D; vp = a.vs + r * D;
        } else {
            const size_t r = (size_t)hk * a.text_rows + sq.text_off + (size_t)(blo + j - ns) * kBT;
            kp = a.kt + r * D; vp = a.vt + r * D;
        }
    };
    {
        const uint16_t *kp, *vp;
        kv_src(0, kp, vp);
        load_tile64<D>(sK, kp, threadIdx.x, 128);
        load_tile64<D>(sV, vp, threadIdx.x, 128);
    }
    b_cp_commit();
    // per-row scalars of this thread's two rows (g0 and g0 + 8 of the warp's 16)
    const int i0 = i_first + warp * 16 + g0, i1 = i0 + 8;
    const float lse0 = a.lse_t[(size_t)h * a.text_rows + sq.text_off + i0], lse1 = a.lse_t[(size_t)h * a.text_rows + sq.text_off + i1];
    const float dl0 = a.delta_t[(size_t)h * a.text_rows + sq.text_off + i0], dl1 = a.delta_t[(size_t)h * a.text_rows + sq.text_off + i1];
    const int lo0 = eq3_lo(a, min(i0, sq.n_text - 1)), lo1 = eq3_lo(a, min(i1, sq.n_text - 1));
    const int cn0 = eq3_cnt(a, min(i0, sq.n_text - 1), sq.n_summ), cn1 = eq3_cnt(a, min(i1, sq.n_text - 1), sq.n_summ);
    const bool ok0 = i0 < sq.n_text, ok1 = i1 < sq.n_text;

    float dq[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }
    uint32_t qa[D / 16][4], ga[D / 16][4];
    bool frags_loaded = false;

    for (int j = 0; j < T; ++j) {
        if (j + 1 < T) {
            const uint16_t *kp, *vp;
            kv_src(j + 1, kp, vp);
            load_tile64<D>(sK + ((j + 1) & 1) * kTileB, kp, threadIdx.x, 128);
            load_tile64<D>(sV + ((j + 1) & 1) * kTileB, vp, threadIdx.x, 128);
        }
        b_cp_commit();
        b_cp_wait<1>();
        __syncthreads();
        if (!frags_loaded) {
            // A fragments of this warp's 16 rows of Q and dO (kept in registers for the whole walk)
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const int row = warp * 16 + (mi & 1) * 8 + r8, chunk = kk * 2 + (mi >> 1);
                b_ldsm4(qa[kk], tile_addr<D>(sQ, row, chunk));
                b_ldsm4(ga[kk], tile_addr<D>(sG, row, chunk));
            }
            frags_loaded = true;
        }
        const uint32_t sk = sK + (j & 1) * kTileB, sv = sV + (j & 1) * kTileB;
        const bool summ = j < ns;
        const int key0 = (summ ? j : (blo + j - ns)) * kBT;             // first key (stream row) of the tile
        float s[8][4], dp[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {                             // pairs of 8-key column tiles
                uint32_t kb[4], vb[4];
                const int key = np * 16 + (mi >> 1) * 8 + r8, chunk = kk * 2 + (mi & 1);
                b_ldsm4(kb, tile_addr<D>(sk, key, chunk));
                b_ldsm4(vb, tile_addr<D>(sv, key, chunk));
                b_mma(s[2 * np], qa[kk], kb[0], kb[1]);  b_mma(s[2 * np + 1], qa[kk], kb[2], kb[3]);
                b_mma(dp[2 * np], ga[kk], vb[0], vb[1]); b_mma(dp[2 * np + 1], ga[kk], vb[2], vb[3]);
            }
        }
        // P = exp(S scale - lse) on visible pairs, dS = P (dP - delta), as A fragments (bf16)
        uint32_t dsa[4][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float ds[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = key0 + nt * 8 + c2 + (e & 1);
                const bool up = e >= 2;
                const int irow = up ? i1 : i0;
                bool vis = up ? ok1 : ok0;
                if (summ) vis = vis && key < (up ? cn1 : cn0);
                else      vis = vis && key <= irow && key >= (up ? lo1 : lo0);
                const float p = vis ? b_ex2(s[nt][e] * a.scale_log2 - (up ? lse1 : lse0)) : 0.f;
                ds[e] = p * (dp[nt][e] - (up ? dl1 : dl0));
            }
            dsa[nt >> 1][(nt & 1) * 2 + 0] = b_pack2(ds[0], ds[1]);
            dsa[nt >> 1][(nt & 1) * 2 + 1] = b_pack2(ds[2], ds[3]);
        }
        // dQ += dS K   (k-steps of 16 keys, B = K[keys, d] through transposing loads)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int n2 = 0; n2 < D / 16; ++n2) {
                uint32_t kb[4];
                const int key = ks * 16 + (mi & 1) * 8 + r8, chunk = n2 * 2 + (mi >> 1);
                b_ldsm4t(kb, tile_addr<D>(sk, key, chunk));
                b_mma(dq[2 * n2], dsa[ks], kb[0], kb[1]);
                b_mma(dq[2 * n2 + 1], dsa[ks], kb[2], kb[3]);
            }
        }
        __syncthreads();
    }
    // dQ rows (times the softmax scale) to their augmented positions (Eq. 1), bf16
    const int s_len = a.k + a.m;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int i = half ? i1 : i0;
        if (i >= sq.n_text) continue;
        const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * s_len + (i % a.k);
        uint16_t* dst = a.dq + aug * a.dq_st + (int64_t)h * a.dq_sh;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt)
            *reinterpret_cast<uint32_t*>(dst + nt * 8 + c2) = b_pack2(dq[nt][half * 2] * a.scale, dq[nt][half * 2 + 1] * a.scale);
    }
}

// =================================================================================================
// dK / dV kernel.  grid (query segments, key tiles of 64 rows, sequences * KV heads); one launch per stream.
// Everything transposed: rows of the MMAs are this warp's 16 keys, columns the 64 queries of a tile.
// =================================================================================================
constexpr int kSegTiles = 16;     // query tiles per segment (times G heads iterations per CTA)

template <int D>
__global__ void __launch_bounds__(128) ksa_bwd_dkv_kernel(BwdArgs a, int summ)
{
    extern __shared__ __align__(128) uint8_t bsm[];
    constexpr int kTileB = kBT * D * 2;
    const int G = a.Hq / a.Hkv;
    const int hk = blockIdx.z % a.Hkv, b = blockIdx.z / a.Hkv;
    const SeqInfo sq = a.seqs[b];
    const int kt = blockIdx.y;                                   // key tile of the stream
    const int n_keys = summ ? sq.n_summ : sq.n_text;
    if (kt * kBT >= n_keys) return;
    const int n_qt = (sq.n_text + kBT - 1) / kBT;
    // query tiles that can see this key tile (Eq. 3)
    int qt_lo, qt_hi;
    if (!summ) {
        const int key_last = min(n_keys, kt * kBT + kBT) - 1;
        qt_lo = kt;
        const long long i_max = ((long long)(key_last / a.k) + a.C + 1) * a.k - 1;
        qt_hi = (int)min((long long)(n_qt - 1), i_max / kBT);
    } else {
        // summary row u is visible to rows with (i/k - C) * m > u
        const long long i_min = ((long long)(kt * kBT) / a.m + 1 + a.C) * a.k;
        if (i_min >= sq.n_text) return;
        qt_lo = (int)(i_min / kBT);
        qt_hi = n_qt - 1;
    }
    const int seg0 = qt_lo + (int)blockIdx.x * kSegTiles;
    const int seg1 = min(qt_hi + 1, seg0 + kSegTiles);
    if (seg0 > qt_hi) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g0 = lane >> 2, c2 = (lane & 3) * 2, mi = lane >> 3, r8 = lane & 7;
    const uint32_t sK = bsm_u32(bsm), sV = sK + kTileB;          // this CTA's keys
    const uint32_t sQ = sV + kTileB, sG = sQ + 2 * kTileB;       // two stages of Q and dO tiles
    float* s_lse = reinterpret_cast<float*>(bsm + 6 * kTileB);   // [2][64] lse, delta and Eq. 3 bound of the query tile
    float* s_dl = s_lse + 2 * kBT;
    int* s_bnd = reinterpret_cast<int*>(s_dl + 2 * kBT);         // text keys: first visible row; summary keys: visible count

    const size_t krow0 = summ ? ((size_t)hk * a.summ_rows + sq.summ_off + (size_t)kt * kBT)
                              : ((size_t)hk * a.text_rows + sq.text_off + (size_t)kt * kBT);
    load_tile64<D>(sK, (summ ? a.ks : a.kt) + krow0 * D, threadIdx.x, 128);
    load_tile64<D>(sV, (summ ? a.vs : a.vt) + krow0 * D, threadIdx.x, 128);
    const int iters = (seg1 - seg0) * G;
    auto issue_tiles = [&](int it) {
        const int qt = seg0 + it / G, h = hk * G + it % G;
        const size_t r = (size_t)h * a.text_rows + sq.text_off + (size_t)qt * kBT;
        load_tile64<D>(sQ + (it & 1) * kTileB, a.qt + r * D, threadIdx.x, 128);
        load_tile64<D>(sG + (it & 1) * kTileB, a.dot + r * D, threadIdx.x, 128);
    };
    issue_tiles(0);
    b_cp_commit();

    float dk[D / 8][4], dv[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f; dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f; }
    // this thread's two keys (rows g0 and g0 + 8 of the warp's 16 keys), in stream coordinates
    const int key_a = kt * kBT + warp * 16 + g0, key_b = key_a + 8;

    for (int it = 0; it < iters; ++it) {
        if (it + 1 < iters) issue_tiles(it + 1);
        b_cp_commit();
        const int qt = seg0 + it / G, h = hk * G + it % G;
        const size_t r = (size_t)h * a.text_rows + sq.text_off + (size_t)qt * kBT;
        if (threadIdx.x < kBT) {
            const int i = qt * kBT + threadIdx.x;
            s_lse[(it & 1) * kBT + threadIdx.x] = a.lse_t[r + threadIdx.x];
            s_dl[(it & 1) * kBT + threadIdx.x] = a.delta_t[r + threadIdx.x];
            s_bnd[(it & 1) * kBT + threadIdx.x] = (i >= sq.n_text) ? (summ ? 0 : 0x7fffffff)
                                                                   : (summ ? eq3_cnt(a, i, sq.n_summ) : eq3_lo(a, i));
        }
        b_cp_wait<1>();
        __syncthreads();
        const uint32_t sq_ = sQ + (it & 1) * kTileB, sg_ = sG + (it & 1) * kTileB;
        const float* lse_q = s_lse + (it & 1) * kBT;
        const float* dl_q = s_dl + (it & 1) * kBT;
        const int* bnd_q = s_bnd + (it & 1) * kBT;
        // S^T = K Q^T and dP^T = V dO^T : A = this warp's 16 keys (from smem), B = the 64 queries
        float st[8][4], dpt[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { st[nt][0] = st[nt][1] = st[nt][2] = st[nt][3] = 0.f; dpt[nt][0] = dpt[nt][1] = dpt[nt][2] = dpt[nt][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t ka[4], va[4];
            {
                const int row = warp * 16 + (mi & 1) * 8 + r8, chunk = kk * 2 + (mi >> 1);
                b_ldsm4(ka, tile_addr<D>(sK, row, chunk));
                b_ldsm4(va, tile_addr<D>(sV, row, chunk));
            }
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t qb[4], gb[4];
                const int qrow = np * 16 + (mi >> 1) * 8 + r8, chunk = kk * 2 + (mi & 1);
                b_ldsm4(qb, tile_addr<D>(sq_, qrow, chunk));
                b_ldsm4(gb, tile_addr<D>(sg_, qrow, chunk));
                b_mma(st[2 * np], ka, qb[0], qb[1]);  b_mma(st[2 * np + 1], ka, qb[2], qb[3]);
                b_mma(dpt[2 * np], va, gb[0], gb[1]); b_mma(dpt[2 * np + 1], va, gb[2], gb[3]);
            }
        }
        // P^T and dS^T as A fragments (rows: keys, k-dimension: queries)
        uint32_t pa[4][4], dsa[4][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float pv[4], ds[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int qi = nt * 8 + c2 + (e & 1);                  // query row within the tile
                const int i = qt * kBT + qi;
                const int key = (e >= 2) ? key_b : key_a;
                const bool vis = summ ? (key < bnd_q[qi]) : (key <= i && key >= bnd_q[qi]);
                const float p = vis ? b_ex2(st[nt][e] * a.scale_log2 - lse_q[qi]) : 0.f;
                pv[e] = p;
                ds[e] = p * (dpt[nt][e] - dl_q[qi]);
            }
            pa[nt >> 1][(nt & 1) * 2 + 0] = b_pack2(pv[0], pv[1]);
            pa[nt >> 1][(nt & 1) * 2 + 1] = b_pack2(pv[2], pv[3]);
            dsa[nt >> 1][(nt & 1) * 2 + 0] = b_pack2(ds[0], ds[1]);
            dsa[nt >> 1][(nt & 1) * 2 + 1] = b_pack2(ds[2], ds[3]);
        }
        // dV += P^T dO, dK += dS^T Q   (k-steps of 16 queries; B = dO / Q [query, d] through transposing loads)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int n2 = 0; n2 < D / 16; ++n2) {
                uint32_t gb[4], qb[4];
                const int qrow = ks * 16 + (mi & 1) * 8 + r8, chunk = n2 * 2 + (mi >> 1);
                b_ldsm4t(gb, tile_addr<D>(sg_, qrow, chunk));
                b_ldsm4t(qb, tile_addr<D>(sq_, qrow, chunk));
                b_mma(dv[2 * n2], pa[ks], gb[0], gb[1]);  b_mma(dv[2 * n2 + 1], pa[ks], gb[2], gb[3]);
                b_mma(dk[2 * n2], dsa[ks], qb[0], qb[1]); b_mma(dk[2 * n2 + 1], dsa[ks], qb[2], qb[3]);
            }
        }
        __syncthreads();
    }
    b_cp_wait<0>();
    // add this segment's partial sums to the fp32 accumulators of the stream
    float* acc_k = (summ ? a.dks : a.dkt) + krow0 * D;
    float* acc_v = (summ ? a.dvs : a.dvt) + krow0 * D;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int rr = warp * 16 + g0 + half * 8;
        if (kt * kBT + rr >= n_keys) continue;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            float* pk = acc_k + (size_t)rr * D + nt * 8 + c2;
            float* pv = acc_v + (size_t)rr * D + nt * 8 + c2;
            atomicAdd(reinterpret_cast<float2*>(pk), make_float2(dk[nt][half * 2] * a.scale, dk[nt][half * 2 + 1] * a.scale));
            atomicAdd(reinterpret_cast<float2*>(pv), make_float2(dv[nt][half * 2], dv[nt][half * 2 + 1]));
        }
    }
}

// =================================================================================================
// preparation: text rows of dO into the packed layout (not in direct mode), lse in log2 units, delta = <dO, O>
// =================================================================================================
__global__ void __launch_bounds__(256) ksa_bwd_prep_kernel(BwdArgs a)
{
    // One 16-byte vector (8 elements) per lane: D / 8 lanes make up a (row, head) unit, a warp holds 32 / (D / 8)
    // units (consecutive heads of one row first: those are contiguous in dout / out).
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int lane = threadIdx.x & 31;
    const int lanes_per_unit = a.D / 8, units_per_warp = 32 / lanes_per_unit;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t unit = warp * units_per_warp + lane / lanes_per_unit;
    const int sub = lane % lanes_per_unit;
    const bool live = unit < (int64_t)sq.text_pad * a.Hq;
    const int i = live ? (int)(unit / a.Hq) : 0, h = live ? (int)(unit % a.Hq) : 0;
    const size_t prow = (size_t)h * a.text_rows + sq.text_off + i;
    float d = 0.f;
    float lse2 = INFINITY;
    uint4 gv = make_uint4(0u, 0u, 0u, 0u);
    const bool real = live && i < sq.n_text;
    if (real) {
        const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * (a.k + a.m) + (i % a.k);
        gv = *reinterpret_cast<const uint4*>(a.dout + aug * a.do_st + (int64_t)h * a.do_sh + sub * 8);
        const uint4 ov = *reinterpret_cast<const uint4*>(a.out + aug * a.o_st + (int64_t)h * a.o_sh + sub * 8);
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, ow[4] = {ov.x, ov.y, ov.z, ov.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            d = fmaf(__uint_as_float(gw[e] << 16), __uint_as_float(ow[e] << 16), d);
            d = fmaf(__uint_as_float(gw[e] & 0xffff0000u), __uint_as_float(ow[e] & 0xffff0000u), d);
        }
        if (sub == 0) lse2 = a.lse[(int64_t)h * a.total_aug + aug] * 1.4426950408889634f;
    }
    // sum over the lanes of the unit (whole warps take part: no early exit above)
    for (int s = lanes_per_unit >> 1; s > 0; s >>= 1) d += __shfl_xor_sync(0xffffffffu, d, s);
    if (!live) return;
    if (!a.direct) *reinterpret_cast<uint4*>(a.dot + prow * a.D + sub * 8) = gv;        // zeros on padding rows
    if (sub == 0) { a.lse_t[prow] = lse2; a.delta_t[prow] = real ? d : 0.f; }
}

// =================================================================================================
// summary query rows (Sec. 2.2.1): one warp per (summary row, query head), at most k + m keys
// =================================================================================================
template <int D>
__global__ void __launch_bounds__(256) ksa_bwd_summary_kernel(BwdArgs a)
{
    constexpr int E = D / 32;
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp >= (int64_t)sq.n_summ * a.Hq) return;
    const int u = (int)(warp / a.Hq), h = (int)(warp % a.Hq);
    const int hk = h / (a.Hq / a.Hkv);
    const int j = u / a.m, r = u - j * a.m, s = a.k + a.m;
    const int64_t key0 = sq.aug_off + (int64_t)j * s, qrow = key0 + a.k + r;
    const int nk = a.k + ((a.flags & 1u) ? 0 : (r + 1));
    float qv[E], gv[E], dqv[E];
    float delta = 0.f;
    {
        const uint16_t* qp = a.q + qrow * a.q_st + (int64_t)h * a.q_sh + lane * E;
        const uint16_t* gp = a.dout + qrow * a.do_st + (int64_t)h * a.do_sh + lane * E;
        const uint16_t* op = a.out + qrow * a.o_st + (int64_t)h * a.o_sh + lane * E;
#pragma unroll
        for (int e = 0; e < E; ++e) { qv[e] = b_bf2f(qp[e]); gv[e] = b_bf2f(gp[e]); dqv[e] = 0.f; delta = fmaf(gv[e], b_bf2f(op[e]), delta); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) delta += __shfl_xor_sync(0xffffffffu, delta, o);
    const float lse = a.lse[(int64_t)h * a.total_aug + qrow];
    for (int t = 0; t < nk; ++t) {
        const uint16_t* kp = a.kx + (key0 + t) * a.k_st + (int64_t)hk * a.k_sh + lane * E;
        const uint16_t* vp = a.v + (key0 + t) * a.v_st + (int64_t)hk * a.v_sh + lane * E;
        float kf[E], dot = 0.f, dp = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) { kf[e] = b_bf2f(kp[e]); dot = fmaf(qv[e], kf[e], dot); dp = fmaf(gv[e], b_bf2f(vp[e]), dp); }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { dot += __shfl_xor_sync(0xffffffffu, dot, o); dp += __shfl_xor_sync(0xffffffffu, dp, o); }
        const float p = __expf(dot * a.scale - lse);
        const float ds = p * (dp - delta) * a.scale;
        // accumulator row of key t: text rows of the chunk, then the chunk's own summaries
        float* ak; float* av;
        if (t < a.k) {
            const size_t row = (size_t)hk * a.text_rows + sq.text_off + (size_t)j * a.k + t;
            ak = a.dkt + row * D; av = a.dvt + row * D;
        } else {
            const size_t row = (size_t)hk * a.summ_rows + sq.summ_off + (size_t)j * a.m + (t - a.k);
            ak = a.dks + row * D; av = a.dvs + row * D;
        }
#pragma unroll
        for (int e = 0; e < E; e += 2) {
            atomicAdd(reinterpret_cast<float2*>(ak + lane * E + e), make_float2(ds * qv[e], ds * qv[e + 1]));
            atomicAdd(reinterpret_cast<float2*>(av + lane * E + e), make_float2(p * gv[e], p * gv[e + 1]));
            dqv[e] = fmaf(ds, kf[e], dqv[e]); dqv[e + 1] = fmaf(ds, kf[e + 1], dqv[e + 1]);
        }
    }
    uint16_t* dp_ = a.dq + qrow * a.dq_st + (int64_t)h * a.dq_sh + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2) *reinterpret_cast<uint32_t*>(dp_ + e) = b_pack2(dqv[e], dqv[e + 1]);
}

// =================================================================================================
// finish: fp32 accumulators of the streams -> bf16 dk, dv at the augmented positions (Eq. 1)
// =================================================================================================
__global__ void __launch_bounds__(256) ksa_bwd_finish_kernel(BwdArgs a)
{
    const SeqInfo sq = a.seqs[blockIdx.y];
    const bool text = (blockIdx.z == 0);
    const int vecs = a.D / 8;
    const int live = text ? sq.n_text : sq.n_summ;
    const int64_t per_row = (int64_t)a.Hkv * vecs;
    const int64_t total = (int64_t)live * per_row;
    const int s = a.k + a.m;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int row = (int)(idx / per_row);
        const int rem = (int)(idx - (int64_t)row * per_row);
        const int hk = rem / vecs, vv = rem - hk * vecs;
        const int64_t aug = text ? sq.aug_off + (int64_t)(row / a.k) * s + (row % a.k)
                                 : sq.aug_off + (int64_t)(row / a.m) * s + a.k + (row % a.m);
        const size_t srow = text ? ((size_t)hk * a.text_rows + sq.text_off + row) : ((size_t)hk * a.summ_rows + sq.summ_off + row);
        const float* fk = (text ? a.dkt : a.dks) + srow * a.D + vv * 8;
        const float* fv = (text ? a.dvt : a.dvs) + srow * a.D + vv * 8;
        uint4 ok, ov;
        ok.x = b_pack2(fk[0], fk[1]); ok.y = b_pack2(fk[2], fk[3]); ok.z = b_pack2(fk[4], fk[5]); ok.w = b_pack2(fk[6], fk[7]);
        ov.x = b_pack2(fv[0], fv[1]); ov.y = b_pack2(fv[2], fv[3]); ov.z = b_pack2(fv[4], fv[5]); ov.w = b_pack2(fv[6], fv[7]);
        *reinterpret_cast<uint4*>(a.dk + aug * a.dk_st + (int64_t)hk * a.dk_sh + vv * 8) = ok;
        *reinterpret_cast<uint4*>(a.dv + aug * a.dv_st + (int64_t)hk * a.dv_sh + vv * 8) = ov;
    }
}

// =================================================================================================
// launchers
// =================================================================================================
template <int D> constexpr int bwd_dq_smem() { return 6 * kBT * D * 2; }
template <int D> constexpr int bwd_dkv_smem() { return 6 * kBT * D * 2 + 6 * kBT * 4; }

cudaError_t setup_bwd()
{
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(ksa_bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bwd_dq_smem<128>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(ksa_bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, bwd_dq_smem<64>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(ksa_bwd_dkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bwd_dkv_smem<128>())) != cudaSuccess) return e;
    return cudaFuncSetAttribute(ksa_bwd_dkv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, bwd_dkv_smem<64>());
}

cudaError_t launch_bwd_prep(const BwdArgs& a, cudaStream_t stream)
{
    const int64_t units = (int64_t)a.max_text_pad * a.Hq;                // (row, head) units, 32 / (D / 8) per warp
    const int64_t warps = (units * (a.D / 8) + 31) / 32;
    dim3 grid((unsigned)((warps + 7) / 8), (unsigned)a.num_seqs, 1);
    ksa_bwd_prep_kernel<<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_bwd_summary(const BwdArgs& a, cudaStream_t stream)
{
    if (a.m <= 0 || a.max_n_summ <= 0) return cudaSuccess;
    if (bwd_summary_mma_applies(a)) return launch_bwd_summary_mma(a, stream);
    const int64_t warps = (int64_t)a.max_n_summ * a.Hq;
    dim3 grid((unsigned)((warps + 7) / 8), (unsigned)a.num_seqs, 1);
    if (a.D == 128) ksa_bwd_summary_kernel<128><<<grid, 256, 0, stream>>>(a);
    else            ksa_bwd_summary_kernel<64><<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_bwd_dq(const BwdArgs& a, cudaStream_t stream)
{
    dim3 grid((unsigned)(a.max_text_pad / kBT), (unsigned)a.Hq, (unsigned)a.num_seqs);
    if (a.D == 128) ksa_bwd_dq_kernel<128><<<grid, 128, bwd_dq_smem<128>(), stream>>>(a);
    else            ksa_bwd_dq_kernel<64><<<grid, 128, bwd_dq_smem<64>(), stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_bwd_dkv(const BwdArgs& a, cudaStream_t stream)
{
    const int n_qt = a.max_text_pad / kBT;
    // text keys are seen by at most (C + 1) k / 64 + 2 query tiles, summary keys by up to all of them
    const long long text_span = std::min<long long>(n_qt, ((long long)a.C + 1) * a.k / kBT + 2);
    for (int summ = 0; summ < 2; ++summ) {
        if (summ && (a.m <= 0 || a.max_n_summ <= 0)) continue;
        const long long span = summ ? n_qt : text_span;
        const int tiles = summ ? (a.max_n_summ + kBT - 1) / kBT : n_qt;
        dim3 grid((unsigned)((span + kSegTiles - 1) / kSegTiles), (unsigned)tiles, (unsigned)(a.num_seqs * a.Hkv));
        if (a.D == 128) ksa_bwd_dkv_kernel<128><<<grid, 128, bwd_dkv_smem<128>(), stream>>>(a, summ);
        else            ksa_bwd_dkv_kernel<64><<<grid, 128, bwd_dkv_smem<64>(), stream>>>(a, summ);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_bwd_finish(const BwdArgs& a, cudaStream_t stream)
{
    const int64_t per_row = (int64_t)a.Hkv * (a.D / 8);
    const int64_t rows = a.max_text_pad > a.max_summ_pad ? a.max_text_pad : a.max_summ_pad;
    int64_t blocks = (rows * per_row + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    dim3 grid((unsigned)blocks, (unsigned)a.num_seqs, a.m > 0 ? 2u : 1u);
    ksa_bwd_finish_kernel<<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace ksa
