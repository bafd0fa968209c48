/*
 * ksa_oracle.h -- plain CPU oracle for Kwai Summary Attention (KSA) forward.
 *
 * TEST INFRASTRUCTURE ONLY.  This library is the slow, obviously-correct statement
 * of what the KSA attention operator computes.  It exists so that tests, the smoke
 * check and the benchmark's CPU-baseline leg can compare the CUDA library against
 * it.  Nothing in the product path may call it, and it shares no code, header,
 * table or helper with the CUDA library.
 *
 * What it follows:
 *   - Eq. 1 (summary token compression): the augmented sequence is
 *     chunk_0, chunk_1, ... with chunk_j = [t_{jk}, ..., t_{jk+k-1}, s_j].
 *   - Eq. 3 (KSA scope): text token i (chunk c = floor(i/k)) sees the summaries
 *     s_0 .. s_{c-C-1} and the text tokens t_{(c-C)k} .. t_i; summaries inside the
 *     sliding-chunk window are not visible to text.
 *   - Sec. 2.2.1, bullet 1: a summary token sees the text tokens of its own chunk
 *     and nothing else (optionally itself, see KSA_ORACLE_SUMMARY_TEXT_ONLY).
 *   - The student attention equation of Sec. 4.1.4:
 *     O = softmax(Q K^T * scale + M_KSA) V with M_KSA in {0, -inf}.
 *
 * Readings taken where the paper is silent (each is pinned by a CPU test):
 *   - Summary self-visibility: by default a summary token also sees itself (the
 *     decode procedure of Sec. 2.3.1 attends over [summary self-KV, chunk text]);
 *     KSA_ORACLE_SUMMARY_TEXT_ONLY gives the strict "text of its chunk only" rule.
 *   - m > 1 summaries per chunk (not in the paper): they follow the k text tokens
 *     in order r = 0..m-1; summary r sees its chunk's text and summaries 0..r of
 *     its own chunk; text sees all m summaries of every distant chunk.
 *   - n not divisible by k: the trailing partial chunk has no summary token
 *     (Sec. 2.3.1 emits a summary only when a chunk is filled).
 *   - c - C < 0 is clamped to chunk 0 (window starts at t_0, no visible summary).
 *   - LSE is the natural log of sum_j exp(scale * <q, k_j>) over visible keys.
 *
 * All functions are pure and thread-safe.  Tensors are HOST memory.
 */
#ifndef KSA_ORACLE_H
#define KSA_ORACLE_H
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

#define KSA_ORACLE_SUMMARY_TEXT_ONLY 1u

/* Eq. 1: augmented length of one sequence, n + floor(n/k)*m. */
int64_t ksa_oracle_aug_len(int64_t n_text, int32_t k, int32_t m);

/* Eq. 1: decode augmented position p of a sequence with n_text text tokens.
 * Returns 0 on success, -1 if p is out of range.
 * *is_summary = 0: *index = text token index i.  *is_summary = 1: *index = chunk j,
 * *r = summary slot within the chunk. */
int ksa_oracle_decode_pos(int64_t n_text, int32_t k, int32_t m, int64_t p,
                          int32_t* is_summary, int64_t* index, int32_t* r);

/* Visibility predicate between two augmented positions of the SAME sequence
 * (query pq, key pk).  Returns 1 visible, 0 masked, -1 bad argument. */
int ksa_oracle_visible(int64_t n_text, int32_t k, int32_t m, int32_t C, uint32_t flags,
                       int64_t pq, int64_t pk);

/* Explicit mask row: row[pk] = visible(pq, pk) for every pk in [0, L).  Returns L or -1. */
int64_t ksa_oracle_mask_row(int64_t n_text, int32_t k, int32_t m, int32_t C, uint32_t flags,
                            int64_t pq, uint8_t* row);

/* Number of set entries of the explicit mask row of pq (built, then counted). */
int64_t ksa_oracle_visible_count(int64_t n_text, int32_t k, int32_t m, int32_t C,
                                 uint32_t flags, int64_t pq);

/* Sum of ksa_oracle_visible_count over every augmented row of every sequence. */
int64_t ksa_oracle_total_pairs(int32_t num_seqs, const int32_t* cu_text_lens, int32_t k,
                               int32_t m, int32_t C, uint32_t flags);

/*
 * KSA attention forward in fp64 from bf16 inputs.
 *   q        [total_aug, Hq,  D] bf16 bit patterns (uint16), packed sequences back to back
 *   kk, v    [total_aug, Hkv, D] bf16 bit patterns
 *   cu_text_lens[num_seqs+1]     prefix sums of the sequences' TEXT lengths
 *   rows     optional list of n_rows global augmented row indices to evaluate
 *            (NULL: all total_aug rows, n_rows ignored)
 *   out      [R, Hq, D] fp64, lse [R, Hq] fp64, R = n_rows or total_aug
 *   count    optional [R] int64: visible keys of each evaluated row (may be NULL)
 * Query head h uses KV head floor(h / (Hq/Hkv)).
 * Returns 0, or -1 on bad arguments.
 */
int ksa_oracle_fwd(const uint16_t* q, const uint16_t* kk, const uint16_t* v,
                   int32_t num_seqs, const int32_t* cu_text_lens,
                   int32_t k, int32_t m, int32_t C,
                   int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                   const int64_t* rows, int64_t n_rows,
                   double* out, double* lse, int64_t* count);

/*
 * Gradients of the same operator (what a training step needs; Sec. 2.3 calls the block-sparse
 * kernel the one "for training and prefill"), in fp64 from bf16 inputs.  With p_ij the softmax
 * weights of row i over its visible keys, o_i = sum_j p_ij v_j and dO given:
 *   dV_j = sum_i p_ij dO_i            dP_ij = <dO_i, v_j>          delta_i = <dO_i, o_i>
 *   dS_ij = p_ij (dP_ij - delta_i)    dQ_i = scale sum_j dS_ij k_j  dK_j = scale sum_i dS_ij q_i
 * (the textbook gradient of softmax(scale Q K^T + M) V; sums over i run over the rows that see j,
 * and for grouped heads dK, dV add up the G query heads of a KV head).
 *   q, kk, v, cu_text_lens, k, m, C, Hq, Hkv, D, scale, flags   as in ksa_oracle_fwd
 *   dout   [total_aug, Hq, D] bf16 bit patterns
 *   dq     [total_aug, Hq, D] fp64;  dk, dv [total_aug, Hkv, D] fp64 (every entry written)
 * Returns 0, or -1 on bad arguments.
 */
int ksa_oracle_bwd(const uint16_t* q, const uint16_t* kk, const uint16_t* v, const uint16_t* dout,
                   int32_t num_seqs, const int32_t* cu_text_lens,
                   int32_t k, int32_t m, int32_t C,
                   int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                   double* dq, double* dk, double* dv);

/* The same gradients on a sample of rows (for inputs too long to differentiate in full): dq [nq, Hq, D] of the
 * query rows q_rows (global augmented rows), dk and dv [nk, Hkv, D] of the key rows k_rows -- the latter summed
 * over every query row of the key's sequence that sees the key, each with its complete softmax over its explicit
 * mask row.  Same arithmetic as ksa_oracle_bwd.  Returns 0, -1 on bad arguments, -2 if out of memory. */
int ksa_oracle_bwd_rows(const uint16_t* q, const uint16_t* kk, const uint16_t* v, const uint16_t* dout,
                        int32_t num_seqs, const int32_t* cu_text_lens,
                        int32_t k, int32_t m, int32_t C,
                        int32_t Hq, int32_t Hkv, int32_t D, double scale, uint32_t flags,
                        const int64_t* q_rows, int64_t nq, double* dq,
                        const int64_t* k_rows, int64_t nk, double* dk, double* dv);

/* Threads the OpenMP loops will use. */
int ksa_oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
