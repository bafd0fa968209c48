/*
 * ksa_decode.h -- C ABI of the decode path: the Summary KV cache of Sec. 2.3.1 and one
 * auto-regressive attention step over it.
 *
 * The cache of one (sequence, KV head) is ONE contiguous run of rows (K and V in two
 * tensors of the same shape), laid out so that every read of a decode step is a single
 * contiguous slice and the layout itself encodes the visibility rule of Eq. 3:
 *
 *   row 0                      scratch slot (the chunk summary's own K/V while it attends)
 *   rows 1 .. k                Current Chunk, filled right to left: token o of the chunk
 *                              (o = 0..k-1) sits at row k - o
 *   rows 1+k .. k+C*k          Sliding Chunk Text, a ring of C chunk slots: chunk c lives in
 *                              slot c mod C (its k rows in the order it had in Current Chunk)
 *   rows 1+k+C*k ..            Summary Token Buffer, grows to the right: summary of chunk j
 *                              at row 1 + k + C*k + j
 *
 *   text token i (chunk c = floor(i/k), offset o = i mod k) attends, after its own K/V was
 *   written, to rows [k - o, 1 + k + min(c, C)*k + max(0, c - C)): the filled part of
 *   Current Chunk, the chunks c-C..c-1 in the ring and the summaries s_0..s_{c-C-1} --
 *   exactly the set of Eq. 3.  The summary token of chunk c attends to rows [0, 1+k)
 *   (itself and its chunk's text; [1, 1+k) under KSA_FLAG_SUMMARY_TEXT_ONLY).
 *
 * One summary per chunk (the paper's layout).  K is cached as it is given (RoPE is the
 * caller's business, as the paper applies it before caching).  Softmax is order-free, so
 * the reversed order inside a chunk and the ring order do not matter.
 *
 * Tensors (DEVICE, bf16 unless said otherwise, 16-byte aligned, contiguous):
 *   kcache, vcache : [batch, num_kv_heads, rows, head_dim], rows = ksa_cache_rows()
 *   state          : int32 [batch, 2]: text tokens cached, summaries inserted
 *   q, out         : [batch, num_q_heads, head_dim];  k_new, v_new : [batch, num_kv_heads, head_dim]
 *   lse            : fp32 [batch, num_q_heads], natural log of the softmax denominator
 * All calls are asynchronous on the given stream; nothing synchronises the host.
 */
#ifndef KSA_DECODE_H
#define KSA_DECODE_H

#include "ksa.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t  struct_size;        /* sizeof(ksa_cache_params) */
    int32_t  batch;              /* sequences decoded together, >= 1 */
    int32_t  chunk_len;          /* k >= 1 */
    int32_t  window_chunks;      /* C >= 0 */
    int32_t  max_summaries;      /* capacity of the Summary Token Buffer: floor(max context / k) */
    int32_t  num_q_heads, num_kv_heads;   /* group size G = num_q_heads / num_kv_heads <= 16 */
    int32_t  head_dim;           /* 64 or 128 */
    float    softmax_scale;
    uint32_t flags;              /* KSA_FLAG_SUMMARY_TEXT_ONLY */
} ksa_cache_params;

/* Rows of one (sequence, KV head) cache: 1 + k + C*k + max_summaries, or < 0 on bad parameters. */
int64_t ksa_cache_rows(const ksa_cache_params* p);
/* Bytes of kcache (= bytes of vcache), of the state array and of the decode workspace. */
int ksa_cache_bytes(const ksa_cache_params* p, size_t* cache_bytes, size_t* state_bytes, size_t* workspace_bytes);
/* The contiguous slice [*row_lo, *row_hi) a decode step reads (Sec. 2.3.1), on the host:
 * for is_summary == 0, the text token that is number `text_tokens_before` (0-based) of its
 * sequence; for is_summary != 0, the summary of the chunk completed by `text_tokens_before`
 * cached tokens (which must be a positive multiple of k). */
int ksa_cache_slice(const ksa_cache_params* p, int64_t text_tokens_before, int is_summary, int64_t* row_lo, int64_t* row_hi);

/* Empties every sequence's cache (state := 0). */
int ksa_cache_reset(ksa_ctx* ctx, int32_t* state, const ksa_cache_params* p, void* cuda_stream);
/*
 * Builds the caches from the K/V of a prefill: k, v are the augmented tensors ksa_attn_fwd
 * takes (layout `prefill`, with summaries_per_chunk == 1, chunk_len / window / heads equal to
 * the cache's, num_seqs == batch).  Afterwards the state equals that of having decoded every
 * token one by one; a sequence whose length is a multiple of k has its last summary inserted.
 */
int ksa_cache_fill_from_prefill(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* k, const void* v,
                                const ksa_params* prefill, const ksa_cache_params* p, void* cuda_stream);
/*
 * One text-token step for every sequence of the batch (Sec. 2.3.1, "Updating the current text
 * chunk"): writes k_new / v_new into the next slot of Current Chunk, attends over the slice,
 * writes out / lse and advances the state.  A sequence whose chunk is full and still waits for
 * its summary (or whose summary buffer is full) is skipped and the device status word of the
 * context is set to KSA_DECODE_STATUS_PENDING_SUMMARY / _FULL; its out row is left untouched.
 * workspace: DEVICE, >= workspace_bytes of ksa_cache_bytes, 256-byte aligned, scratch.
 */
int ksa_decode_text(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* q, const void* k_new,
                    const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                    const ksa_cache_params* p, void* cuda_stream);
/*
 * The summary step ("Chunk eviction and summary token insertion") for every sequence whose
 * current chunk has just been filled: (i) the summary's K/V go to the scratch slot and it
 * attends over [scratch, chunk text]; (ii) the chunk is copied into the ring slot c mod C;
 * (iii) the summary K/V are appended to the Summary Token Buffer.  Sequences that are not due
 * are skipped (out untouched).  Same tensor shapes as ksa_decode_text.
 */
int ksa_decode_summary(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* q, const void* k_new,
                       const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                       const ksa_cache_params* p, void* cuda_stream);

#define KSA_DECODE_STATUS_PENDING_SUMMARY  101   /* a text step met a full chunk without its summary */
#define KSA_DECODE_STATUS_FULL             102   /* the Summary Token Buffer has no room left        */

#ifdef __cplusplus
}
#endif
#endif /* KSA_DECODE_H */
