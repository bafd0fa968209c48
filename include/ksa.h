/*
 * ksa.h -- C ABI of the B200 (sm_100a) Kwai Summary Attention forward library.
 *
 * The library computes the KSA attention operator of the paper,
 *     O = softmax(Q K^T * scale + M_KSA) V          (student attention equation, Sec. 4.1.4)
 * over the augmented sequence of Eq. 1 (k text tokens followed by the chunk's summary
 * token(s), chunk after chunk), with the visibility mask M_KSA of Eq. 3 for text
 * rows and the "own chunk only" rule of Sec. 2.2.1 for summary rows, without ever
 * materialising the mask: a block-sparse schedule lists, per query tile, only the
 * key/value tiles that hold at least one visible pair (the block-sparse training /
 * prefill kernel of Sec. 2.3).
 *
 * Conventions
 *   - Every function returns an int status: KSA_OK (0) or a negative KSA_ERR_* code.
 *     Nothing throws, aborts or prints.  Invalid arguments never launch a kernel.
 *   - "HOST" / "DEVICE" in a comment says where a pointer must live.
 *   - The caller owns every buffer it passes (q, k, v, out, lse, workspace); the
 *     library neither frees nor keeps them beyond the completion of the stream work
 *     it enqueued.  A ksa_ctx owns only its cached schedule and a few small device
 *     tables, which ksa_destroy releases.
 *   - ksa_attn_fwd is asynchronous on the given CUDA stream and performs no host
 *     synchronisation once the schedule for the given lengths is cached (the first
 *     call with a new set of lengths builds and uploads it with a blocking copy).
 *     The same holds for ksa_attn_bwd, ksa_attn_fwd_part and ksa_qkv_prepare: after
 *     that first call they may be recorded into a CUDA graph (stream capture) and
 *     replayed on the same buffers.
 *   - There is no CPU fallback: on a machine without an sm_100 device ksa_create fails.
 *
 * Layout of one packed batch (Eq. 1, generalised to m summaries per chunk):
 *   sequence b has n_b text tokens, J_b = floor(n_b / k) full chunks and
 *   L_b = n_b + J_b * m augmented rows; chunk j occupies rows j*(k+m) .. j*(k+m)+k+m-1
 *   (k text rows, then m summary rows); a trailing partial chunk has text rows only.
 *   Sequences are stored back to back: total_aug = sum_b L_b rows.
 *   q, out : [total_aug, num_q_heads,  head_dim] bf16 (strides given in elements)
 *   k, v   : [total_aug, num_kv_heads, head_dim] bf16
 *   lse    : [num_q_heads, total_aug] fp32, natural log of sum_j exp(scale * <q, k_j>)
 *            over the row's visible keys.
 *   Query head h reads KV head floor(h / (num_q_heads / num_kv_heads)).
 */
#ifndef KSA_H
#define KSA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------------------- */
#define KSA_OK                 0
#define KSA_ERR_INVALID_ARG   -1   /* null pointer, k < 1, m < 0, C < 0, bad lengths/strides/alignment */
#define KSA_ERR_UNSUPPORTED   -2   /* head_dim not 64/128, device is not sm_100, limits exceeded (more than 65,535 sequences, 1,024 query heads, 2^30 packed rows) */
#define KSA_ERR_WORKSPACE     -3   /* workspace missing or smaller than ksa_workspace_bytes            */
#define KSA_ERR_CUDA          -4   /* a CUDA runtime/driver call failed (see ksa_last_cuda_error)      */
#define KSA_ERR_TIMEOUT       -5   /* a bounded device-side wait gave up (see ksa_last_device_status)  */
#define KSA_ERR_NOMEM         -6   /* host allocation failed                                           */
#define KSA_ERR_INTERNAL      -7   /* the library's own schedule failed its range check: nothing was launched */

/* ---- flags -------------------------------------------------------------------------- */
/* Summary rows see the text of their own chunk only (strict reading of Sec. 2.2.1).
 * Default (flag clear): summary r of a chunk also sees summaries 0..r of that chunk,
 * itself included, as the decode procedure of Sec. 2.3.1 does. */
#define KSA_FLAG_SUMMARY_TEXT_ONLY   0x1u
/* Run the text rows through the plain CUDA-core cross-check kernel instead of the
 * tensor-core kernel.  Same schedule, same packed streams; slow; for debugging. */
#define KSA_FLAG_REFERENCE_KERNEL    0x2u
/* Run the text rows through the tensor-core kernel that keeps both query heads of a work
 * item in ONE CTA, even where the CTA-pair kernel applies (head_dim 128, an even number of
 * query heads per KV head; with whole-chunk lengths also k | 64 and m | 64).  Same results
 * up to rounding order; for comparison and debugging. */
#define KSA_FLAG_SINGLE_CTA_KERNEL   0x4u
/* Run the text rows through the CTA-pair kernel wherever it applies (see above), whatever the
 * library would pick by itself.  Ignored where it does not apply. */
#define KSA_FLAG_CTA_PAIR_KERNEL     0x8u
/* ksa_attn_bwd only: run dQ and dK / dV of the text rows through the mma.sync kernels (the first
 * version of the backward pass) instead of the tcgen05 kernels.  Same results up to rounding
 * order; several times slower; an on-device cross-check.  Ignored by the other calls. */
#define KSA_FLAG_BWD_MMA_SYNC_KERNELS 0x10u

typedef struct ksa_ctx ksa_ctx;    /* opaque */

/* Problem statement of one forward call. */
typedef struct ksa_params {
    int32_t  struct_size;          /* = sizeof(ksa_params); ABI check                              */
    int32_t  num_seqs;             /* B >= 1 packed sequences                                      */
    const int32_t* cu_text_lens;   /* HOST, B+1 entries: prefix sums of the TEXT lengths, [0] = 0  */
    int32_t  chunk_len;            /* k >= 1 text tokens per chunk (Eq. 1)                         */
    int32_t  summaries_per_chunk;  /* m >= 0 (paper: 1; 0 = sliding chunk attention alone, Eq. 2)  */
    int32_t  window_chunks;        /* C >= 0, the sliding chunk number of Eqs. 2-3                 */
    int32_t  num_q_heads;
    int32_t  num_kv_heads;         /* must divide num_q_heads                                      */
    int32_t  head_dim;             /* 64 or 128; innermost, stride 1                               */
    float    softmax_scale;        /* e.g. 1/sqrt(head_dim)                                        */
    int64_t  q_stride_tok, q_stride_head;   /* element strides; multiples of 8                     */
    int64_t  k_stride_tok, k_stride_head;
    int64_t  v_stride_tok, v_stride_head;
    int64_t  o_stride_tok, o_stride_head;
    uint32_t flags;                /* KSA_FLAG_*                                                   */
    uint32_t reserved;             /* must be 0                                                    */
} ksa_params;

/* One visited (query tile, key/value tile) pair of the schedule (see ksa_schedule_dump).
 * Rows are in per-sequence STREAM coordinates: the text stream of a sequence is its
 * text tokens 0..n-1 in order; the summary stream is its summaries in order
 * (chunk j, slot r) -> j*m + r. */
#define KSA_STREAM_TEXT     0
#define KSA_STREAM_SUMMARY  1
typedef struct ksa_tile_rec {
    int32_t seq;
    int32_t q_stream;              /* KSA_STREAM_TEXT (summary rows are not tiled)                 */
    int32_t q_row0, q_rows;        /* query rows [q_row0, q_row0 + q_rows) of the text stream      */
    int32_t kv_stream;             /* KSA_STREAM_TEXT or KSA_STREAM_SUMMARY                        */
    int32_t kv_row0, kv_rows;      /* in-range key rows of the tile                                */
    int32_t is_full;               /* 1: every (query, key) pair of the rectangle is visible       */
} ksa_tile_rec;

/* ---- context ------------------------------------------------------------------------ */
/* Creates a context bound to CUDA device `cuda_device` (which becomes current on the
 * calling thread).  Fails with KSA_ERR_UNSUPPORTED unless the device is compute
 * capability 10.x, and with KSA_ERR_CUDA if no usable device/driver exists. */
int ksa_create(ksa_ctx** out, int cuda_device);
/* Releases the context's own host and device memory.  Work previously enqueued with
 * this context must have completed.  NULL is accepted. */
int ksa_destroy(ksa_ctx* ctx);

/* ---- layout helpers (host, pure) ------------------------------------------------------ */
/* Eq. 1: augmented length n + floor(n/k)*m of one sequence; -1 on bad arguments. */
int64_t ksa_aug_len(int64_t n_text, int32_t k, int32_t m);
/* Sum of ksa_aug_len over the packed batch described by p; <0 = status code. */
int64_t ksa_total_aug_len(const ksa_params* p);
/* Bytes of DEVICE workspace ksa_attn_fwd needs for p (packed Q/K/V streams, 256-byte
 * aligned sub-buffers).  ctx may be NULL. */
int ksa_workspace_bytes(const ksa_ctx* ctx, const ksa_params* p, size_t* bytes);
/* Visible (query, key) pairs of the whole batch, text and summary rows, per query
 * head (closed form of Eq. 3); visible FLOPs = 4 * head_dim * num_q_heads * pairs. */
int ksa_visible_pairs(const ksa_params* p, int64_t* pairs);

/* ---- forward ------------------------------------------------------------------------ */
/*
 * KSA attention forward (Eq. 3 mask, softmax(QK^T*scale + M)V).
 *   q, k, v   DEVICE bf16, layouts above, 16-byte aligned
 *   out       DEVICE bf16, same shape as q (strides o_stride_*); every row is written
 *   lse       DEVICE fp32 [num_q_heads, total_aug]; every entry is written
 *   workspace DEVICE, >= ksa_workspace_bytes, 256-byte aligned; contents are scratch and
 *             must not be used by other work on other streams while the call runs.  When
 *             every sequence is a whole number of chunks (the paper's assumption) and a
 *             128-row tile is a whole number of chunks (128 % k == 0, 128 % m == 0 or
 *             m == 0), ksa_workspace_bytes is 256 and the workspace is not touched: the
 *             text-row kernel reads its tiles straight from q, k, v through chunked
 *             4-D tensor maps and nothing is packed
 *   cuda_stream  a cudaStream_t (NULL = legacy default stream)
 * Steps enqueued: pack (de-interleave text Q/K/V and summary K/V into dense streams;
 * skipped in the case above), summary-row attention, text-row attention over the
 * scheduled tiles.  In the no-pack case the padding rows of a partial tile hold rows
 * of the following sequence; they are masked, but like any masked row their V values
 * must be finite (a NaN or Inf there would reach the accumulators as 0 * NaN).
 * Errors: KSA_ERR_INVALID_ARG / UNSUPPORTED / WORKSPACE before anything is launched;
 * KSA_ERR_CUDA if a launch fails.  Device-side bounded waits report through
 * ksa_last_device_status after the stream has been synchronised.
 */
int ksa_attn_fwd(ksa_ctx* ctx, const void* q, const void* k, const void* v,
                 void* out, float* lse, void* workspace, size_t workspace_bytes,
                 const ksa_params* p, void* cuda_stream);

/* ---- sequence-parallel parts ----------------------------------------------------------- */
/*
 * The same operator on a contiguous part of the query rows only, so that num_parts processes (one per
 * GPU) can share one long batch: part `part` (0 .. num_parts - 1) computes the rows
 * [*aug_begin, *aug_end) that ksa_part_rows reports -- contiguous, in order, disjoint, covering every
 * row, and cut so that the parts carry about the same number of visible tiles (under Eq. 3 later
 * rows cost more).  A text row only attends to rows at or before its own and a summary row to
 * its own chunk, so the call needs q for its own rows and k, v for the rows [0, *aug_end) -- the
 * exchange step of a sequence-parallel run is an all-gather of k and v (or a gather from the lower
 * ranks).  Tensors, layouts, workspace and errors are those of ksa_attn_fwd (full-size tensors,
 * indexed by global augmented row; rows of out / lse outside the part are not touched; rows of k, v
 * after *aug_end must hold finite values).
 */
int ksa_part_rows(ksa_ctx* ctx, const ksa_params* p, int32_t part, int32_t num_parts, int64_t* aug_begin, int64_t* aug_end);
int ksa_attn_fwd_part(ksa_ctx* ctx, const void* q, const void* k, const void* v, void* out, float* lse,
                      void* workspace, size_t workspace_bytes, const ksa_params* p, int32_t part, int32_t num_parts,
                      void* cuda_stream);

/* ---- backward ----------------------------------------------------------------------- */
/* Bytes of DEVICE workspace ksa_attn_bwd needs for this problem: the fp32 accumulators of dK / dV and two fp32
 * scalars per text row and query head, plus packed copies of q, k, v and dout unless they can be read in place
 * (every sequence a whole number of chunks, 128 a multiple of the chunk length and of the summaries per chunk). */
int ksa_bwd_workspace_bytes(const ksa_ctx* ctx, const ksa_params* p, size_t* bytes);
/*
 * Gradients of ksa_attn_fwd (the kernel of Sec. 2.3 is the one "for training and prefill"):
 * with P the softmax weights of the forward pass (recomputed from q, k and lse),
 *   dV = P^T dO,  dP = dO V^T,  dS = P o (dP - rowsum(dO o O)),  dQ = scale dS K,  dK = scale dS^T Q
 * under the same mask (Eq. 3 for text rows, own chunk for summary rows); for grouped heads dK and
 * dV add up the query heads of their KV head.
 *   q, k, v, out, lse   DEVICE, the tensors given to / written by ksa_attn_fwd (same p)
 *   dout                DEVICE bf16, gradient w.r.t. out, layout and strides of out
 *   dq                  DEVICE bf16, layout and strides of q; every row is written
 *   dk, dv              DEVICE bf16, layouts and strides of k and v; every row is written
 *   workspace           DEVICE, >= ksa_bwd_workspace_bytes, 256-byte aligned, scratch
 * Asynchronous on cuda_stream.  KSA_FLAG_REFERENCE_KERNEL is not accepted here.
 * With every sequence a whole number of chunks (the no-pack case of ksa_attn_fwd) the
 * tensor-core kernels read q, k, v and dout in place: rows of other
 * sequences that share a 128-row tile are masked, so all of these tensors must hold finite
 * values everywhere.
 * Errors as for ksa_attn_fwd.
 */
int ksa_attn_bwd(ksa_ctx* ctx, const void* q, const void* k, const void* v, const void* out, const float* lse,
                 const void* dout, void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes,
                 const ksa_params* p, void* cuda_stream);

/* Bytes of DEVICE staging ksa_attn_fwd_host needs (q, k, v, out, lse images plus the
 * workspace of ksa_attn_fwd). */
int ksa_host_staging_bytes(const ksa_ctx* ctx, const ksa_params* p, size_t* bytes);
/*
 * Same operator with HOST tensors (contiguous [total_aug, H, D]; strides in p are
 * ignored).  The query tiles are cut into about sixteen row chunks in sequence order and
 * pipelined: while one chunk's rows of q, k, v are copied to the device staging buffer
 * (on a copy stream the context owns), the previous chunk is packed and computed on
 * cuda_stream, and the one before that has its rows of out and lse copied back (on a
 * second owned stream).  A chunk needs only keys at or before its own rows (Eq. 3), which
 * earlier stages have uploaded.  Returns after both the last download and cuda_stream's
 * work have completed.  Pinned host memory is needed for the copies to overlap.
 * staging: DEVICE, >= ksa_host_staging_bytes, 256-byte aligned; scratch.
 * The first call creates the two streams and a few events (kept until ksa_destroy).
 */
int ksa_attn_fwd_host(ksa_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                      void* out_host, float* lse_host, void* staging, size_t staging_bytes,
                      const ksa_params* p, void* cuda_stream);

/* ---- forward without device allocation -------------------------------------------------- */
/*
 * (No counterpart in the paper: this is a packaging variant of ksa_attn_fwd.)
 *
 * Some programs that want this operator are not allowed to obtain device memory at the
 * moment they call it: an inference server whose whole GPU has been handed to its own
 * memory pool at start-up, so that a raw cudaMalloc from a plug-in fails or is forbidden
 * by policy; a latency-critical loop that cannot tolerate the device-wide
 * synchronisation cudaMalloc/cudaFree imply; a component that simply has no allocator
 * handle to pass down.  ksa_create (device tables) and the caller-provided workspace of
 * ksa_attn_fwd both presuppose an allocator.  This entry point presupposes none: it
 * needs no context and no workspace, and calls neither cudaMalloc nor cudaFree nor any
 * other allocating routine.  All of its scratch -- the status word of the bounded waits,
 * the sequence table, the work list and the packed Q/K/V streams -- lives in one
 * fixed-size array in the library's device image, KSA_NOALLOC_MAX_SCRATCH_BYTES long,
 * which every GPU that loads the library holds from load until the process exits.
 *
 * Arguments q, k, v, out, lse, p, cuda_stream: exactly as for ksa_attn_fwd, on the
 * CURRENT device; results are identical to ksa_attn_fwd's.
 * Limits and behaviour:
 *   - Problems whose scratch exceeds the array are rejected with KSA_ERR_WORKSPACE
 *     before anything is enqueued.  This entry point ALWAYS packs the text and summary rows
 *     into dense streams (ksa_attn_fwd skips that for whole-chunk batches and then reports
 *     a 256-byte workspace, which is NOT what counts here).  Scratch = 1,280 B + 48 B per
 *     sequence + 48 B per work item (query tiles x pairs of query heads; single heads if
 *     the number of query heads is odd) + the packed streams: 2 * head_dim bytes x
 *     [(num_q_heads + 2 * num_kv_heads) x text rows + 2 * num_kv_heads x summary rows],
 *     each sequence's rows rounded up to a multiple of 128.  Of the five benchmark
 *     workloads only the 1,024-token one fits.
 *   - The first call on each device resolves the array's device address and opts the
 *     kernels into their shared-memory size; make that first call outside any stream
 *     capture.
 *   - The call uploads its tables with cudaMemcpyAsync and waits for the stream once
 *     before launching, so it is not fully asynchronous.
 *   - All calls in a process share the one array per device and the array keeps the
 *     previous call's contents (the call re-zeroes what must start at zero).  Two calls
 *     whose GPU work overlaps -- different streams, or different host threads -- race on
 *     it: serialise them.
 */
#define KSA_NOALLOC_MAX_SCRATCH_BYTES (32u * 1024u * 1024u)
int ksa_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* out, float* lse,
                         const ksa_params* p, void* cuda_stream);
/* The status word of ksa_attn_fwd_noalloc's bounded waits on the CURRENT device (it lives in the
 * fixed array, so no context is needed): a blocking 4-byte copy, no allocation.  *status = 0 and
 * KSA_OK if no wait gave up since the last call started (each call re-zeroes the word before its
 * kernels run, so read it after the stream has finished and before the next call); otherwise the
 * code of the first wait that gave up, and KSA_ERR_TIMEOUT -- out and lse of that call are then
 * not valid.  (No counterpart in the paper.) */
int ksa_noalloc_last_device_status(int32_t* status);

/* ---- schedule inspection ------------------------------------------------------------ */
/*
 * Lists every (query tile, key/value tile) pair the text-row kernel visits for p, in
 * the order: sequence, query tile, summary tiles ascending, text tiles ascending.
 * (Heads share the schedule.)  recs: HOST array of capacity cap (may be NULL to count);
 * *count receives the number of records.  Returns KSA_ERR_INVALID_ARG if cap is too
 * small (count still set).  A tile is listed iff it holds at least one visible pair.
 */
int ksa_schedule_dump(ksa_ctx* ctx, const ksa_params* p, ksa_tile_rec* recs, int64_t cap,
                      int64_t* count);

/* ---- diagnostics -------------------------------------------------------------------- */
/* Reads (with a blocking copy) the device status word written by bounded waits:
 * 0 = no wait gave up since the word was last cleared (returns KSA_OK); otherwise a code naming
 * the first wait that did (9: a kernel found that its shared-memory layout does not fit the
 * window it was given, and did nothing) and the call returns KSA_ERR_TIMEOUT: the results of
 * the calls enqueued since the last clear are not valid.  Every device-side wait of the library
 * is bounded (about a second); a kernel whose wait gives up leaves its loops, waits (bounded)
 * for its copies in flight, frees its TMEM and returns, so the context stays usable. */
int ksa_last_device_status(ksa_ctx* ctx, int32_t* status);
/* Self-test of that path (no counterpart in the paper): a one-warp kernel waits with the library's
 * bounded-wait helper, limited to limit_cycles SM cycles (1 .. 2^31), on a barrier that nothing
 * arrives at.  Afterwards ksa_last_device_status reports code 8 and KSA_ERR_TIMEOUT, and
 * report5_device (DEVICE, five int32) holds {first wait succeeded (0 expected), second wait
 * succeeded (0: it saw the abort flag), abort flag (1), kilo-cycles in the first wait, in the second}.
 * Asynchronous on cuda_stream. */
int ksa_selftest_bounded_wait(ksa_ctx* ctx, int64_t limit_cycles, int32_t* report5_device, void* cuda_stream);
/* Clears the device status word (blocking copy). */
int ksa_clear_device_status(ksa_ctx* ctx);
/* Last cudaError_t / CUresult seen by this context (0 = none). */
int ksa_last_cuda_error(const ksa_ctx* ctx);
/* Kernels launched by this context since creation (pack + summary + text kernels). */
int64_t ksa_launch_count(const ksa_ctx* ctx);
/* The device as the text-row kernels use it: its SM count (the one-CTA kernel runs one persistent CTA
 * on each) and the number of two-CTA clusters it runs at once (the CTA-pair kernel runs that many
 * persistent pairs; 0 would switch that kernel off).  Either pointer may be NULL. */
int ksa_device_info(ksa_ctx* ctx, int32_t* num_sms, int32_t* max_cta_pairs);
/* Optional per-kernel timing: when enabled, ksa_attn_fwd records CUDA events on the
 * caller's stream before and after the text-row kernel (the dominant kernel).
 * ksa_text_kernel_ms waits for the most recent pair and returns the elapsed device
 * time in milliseconds.  Off by default (no events are recorded). */
int ksa_enable_kernel_timing(ksa_ctx* ctx, int on);
int ksa_text_kernel_ms(ksa_ctx* ctx, float* ms);
const char* ksa_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* KSA_H */
