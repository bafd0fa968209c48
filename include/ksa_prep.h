/*
 * ksa_prep.h -- C ABI of the step between the Q/K/V projections and the KSA attention operator:
 * position ids of the augmented sequence, interpolation of the two projections at summary positions
 * and the rotary position embedding, in one pass over q, k, v.
 *
 *   position ids   a text token keeps its index in the original sequence; a summary token takes the
 *                  position id of its own chunk's last text token (second bullet of Sec. 2.2.1; with
 *                  several summary tokens per chunk all of them do); every sequence starts at 0
 *   interpolation  at a summary position  x = lambda x_s + (1 - lambda) x_main  for x in {q, k, v}: the
 *                  projection with the summary weights and the one with the shared weights of the same
 *                  hidden state ("Parameter annealing for CPT", Sec. 4.1); text positions take x_main
 *   rotation       q and k (not v) get the rotary embedding with base rope_theta (Table 3; keys carry it
 *                  into the cache, Sec. 2.3.1): element d of the first half of a head is paired with
 *                  element d + head_dim / 2 and the pair turns by  pos * rope_theta^(-2 d / head_dim)
 *                  (angles in double precision, arithmetic on the values in fp32, one rounding to bf16)
 *
 * Tensors are DEVICE bf16.  q_main, k_main, v_main and the outputs have the layouts and strides of q, k, v
 * in ksa_params ([total_aug, heads, head_dim]); an output may be the same tensor as its _main input.
 * q_summ, k_summ, v_summ are contiguous [S, heads, head_dim], S = the summary rows of the batch in order
 * (sequence by sequence, chunk by chunk); they may be NULL when lambda == 0.  All pointers 16-byte aligned.
 */
#ifndef KSA_PREP_H
#define KSA_PREP_H

#include "ksa.h"

#ifdef __cplusplus
extern "C" {
#endif

#define KSA_PREP_NO_ROPE  1u   /* interpolate only */

/* lambda of the annealing schedule at training step `step`: 1 up to s_start, 0 from s_end on, linear in
 * between (Sec. 4.1).  s_end must be > s_start.  Host only. */
int ksa_anneal_lambda(int64_t step, int64_t s_start, int64_t s_end, float* lambda);
/* Position id of every augmented row of the batch (HOST array of ksa_total_aug_len entries). */
int ksa_position_ids(const ksa_params* p, int32_t* position_ids);
/* Number of summary rows of the batch (the S above). */
int64_t ksa_total_summary_rows(const ksa_params* p);
/*
 * The pass itself, asynchronous on cuda_stream.  lambda in [0, 1]; rope_theta > 0 unless
 * prep_flags has KSA_PREP_NO_ROPE.  Errors: KSA_ERR_INVALID_ARG (null / misaligned pointers, bad lambda or
 * theta, bad p), KSA_ERR_CUDA.
 */
int ksa_qkv_prepare(ksa_ctx* ctx, const void* q_main, const void* k_main, const void* v_main,
                    const void* q_summ, const void* k_summ, const void* v_summ,
                    void* q_out, void* k_out, void* v_out, float lambda, float rope_theta, uint32_t prep_flags,
                    const ksa_params* p, void* cuda_stream);

/*
 * Preparation and attention in one call, with the preparation folded into the pass that de-interleaves
 * q, k, v for the attention kernels: the projections are read once, position ids (Sec. 2.2.1), interpolation
 * at summary positions (Sec. 4.1) and rotation are applied on the way, and the prepared rows are written
 * straight into the packed streams the tensor-core kernel reads -- no prepared copy of q, k, v is ever
 * stored in the interleaved layout, and the whole step moves q, k and v through HBM once in and once out
 * (what ksa_qkv_prepare alone costs).  Works for any lengths; results equal
 * ksa_qkv_prepare followed by ksa_attn_fwd bit for bit (same arithmetic on the same rows).
 * q_main .. v_summ, lambda, rope_theta, prep_flags: as for ksa_qkv_prepare; out, lse, p, cuda_stream: as for
 * ksa_attn_fwd (KSA_FLAG_REFERENCE_KERNEL is not accepted).  workspace: DEVICE, 256-byte aligned,
 * >= ksa_prepared_workspace_bytes (the packed streams plus the prepared query rows of the summary tokens).
 */
int ksa_prepared_workspace_bytes(const ksa_ctx* ctx, const ksa_params* p, size_t* bytes);
int ksa_attn_fwd_prepared(ksa_ctx* ctx, const void* q_main, const void* k_main, const void* v_main,
                          const void* q_summ, const void* k_summ, const void* v_summ,
                          float lambda, float rope_theta, uint32_t prep_flags,
                          void* out, float* lse, void* workspace, size_t workspace_bytes,
                          const ksa_params* p, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* KSA_PREP_H */
