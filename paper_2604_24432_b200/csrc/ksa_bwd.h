// Internal interface of the backward pass (kernel arguments and launchers).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "ksa_common.h"

namespace ksa {

struct BwdArgs {
    const SeqInfo* seqs;
    int32_t num_seqs;
    int32_t k, m, C, Hq, Hkv, D;
    uint32_t flags;
    float scale, scale_log2;
    int64_t total_aug, text_rows, summ_rows;
    int32_t max_text_pad, max_summ_pad, max_n_summ;
    // caller tensors (bf16 bit patterns; lse fp32 [Hq, total_aug])
    const uint16_t* q; const uint16_t* kx; const uint16_t* v; const uint16_t* out; const uint16_t* dout; const float* lse;
    uint16_t* dq; uint16_t* dk; uint16_t* dv;
    int64_t q_st, q_sh, k_st, k_sh, v_st, v_sh, o_st, o_sh, do_st, do_sh, dq_st, dq_sh, dk_st, dk_sh, dv_st, dv_sh;
    // workspace: packed streams of the forward pass, packed dO, per-row scalars, fp32 accumulators
    const uint16_t* qt; const uint16_t* kt; const uint16_t* vt; const uint16_t* ks; const uint16_t* vs;
    uint16_t* dot;              // [Hq][text_rows][D]
    float* lse_t;               // [Hq][text_rows], times log2(e); +inf on padding rows
    float* delta_t;             // [Hq][text_rows], <dO, O>
    float* dkt; float* dvt;     // [Hkv][text_rows][D] fp32
    float* dks; float* dvs;     // [Hkv][summ_rows][D] fp32
    int32_t* status;            // device status word of the context (bounded waits report here)
    int32_t direct;             // tensor-core kernels read q, k, v, dout through chunked views: no packed copies
};

// Tensor maps for the tensor-core kernels (128-byte swizzle, boxes of 64 elements x 128 rows): Q and dO per query
// head, K and V of the text and the summary rows per KV head -- of the packed streams, or (direct mode) chunked
// 4-D views of the caller's interleaved tensors.
struct BwdMaps { CUtensorMap qt, dot, kt, vt, ks, vs; };

// Packs the text rows of dO, lse (in log2 units) and delta = <dO, O>.
cudaError_t launch_bwd_prep(const BwdArgs& a, cudaStream_t stream);
// Summary query rows: their dQ rows directly, their dK / dV contributions into the accumulators.
cudaError_t launch_bwd_summary(const BwdArgs& a, cudaStream_t stream);
// The same on mma.sync tiles, one block per (chunk, KV head) or per group of short chunks; launch_bwd_summary dispatches
// to it when bwd_summary_mma_applies (at most 128 query rows m G and 128 keys k + m per chunk).
bool bwd_summary_mma_applies(const BwdArgs& a);
cudaError_t launch_bwd_summary_mma(const BwdArgs& a, cudaStream_t stream);
// Text query rows: dQ (written directly), then dK / dV into the accumulators.
cudaError_t launch_bwd_dq(const BwdArgs& a, cudaStream_t stream);
cudaError_t launch_bwd_dkv(const BwdArgs& a, cudaStream_t stream);
// Accumulators -> bf16 dk / dv at the augmented positions.
cudaError_t launch_bwd_finish(const BwdArgs& a, cudaStream_t stream);
cudaError_t setup_bwd();
// dQ and dK / dV of the text rows on the tcgen05 tensor cores (head_dim 128 and 64).
cudaError_t launch_bwd_dq_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream);
cudaError_t launch_bwd_dkv_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream);
// True if launch_bwd_dkv_tc writes the text keys' accumulator rows with plain stores (one CTA per key tile covers every
// query tile that sees it): it must then run before anything adds to those rows, and they need no clear.
bool bwd_text_keys_stored(const BwdArgs& a);
cudaError_t setup_bwd_tc();

}  // namespace ksa
