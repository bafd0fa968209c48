// Internal launch interface between the C ABI (ksa_api.cu) and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "ksa_common.h"

namespace ksa {

// De-interleaves text Q/K/V rows and summary K/V rows of the augmented layout (Eq. 1)
// into dense head-major streams; padding rows are written as zeros.
cudaError_t launch_pack(const KernelArgs& a, cudaStream_t stream);

// Summary rows: each attends to the (at most k + m) keys of its own chunk.
cudaError_t launch_summary(const KernelArgs& a, cudaStream_t stream);
// The same on mma.sync tiles: one block per (chunk, KV head), or per group of chunks stacked up to 64 query rows;
// launch_summary dispatches to it for chunks of more than 12 keys when summary_mma_applies (at most 128 query rows m G
// and 128 keys k + m per chunk).  Chunks of up to 12 keys are faster on the short-chunk kernel (measured).
bool summary_mma_applies(const KernelArgs& a);
cudaError_t launch_summary_mma(const KernelArgs& a, int max_chunks, unsigned ny, cudaStream_t stream);

// Text rows, CUDA-core cross-check kernel (KSA_FLAG_REFERENCE_KERNEL).
cudaError_t launch_text_ref(const KernelArgs& a, cudaStream_t stream);

// Text rows, tcgen05/TMA kernel.  The five tensor maps describe the packed streams
// as [D, rows, H] with a {64, 128, 1} box and 128-byte swizzle, or (KernelArgs::direct) the
// caller's interleaved tensors as [D, k, chunks, H] (text rows; box {64, k, 128/k, 1}) and
// [D, m, chunks, H] starting k rows in (summary rows; box {64, m, 128/m, 1}): the box lands in
// shared memory as the same dense 128-row tile either way.
struct TextMaps { CUtensorMap qt, kt, vt, ks, vs; };
cudaError_t launch_text_tc(const KernelArgs& a, const TextMaps& maps, int num_sms, cudaStream_t stream);
// One-time per-device setup (dynamic shared memory opt-in).
cudaError_t setup_text_tc();

// Text rows on CTA pairs (head_dim 128, work items of two query heads): same tensor maps, except that kt and ks
// have boxes of 64 key rows ({64, 64, 1}; direct: {64, k, 64 / k, 1} and {64, m, 64 / m, 1}) -- each CTA of a pair
// loads half of a K tile.  max_pairs = clusters of two CTAs the device runs at once (from setup_text_pair).
struct PairMaps { CUtensorMap qt, kt, vt, ks, vs; };
cudaError_t launch_text_pair(const KernelArgs& a, const PairMaps& maps, int max_pairs, cudaStream_t stream);
cudaError_t setup_text_pair(int* max_pairs);

// Q/K/V preparation upstream of the attention (position ids, interpolation at summary positions, rotary
// embedding): one pass over the augmented rows.
struct PrepArgs {
    const SeqInfo* seqs;
    int32_t k, m, Hq, Hkv, D;
    int32_t rope;                  // 0: interpolate only
    float lambda;
    double inv_freq[64];           // theta^(-2 d / D), d = 0 .. D/2 - 1 (head_dim <= 128)
    const uint16_t* qm; const uint16_t* km; const uint16_t* vm;     // projections with the shared weights
    const uint16_t* qs; const uint16_t* ks; const uint16_t* vs;     // ... with the summary weights, [S, H, D]
    uint16_t* qo; uint16_t* ko; uint16_t* vo;
    int64_t q_st, q_sh, k_st, k_sh, v_st, v_sh;
    // to_streams != 0: the prepared rows go straight into the packed head-major streams of the attention kernels
    // (text rows of q, k, v -> qt, kt, vt; summary rows of k, v, q -> ks_out, vs_out, qs_out) instead of qo / ko / vo:
    // preparation and packing in one pass over q, k, v
    int32_t to_streams;
    uint16_t* qt; uint16_t* kt; uint16_t* vt; uint16_t* ks_out; uint16_t* vs_out; uint16_t* qs_out;
    int64_t text_rows, summ_rows;
};
cudaError_t launch_prep(const PrepArgs& a, int64_t max_aug_len, int num_seqs, cudaStream_t stream);
// Zeroes the padding rows of the packed streams (text: qt, kt, vt; summary: ks, vs, qs) that launch_prep in stream mode
// does not write.
cudaError_t launch_zero_stream_pads(const PrepArgs& a, int num_seqs, cudaStream_t stream);
// Summary rows from the packed streams (query rows in qs): each attends to the keys of its own chunk.
cudaError_t launch_summary_streams(const KernelArgs& a, const uint16_t* qs, cudaStream_t stream);

}  // namespace ksa
