// Shared host/device declarations of the KSA forward library (internal).
#pragma once
#include <stdint.h>

namespace ksa {

constexpr int kTileM = 128;   // query rows per tile
constexpr int kTileN = 128;   // key/value rows per tile

// Per-sequence layout (Eq. 1): derived once on the host, read by every kernel.
struct SeqInfo {
    int64_t aug_off;    // first augmented row of the sequence in q/k/v/out
    int32_t n_text;     // n_b
    int32_t n_chunks;   // J_b = floor(n_b / k) full chunks
    int32_t n_summ;     // J_b * m rows of the summary stream
    int32_t text_off;   // first row of the sequence in the packed text stream (multiple of kTileM)
    int32_t summ_off;   // first row in the packed summary stream (multiple of kTileN)
    int32_t text_pad;   // padded text rows (multiple of kTileM)
    int32_t summ_pad;   // padded summary rows (multiple of kTileN)
    int32_t chunk0;     // aug_off / (k + m): first chunk of the sequence in the direct views (valid if every length is a multiple of k)
    int32_t summ_base;  // summary rows of the sequences before this one (unpadded count)
};

// One unit of work of the text-row kernel: one query tile, one or two query heads that
// share a KV head, and the key/value tiles Eq. 3 makes visible to that tile.
struct WorkItem {
    int32_t seq;
    int32_t q_tile;           // query rows [q_tile*kTileM, +kTileM) of the text stream
    int32_t head0;            // first query head
    int32_t n_heads;          // 1 or 2 (head0, head0+1)
    int32_t ns_tiles;         // summary-stream tiles [0, ns_tiles) are visited
    int32_t ns_nomask;        // of those, tiles [0, ns_nomask) need no in-tile mask
    int32_t band_lo, band_hi; // text-stream tiles [band_lo, band_hi] are visited
    int32_t band_nomask_lo;   // text tiles [band_nomask_lo, band_nomask_hi) need no mask
    int32_t band_nomask_hi;
    int32_t reserved0, reserved1;
};
static_assert(sizeof(WorkItem) == 48, "WorkItem layout");

// Arguments common to the kernels.
struct KernelArgs {
    const SeqInfo* seqs;
    const WorkItem* work;
    int32_t num_seqs;
    int32_t num_work;
    int32_t k, m, C;
    int32_t Hq, Hkv, D;
    uint32_t flags;
    float scale;            // softmax scale
    float scale_log2;       // scale * log2(e)
    int64_t total_aug;
    int64_t text_rows;      // padded rows of the packed text stream
    int64_t summ_rows;      // padded rows of the packed summary stream
    int32_t max_text_pad;   // largest per-sequence padded text rows
    int32_t max_summ_pad;   // largest per-sequence padded summary rows
    int32_t max_n_summ;     // largest per-sequence summary count
    // Row range (pack and summary kernels): r_seq < 0 means every sequence in full; otherwise only
    // sequence r_seq, packed text rows [r_text0, r_text1), summary-stream rows [r_summ0, r_summ1)
    // (pack) and summary query rows [r_summ0, r_summq1) (summary-row kernel).
    int32_t direct;         // text kernel reads Q/K/V tiles straight from the caller's tensors (no packed streams)
    int32_t r_seq;
    int32_t r_text0, r_text1, r_summ0, r_summ1, r_summq1;
    // user tensors (bf16 as uint16)
    const uint16_t* q; const uint16_t* kx; const uint16_t* v; uint16_t* out; float* lse;
    int64_t q_st, q_sh, k_st, k_sh, v_st, v_sh, o_st, o_sh;
    // packed streams in the workspace, head-major [H][rows][D]
    uint16_t* qt; uint16_t* kt; uint16_t* vt; uint16_t* ks; uint16_t* vs;
    int32_t* status;        // device status word for bounded waits
};

// Device status codes (which bounded wait gave up first).
enum DeviceStatus : int32_t {
    kStatusOk = 0,
    kStatusWaitQFull = 1, kStatusWaitQEmpty = 2, kStatusWaitKvFull = 3, kStatusWaitKvEmpty = 4,
    kStatusWaitSFull = 5, kStatusWaitPFull = 6, kStatusWaitOFull = 7, kStatusWaitTest = 8,
    kStatusSmemLayout = 9,      // the dynamic shared memory window did not hold the 1024-byte aligned layout
    kStatusWaitMaxPub = 10,     // CTA-pair kernel: the other softmax group's reference maximum
    kStatusWaitRowSums = 11,    // CTA-pair kernel: the other softmax group's row sums
    kStatusWaitPvDone = 12,     // CTA-pair kernel: completion of O += P V
    kStatusWaitOEmpty = 13,     // CTA-pair kernel: the epilogue's read of O
    kStatusBounds = 14,         // KSA_DEBUG builds: a global output index was outside its tensor; the access was skipped
};

// KSA_DEBUG builds (the stand-in for a memory checker): every global store of the kernels goes through ksa_in_bounds,
// which records kStatusBounds and makes the caller skip the access when the index is outside the tensor.
#if defined(__CUDACC__)
#ifdef KSA_DEBUG
__device__ __forceinline__ bool ksa_in_bounds(bool ok, int32_t* status)
{
    if (!ok) atomicCAS(status, 0, (int32_t)kStatusBounds);
    return ok;
}
#else
__device__ __forceinline__ bool ksa_in_bounds(bool, int32_t*) { return true; }
#endif
// a row of out (and its lse entry) addressed by augmented row and query head
__device__ __forceinline__ bool ksa_out_row_ok(const KernelArgs& a, int64_t aug, int h)
{
    return ksa_in_bounds(aug >= 0 && aug < a.total_aug && h >= 0 && h < a.Hq, a.status);
}
#endif

}  // namespace ksa
