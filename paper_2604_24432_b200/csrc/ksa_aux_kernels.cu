// Pack (de-interleave) kernel, summary-row kernel and the CUDA-core cross-check
// kernel for text rows.  All three are bandwidth- or latency-bound helpers around the
// tensor-core text kernel.
#include <cuda_bf16.h>

#include <type_traits>

#include "ksa_launch.h"

namespace ksa {

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f)
{
    __nv_bfloat16 h = __float2bfloat16_rn(f);
    return *reinterpret_cast<uint16_t*>(&h);
}

// ---------------------------------------------------------------------------------------
// Pack.  grid = (blocks, num_seqs, 2): z = 0 packs the text stream (Q, K, V rows of text
// tokens), z = 1 the summary stream (K, V rows of summary tokens).  One thread moves one
// 16-byte vector.  Text token i of a sequence sits at augmented row (i/k)*(k+m) + i%k,
// summary (j, r) at j*(k+m) + k + r (Eq. 1).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) ksa_pack_kernel(KernelArgs a)
{
    const bool ranged = a.r_seq >= 0;
    const SeqInfo sq = a.seqs[ranged ? a.r_seq : (int)blockIdx.y];
    const bool text = (blockIdx.z == 0);
    const int vecs = a.D / 8;
    const int slots = text ? (a.Hq + 2 * a.Hkv) : (2 * a.Hkv);
    const int row_first = ranged ? (text ? a.r_text0 : a.r_summ0) : 0;
    const int pad_rows = (ranged ? (text ? a.r_text1 : a.r_summ1) : (text ? sq.text_pad : sq.summ_pad)) - row_first;
    const int live_rows = text ? sq.n_text : sq.n_summ;
    const int64_t per_row = (int64_t)slots * vecs;
    const int64_t total = (int64_t)pad_rows * per_row;
    const int s = a.k + a.m;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int row_rel = (int)(idx / per_row);
        const int rem = (int)(idx - (int64_t)row_rel * per_row);
        const int row = row_first + row_rel;
        const int slot = rem / vecs;
        const int vec = rem - slot * vecs;
        int64_t aug = 0;
        if (row < live_rows) {
            if (text) aug = sq.aug_off + (int64_t)(row / a.k) * s + (row % a.k);
            else      aug = sq.aug_off + (int64_t)(row / a.m) * s + a.k + (row % a.m);
        }
        const uint16_t* src;
        uint16_t* dst;
        if (text) {
            const int64_t drow = (int64_t)sq.text_off + row;
            if (slot < a.Hq) {
                src = a.q + aug * a.q_st + (int64_t)slot * a.q_sh;
                dst = a.qt + ((int64_t)slot * a.text_rows + drow) * a.D;
            } else if (slot < a.Hq + a.Hkv) {
                const int h = slot - a.Hq;
                src = a.kx + aug * a.k_st + (int64_t)h * a.k_sh;
                dst = a.kt + ((int64_t)h * a.text_rows + drow) * a.D;
            } else {
                const int h = slot - a.Hq - a.Hkv;
                src = a.v + aug * a.v_st + (int64_t)h * a.v_sh;
                dst = a.vt + ((int64_t)h * a.text_rows + drow) * a.D;
            }
        } else {
            const int64_t drow = (int64_t)sq.summ_off + row;
            if (slot < a.Hkv) {
                src = a.kx + aug * a.k_st + (int64_t)slot * a.k_sh;
                dst = a.ks + ((int64_t)slot * a.summ_rows + drow) * a.D;
            } else {
                const int h = slot - a.Hkv;
                src = a.v + aug * a.v_st + (int64_t)h * a.v_sh;
                dst = a.vs + ((int64_t)h * a.summ_rows + drow) * a.D;
            }
        }
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        // (debug builds) the source row inside the caller's tensors, the destination row inside its stream
        const bool in_range = ksa_in_bounds(aug >= 0 && aug < a.total_aug && row >= 0 &&
                                            (int64_t)(text ? sq.text_off : sq.summ_off) + row < (text ? a.text_rows : a.summ_rows), a.status);
        if (!in_range) continue;
        if (row < live_rows) val = *reinterpret_cast<const uint4*>(src + vec * 8);
        *reinterpret_cast<uint4*>(dst + vec * 8) = val;
    }
}

cudaError_t launch_pack(const KernelArgs& a, cudaStream_t stream)
{
    // grid.x covers the longest padded stream of any sequence (grid-stride loop beyond the cap).
    const int64_t per_row = (int64_t)(a.Hq + 2 * a.Hkv) * (a.D / 8);
    int64_t rows = a.max_text_pad > a.max_summ_pad ? a.max_text_pad : a.max_summ_pad;
    if (a.r_seq >= 0) rows = (a.r_text1 - a.r_text0) > (a.r_summ1 - a.r_summ0) ? (a.r_text1 - a.r_text0) : (a.r_summ1 - a.r_summ0);
    int64_t blocks = (rows * per_row + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (blocks < 1) blocks = 1;
    dim3 grid((unsigned)blocks, a.r_seq >= 0 ? 1u : (unsigned)a.num_seqs, a.m > 0 ? 2u : 1u);
    ksa_pack_kernel<<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Summary rows (Sec. 2.2.1, first bullet), chunks of any length.  The keys of summary r of chunk j are the
// contiguous augmented rows j*(k+m) .. j*(k+m) + k - 1 (+ r + 1 own-chunk summaries unless
// KSA_FLAG_SUMMARY_TEXT_ONLY).  One warp per (chunk, KV head, block of eight (summary row, query head) tasks),
// the task blocks of a chunk in neighbouring warps;
// its lanes form four groups of eight, a group takes one task at a time and each lane D / 8 consecutive
// elements of the head dimension (16-byte vectors; three shuffle steps per dot product; the four groups read
// the same K / V addresses).  The keys go by in batches of kSummBatch with a running maximum and sum.
// ---------------------------------------------------------------------------------------
constexpr int kSummBatch = 8;
constexpr int kSummTaskBlock = 8;   // tasks per warp
constexpr int kSummChunks = 8;      // short chunks: chunks (= warps) per block

// The warp asks for the 128-byte lines of rows [0, rows) of one head (D elements per row, row stride st elements)
// ahead of their use: the loads that follow then find them in L1 instead of waiting for L2 / HBM one key at a time.
template <int D>
__device__ __forceinline__ void summ_prefetch_rows(const uint16_t* base, int64_t st, int rows, int lane)
{
    constexpr int kLines = D * 2 / 128 > 0 ? D * 2 / 128 : 1;
    for (int idx = lane; idx < rows * kLines; idx += 32) {
        const uint16_t* p = base + (int64_t)(idx / kLines) * st + (idx % kLines) * 64;
        asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
    }
}

__device__ __forceinline__ void summ_unpack(const uint4& raw, float* f)
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        f[2 * e] = __uint_as_float(w[e] << 16);
        f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
}

// The tasks [task_lo, task_hi) of one chunk and KV head by one warp; kp / vp point at the lane's elements of the
// chunk's first K / V row (global or shared memory), kst / vst are the row strides in elements.
template <int D>
__device__ __forceinline__ void summ_long_tasks(const KernelArgs& a, const uint16_t* kp, int64_t kst, const uint16_t* vp, int64_t vst,
                                                int64_t row0, int hk, int G, int own, int task_lo, int task_hi, int lane)
{
    constexpr int E = D / 8;
    constexpr int V4 = E / 8;
    const int sub = lane & 7, grp = lane >> 3;
    for (int t0 = task_lo; t0 < task_hi; t0 += 4) {
        const int task = t0 + grp;
        const bool live = task < task_hi;
        const int tk = live ? task : task_hi - 1;                      // idle groups shadow the last task (no stores)
        const int r = tk / G, g = tk - r * G;
        const int h = hk * G + g;
        const int64_t qrow = row0 + a.k + r;
        const int nk = a.k + own * (r + 1);
        const int nk_max = a.k + own * ((min(t0 + 3, task_hi - 1)) / G + 1);   // of the four tasks: uniform over the warp
        float qv[E], acc[E];
        {
            const uint16_t* qp = a.q + qrow * a.q_st + (int64_t)h * a.q_sh + sub * E;
#pragma unroll
            for (int c = 0; c < V4; ++c) summ_unpack(*reinterpret_cast<const uint4*>(qp + 8 * c), qv + 8 * c);
        }
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        float mx = -INFINITY, l = 0.f;
        for (int b0 = 0; b0 < nk_max; b0 += kSummBatch) {
            float x[kSummBatch];
#pragma unroll
            for (int i = 0; i < kSummBatch; ++i) {
                float dot = 0.f;
                if (b0 + i < nk_max) {
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        float kf[8];
                        summ_unpack(*reinterpret_cast<const uint4*>(kp + (int64_t)(b0 + i) * kst + 8 * c), kf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) dot = fmaf(qv[8 * c + e], kf[e], dot);
                    }
                }
                x[i] = dot;
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
#pragma unroll
                for (int i = 0; i < kSummBatch; ++i) x[i] += __shfl_xor_sync(0xffffffffu, x[i], o);
            }
            float mn = mx;
#pragma unroll
            for (int i = 0; i < kSummBatch; ++i) {
                x[i] = (b0 + i < nk) ? x[i] * a.scale : -INFINITY;
                mn = fmaxf(mn, x[i]);
            }
            // key 0 is visible to every task, so mn is finite from the first batch on
            const float alpha = __expf(mx - mn);                       // exp(-inf) = 0 on the first batch
            mx = mn;
            l *= alpha;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] *= alpha;
#pragma unroll
            for (int i = 0; i < kSummBatch; ++i) {
                if (b0 + i < nk_max) {
                    const float p = __expf(x[i] - mn);                 // 0 on the keys this task does not see
                    l += p;
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        float vf[8];
                        summ_unpack(*reinterpret_cast<const uint4*>(vp + (int64_t)(b0 + i) * vst + 8 * c), vf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[8 * c + e] = fmaf(p, vf[e], acc[8 * c + e]);
                    }
                }
            }
        }
        if (live && ksa_out_row_ok(a, qrow, h)) {
            const float inv = 1.f / l;
            uint16_t* op = a.out + qrow * a.o_st + (int64_t)h * a.o_sh + sub * E;
#pragma unroll
            for (int c = 0; c < V4; ++c) {
                uint4 ov;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    ow[e] = (uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e] * inv) | ((uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e + 1] * inv) << 16);
                *reinterpret_cast<uint4*>(op + 8 * c) = ov;
            }
            if (sub == 0) a.lse[(int64_t)h * a.total_aug + qrow] = mx + __logf(l);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(256, 2) ksa_summary_kernel(KernelArgs a)
{
    constexpr int E = D / 8;                      // elements per lane: 16 (two 16-byte vectors) or 8 (one)
    const bool ranged = a.r_seq >= 0;
    const SeqInfo sq = a.seqs[ranged ? a.r_seq : (int)blockIdx.y];
    const int hk = blockIdx.z;
    const int G = a.Hq / a.Hkv;
    const int tasks = a.m * G;
    const int task_blocks = (tasks + kSummTaskBlock - 1) / kSummTaskBlock;
    // whole chunks only: a range starts and ends on chunk boundaries of the summary stream
    const int j_first = ranged ? a.r_summ0 / a.m : 0;
    const int j_end = ranged ? a.r_summq1 / a.m : sq.n_chunks;
    // consecutive warps take the task blocks of one chunk (they read the same K / V rows), then the next chunk's
    const int64_t gw = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int j = j_first + (int)(gw / task_blocks);
    if (j >= j_end) return;                                            // warp-uniform
    const int task_lo = (int)(gw % task_blocks) * kSummTaskBlock;
    const int task_hi = min(tasks, task_lo + kSummTaskBlock);
    const int lane = threadIdx.x & 31, sub = lane & 7;
    const int s = a.k + a.m;
    const int own = (a.flags & 1u) ? 0 : 1;                            // a summary sees the chunk's summaries up to itself
    const int64_t row0 = sq.aug_off + (int64_t)j * s;                  // first row of the chunk
    const uint16_t* kp = a.kx + row0 * a.k_st + (int64_t)hk * a.k_sh + sub * E;
    const uint16_t* vp = a.v + row0 * a.v_st + (int64_t)hk * a.v_sh + sub * E;
    {
        const int rows_seen = a.k + own * ((task_hi - 1) / G + 1);     // keys of the warp's last task
        summ_prefetch_rows<D>(a.kx + row0 * a.k_st + (int64_t)hk * a.k_sh, a.k_st, rows_seen, lane);
        summ_prefetch_rows<D>(a.v + row0 * a.v_st + (int64_t)hk * a.v_sh, a.v_st, rows_seen, lane);
    }
    summ_long_tasks<D>(a, kp, a.k_st, vp, a.v_st, row0, hk, G, own, task_lo, task_hi, lane);
}

// The same with the chunk's K and V rows of the KV head staged in shared memory first (2 (k + m) D bf16, dynamic):
// one block per (chunk, KV head), all its loads in flight at once, its warps take the chunk's task blocks in turn.
template <int D>
__global__ void __launch_bounds__(256, 2) ksa_summary_staged_kernel(KernelArgs a)
{
    constexpr int E = D / 8;
    extern __shared__ __align__(16) uint16_t summ_smem[];
    const bool ranged = a.r_seq >= 0;
    const SeqInfo sq = a.seqs[ranged ? a.r_seq : (int)blockIdx.y];
    const int hk = blockIdx.z;
    const int G = a.Hq / a.Hkv;
    const int tasks = a.m * G;
    const int j_first = ranged ? a.r_summ0 / a.m : 0;
    const int j_end = ranged ? a.r_summq1 / a.m : sq.n_chunks;
    const int j = j_first + (int)blockIdx.x;
    if (j >= j_end) return;                                            // block-uniform
    const int s = a.k + a.m;
    const int own = (a.flags & 1u) ? 0 : 1;
    const int64_t row0 = sq.aug_off + (int64_t)j * s;
    uint16_t* sK = summ_smem;
    uint16_t* sV = summ_smem + s * D;
    {
        constexpr int vecs = D / 8;
        const int total = s * vecs;
        for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
            const int rr = idx / vecs, vv = idx - rr * vecs;
            const uint4 kx = *reinterpret_cast<const uint4*>(a.kx + (row0 + rr) * a.k_st + (int64_t)hk * a.k_sh + vv * 8);
            const uint4 vx = *reinterpret_cast<const uint4*>(a.v + (row0 + rr) * a.v_st + (int64_t)hk * a.v_sh + vv * 8);
            *reinterpret_cast<uint4*>(sK + rr * D + vv * 8) = kx;
            *reinterpret_cast<uint4*>(sV + rr * D + vv * 8) = vx;
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, sub = lane & 7;
    for (int task_lo = (int)(threadIdx.x >> 5) * kSummTaskBlock; task_lo < tasks; task_lo += (int)(blockDim.x >> 5) * kSummTaskBlock)
        summ_long_tasks<D>(a, sK + sub * E, D, sV + sub * E, D, row0, hk, G, own, task_lo, min(tasks, task_lo + kSummTaskBlock), lane);
}

// Summary rows, short chunks (k + m <= kSummMaxKeys; the paper's layout has 9 keys per row).
// A block stages the K and V rows of kSummChunks consecutive chunks of one KV head in shared memory (each row
// is read from global memory once, whatever the GQA group size, with every load of the block in flight at
// once); then one warp per chunk: its lanes form four groups of eight, a group takes one (summary row, query
// head) task at a time, each lane 8 consecutive elements of each 64-element half of the head dimension
// (16-byte vectors, neighbouring lanes on neighbouring banks), so a dot product needs three shuffle steps
// and the four groups read the very same shared-memory addresses.
constexpr int kSummMaxKeys = 12;

template <int D>
__global__ void __launch_bounds__(256) ksa_summary_short_kernel(KernelArgs a)
{
    constexpr int E = D / 8;                      // elements per lane: 16 (two 16-byte vectors) or 8 (one)
    constexpr int V4 = E / 8;
    __shared__ __align__(16) uint16_t sK[kSummChunks * kSummMaxKeys * D];
    __shared__ __align__(16) uint16_t sV[kSummChunks * kSummMaxKeys * D];
    const bool ranged = a.r_seq >= 0;
    const SeqInfo sq = a.seqs[ranged ? a.r_seq : (int)blockIdx.y];
    const int hk = blockIdx.z;
    // whole chunks only: a range starts and ends on chunk boundaries of the summary stream
    const int j_first = ranged ? a.r_summ0 / a.m : 0;
    const int j_end = ranged ? a.r_summq1 / a.m : sq.n_chunks;
    const int j0 = j_first + blockIdx.x * kSummChunks;
    if (j0 >= j_end) return;                                           // block-uniform
    const int nch = min(kSummChunks, j_end - j0);
    const int s = a.k + a.m;
    const int G = a.Hq / a.Hkv;
    // the block's nch * s rows of K and V of this KV head (contiguous augmented rows), 16-byte vectors
    {
        constexpr int vecs = D / 8;
        const int64_t r0 = sq.aug_off + (int64_t)j0 * s;
        const int total = nch * s * vecs;
        for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
            const int rr = idx / vecs, vv = idx - rr * vecs;
            const uint4 kx = *reinterpret_cast<const uint4*>(a.kx + (r0 + rr) * a.k_st + (int64_t)hk * a.k_sh + vv * 8);
            const uint4 vx = *reinterpret_cast<const uint4*>(a.v + (r0 + rr) * a.v_st + (int64_t)hk * a.v_sh + vv * 8);
            *reinterpret_cast<uint4*>(sK + rr * D + vv * 8) = kx;
            *reinterpret_cast<uint4*>(sV + rr * D + vv * 8) = vx;
        }
    }
    __syncthreads();
    const int wid = threadIdx.x >> 5;
    if (wid >= nch) return;                                            // warp-uniform, after the only barrier
    const int j = j0 + wid;
    const int lane = threadIdx.x & 31, sub = lane & 7, grp = lane >> 3;
    const int64_t row0 = sq.aug_off + (int64_t)j * s;                  // first row of the chunk
    // a lane's elements: 8 sub .. 8 sub + 7 of each 64-element half (neighbouring lanes read neighbouring 16 bytes)
    const uint16_t* kp = sK + wid * s * D + sub * 8;
    const uint16_t* vp = sV + wid * s * D + sub * 8;
    auto unpack = [](const uint4& raw, float* f) {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            f[2 * e] = __uint_as_float(w[e] << 16);
            f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
    };
    const int tasks = a.m * G;
    for (int t0 = 0; t0 < tasks; t0 += 4) {
        const int task = t0 + grp;
        const bool live = task < tasks;
        const int tk = live ? task : tasks - 1;                        // idle groups shadow the last task (no stores)
        const int r = tk / G, g = tk - r * G;
        const int h = hk * G + g;
        const int64_t qrow = row0 + a.k + r;
        const int nk = a.k + ((a.flags & 1u) ? 0 : (r + 1));           // own-chunk text (+ own summaries 0..r)
        float qv[E];
        {
            const uint16_t* qp = a.q + qrow * a.q_st + (int64_t)h * a.q_sh + sub * 8;
#pragma unroll
            for (int c = 0; c < V4; ++c) unpack(*reinterpret_cast<const uint4*>(qp + 64 * c), qv + 8 * c);
        }
        float x[kSummMaxKeys];
#pragma unroll
        for (int t = 0; t < kSummMaxKeys; ++t) {
            float dot = 0.f;
            if (t < s) {                                               // uniform: rows of the chunk
#pragma unroll
                for (int c = 0; c < V4; ++c) {
                    float kf[8];
                    unpack(*reinterpret_cast<const uint4*>(kp + t * D + 64 * c), kf);
#pragma unroll
                    for (int e = 0; e < 8; ++e) dot = fmaf(qv[8 * c + e], kf[e], dot);
                }
            }
            x[t] = dot;
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
#pragma unroll
            for (int t = 0; t < kSummMaxKeys; ++t)
                if (t < s) x[t] += __shfl_xor_sync(0xffffffffu, x[t], o);
        }
        float mx = -INFINITY;
#pragma unroll
        for (int t = 0; t < kSummMaxKeys; ++t) {
            x[t] = (t < nk) ? x[t] * a.scale : -INFINITY;
            mx = fmaxf(mx, x[t]);
        }
        float l = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
#pragma unroll
        for (int t = 0; t < kSummMaxKeys; ++t) {
            if (t < s) {
                const float p = (t < nk) ? __expf(x[t] - mx) : 0.f;
                l += p;
#pragma unroll
                for (int c = 0; c < V4; ++c) {
                    float vf[8];
                    unpack(*reinterpret_cast<const uint4*>(vp + t * D + 64 * c), vf);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[8 * c + e] = fmaf(p, vf[e], acc[8 * c + e]);
                }
            }
        }
        if (live && ksa_out_row_ok(a, qrow, h)) {
            const float inv = 1.f / l;
            uint16_t* op = a.out + qrow * a.o_st + (int64_t)h * a.o_sh + sub * 8;
#pragma unroll
            for (int c = 0; c < V4; ++c) {
                uint4 ov;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    ow[e] = (uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e] * inv) | ((uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e + 1] * inv) << 16);
                *reinterpret_cast<uint4*>(op + 64 * c) = ov;
            }
            if (sub == 0) a.lse[(int64_t)h * a.total_aug + qrow] = mx + __logf(l);
        }
    }
}

cudaError_t launch_summary(const KernelArgs& a, cudaStream_t stream)
{
    if (a.m <= 0 || a.max_n_summ <= 0) return cudaSuccess;
    // grid.x covers the sequence with the most summary rows; shorter ones exit early.
    const int rows = a.r_seq >= 0 ? (a.r_summq1 - a.r_summ0) : a.max_n_summ;
    if (rows <= 0) return cudaSuccess;
    const unsigned ny = a.r_seq >= 0 ? 1u : (unsigned)a.num_seqs;
    const int max_chunks = rows / a.m;
    const int chunk_groups = (max_chunks + kSummChunks - 1) / kSummChunks;
    if (a.k + a.m <= kSummMaxKeys) {
        dim3 g2((unsigned)chunk_groups, ny, (unsigned)a.Hkv);
        if (a.D == 128) ksa_summary_short_kernel<128><<<g2, 256, 0, stream>>>(a);
        else            ksa_summary_short_kernel<64><<<g2, 256, 0, stream>>>(a);
    } else if (summary_mma_applies(a)) {
        return launch_summary_mma(a, max_chunks, ny, stream);
    } else {
        const int tasks = a.m * (a.Hq / a.Hkv);
        const int task_blocks = (tasks + kSummTaskBlock - 1) / kSummTaskBlock;
        const size_t stage_bytes = (size_t)2 * (a.k + a.m) * a.D * sizeof(uint16_t);
        if (stage_bytes <= 48 * 1024) {                   // the chunk's K / V rows fit the default dynamic window
            dim3 g4((unsigned)max_chunks, ny, (unsigned)a.Hkv);
            if (a.D == 128) ksa_summary_staged_kernel<128><<<g4, 256, stage_bytes, stream>>>(a);
            else            ksa_summary_staged_kernel<64><<<g4, 256, stage_bytes, stream>>>(a);
        } else {
            dim3 g3((unsigned)(((int64_t)max_chunks * task_blocks + 7) / 8), ny, (unsigned)a.Hkv);
            if (a.D == 128) ksa_summary_kernel<128><<<g3, 256, 0, stream>>>(a);
            else            ksa_summary_kernel<64><<<g3, 256, 0, stream>>>(a);
        }
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Text rows, cross-check kernel.  One block per work item, one warp per (row, head) in
// turn.  Walks exactly the tiles the schedule lists, applies the per-row column interval
// of Eq. 3 inside each tile, fp32 online softmax on CUDA cores.
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) ksa_text_ref_kernel(KernelArgs a)
{
    constexpr int E = D / 32;
    const WorkItem w = a.work[blockIdx.x];
    const SeqInfo sq = a.seqs[w.seq];
    const int lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    const int s = a.k + a.m;
    for (int job = threadIdx.x >> 5; job < kTileM * w.n_heads; job += nwarps) {
        const int rl = job % kTileM;
        const int h = w.head0 + job / kTileM;
        const int hk = h / (a.Hq / a.Hkv);
        const int i = w.q_tile * kTileM + rl;
        if (i >= sq.n_text) continue;
        const int c = i / a.k;
        const int far = max(0, c - a.C);
        const int lo_i = far * a.k;       // first visible text token
        const int cnt_i = far * a.m;      // visible summaries: stream rows [0, cnt_i)

        float qv[E], acc[E];
        const uint16_t* qp = a.qt + ((int64_t)h * a.text_rows + sq.text_off + i) * D + lane * E;
#pragma unroll
        for (int e = 0; e < E; ++e) { qv[e] = bf16_bits_to_float(qp[e]); acc[e] = 0.f; }
        float mx = -INFINITY, l = 0.f;

        auto visit = [&](const uint16_t* kbase, const uint16_t* vbase, int c0, int c1) {
            for (int t = c0; t < c1; ++t) {
                const uint16_t* kp = kbase + (int64_t)t * D + lane * E;
                float dot = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) dot = fmaf(qv[e], bf16_bits_to_float(kp[e]), dot);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                const float x = dot * a.scale;
                const float mn = fmaxf(mx, x);
                const float alpha = __expf(mx - mn);
                const float p = __expf(x - mn);
                l = l * alpha + p;
                const uint16_t* vp = vbase + (int64_t)t * D + lane * E;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(acc[e], alpha, p * bf16_bits_to_float(vp[e]));
                mx = mn;
            }
        };
        {   // summary tiles [0, ns_tiles)
            const uint16_t* kb = a.ks + ((int64_t)hk * a.summ_rows + sq.summ_off) * D;
            const uint16_t* vb = a.vs + ((int64_t)hk * a.summ_rows + sq.summ_off) * D;
            for (int ut = 0; ut < w.ns_tiles; ++ut)
                visit(kb, vb, ut * kTileN, min(cnt_i, ut * kTileN + kTileN));
        }
        {   // text tiles [band_lo, band_hi]
            const uint16_t* kb = a.kt + ((int64_t)hk * a.text_rows + sq.text_off) * D;
            const uint16_t* vb = a.vt + ((int64_t)hk * a.text_rows + sq.text_off) * D;
            for (int bt = w.band_lo; bt <= w.band_hi; ++bt)
                visit(kb, vb, max(lo_i, bt * kTileN), min(i + 1, bt * kTileN + kTileN));
        }
        const float inv = 1.f / l;
        const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * s + (i % a.k);
        if (ksa_out_row_ok(a, aug, h)) {
            uint16_t* op = a.out + aug * a.o_st + (int64_t)h * a.o_sh + lane * E;
#pragma unroll
            for (int e = 0; e < E; ++e) op[e] = float_to_bf16_bits(acc[e] * inv);
            if (lane == 0) a.lse[(int64_t)h * a.total_aug + aug] = mx + __logf(l);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Summary rows from the packed streams (the path whose preparation pass wrote the streams directly, so that no
// prepared interleaved tensors exist).  A warp takes one (summary row, KV head, round of four query heads): its four
// groups of eight lanes each take one query head of the group, every lane D / 8 elements, so a dot product needs three
// shuffle steps and the four groups read the same K / V addresses.  Keys of summary (j, r): text rows [j k, j k + k)
// of the text stream, then summary rows j m .. j m + r of the summary stream (Sec. 2.2.1; the latter not under
// KSA_FLAG_SUMMARY_TEXT_ONLY).  Keys go in batches of sixteen (all loads of a batch in flight together), with a
// running maximum and sum across batches.
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) ksa_summary_streams_kernel(KernelArgs a, const uint16_t* __restrict__ qs)
{
    constexpr int E = D / 8;              // elements per lane
    constexpr int V4 = E / 8;             // 16-byte vectors per lane
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int lane = threadIdx.x & 31, lg = lane >> 3, sub = lane & 7;
    const int G = a.Hq / a.Hkv;
    const int rounds = (G + 3) / 4;
    const int64_t tasks = (int64_t)sq.n_summ * a.Hkv * rounds;
    for (int64_t task = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); task < tasks; task += (int64_t)gridDim.x * 8) {
        const int rd = (int)(task % rounds);
        const int hk = (int)((task / rounds) % a.Hkv);
        const int u = (int)(task / ((int64_t)rounds * a.Hkv));
        const int j = u / a.m, r = u % a.m;
        const int gi = rd * 4 + lg;
        const bool live = gi < G;
        const int h = hk * G + (live ? gi : 0);
        float qv[E];
        {
            const uint16_t* qp = qs + ((int64_t)h * a.summ_rows + sq.summ_off + u) * D + sub * E;
#pragma unroll
            for (int c = 0; c < V4; ++c) summ_unpack(*reinterpret_cast<const uint4*>(qp + 8 * c), qv + 8 * c);
        }
        float mx = -INFINITY, l = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        const int nkeys = a.k + ((a.flags & 0x1u) ? 0 : r + 1);
        const int64_t text0 = ((int64_t)hk * a.text_rows + sq.text_off + (int64_t)j * a.k) * D + sub * E;
        const int64_t summ0 = ((int64_t)hk * a.summ_rows + sq.summ_off + (int64_t)j * a.m) * D + sub * E;
        for (int c0 = 0; c0 < nkeys; c0 += 16) {
            float sc[16];
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                const int key = c0 + t;
                float dot = 0.f;
                if (key < nkeys) {
                    const uint16_t* kp = key < a.k ? a.kt + text0 + (int64_t)key * D : a.ks + summ0 + (int64_t)(key - a.k) * D;
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        float kf[8];
                        summ_unpack(*reinterpret_cast<const uint4*>(kp + 8 * c), kf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) dot = fmaf(qv[8 * c + e], kf[e], dot);
                    }
                }
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                sc[t] = key < nkeys ? dot * a.scale : -INFINITY;
            }
            float cm = sc[0];
#pragma unroll
            for (int t = 1; t < 16; ++t) cm = fmaxf(cm, sc[t]);
            const float m_new = fmaxf(mx, cm);
            const float corr = __expf(mx - m_new);
            l *= corr;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] *= corr;
            mx = m_new;
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                const int key = c0 + t;
                if (key < nkeys) {
                    const float p = __expf(sc[t] - mx);
                    l += p;
                    const uint16_t* vp = key < a.k ? a.vt + text0 + (int64_t)key * D : a.vs + summ0 + (int64_t)(key - a.k) * D;
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        float vf[8];
                        summ_unpack(*reinterpret_cast<const uint4*>(vp + 8 * c), vf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[8 * c + e] = fmaf(p, vf[e], acc[8 * c + e]);
                    }
                }
            }
        }
        const int64_t aug = sq.aug_off + (int64_t)j * (a.k + a.m) + a.k + r;
        if (live && ksa_out_row_ok(a, aug, h)) {
            const float inv = 1.f / l;
            uint16_t* op = a.out + aug * a.o_st + (int64_t)h * a.o_sh + sub * E;
#pragma unroll
            for (int c = 0; c < V4; ++c) {
                uint4 ov;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    ow[e] = (uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e] * inv) | ((uint32_t)float_to_bf16_bits(acc[8 * c + 2 * e + 1] * inv) << 16);
                *reinterpret_cast<uint4*>(op + 8 * c) = ov;
            }
            if (sub == 0) a.lse[(int64_t)h * a.total_aug + aug] = mx + __logf(l);
        }
    }
}

cudaError_t launch_summary_streams(const KernelArgs& a, const uint16_t* qs, cudaStream_t stream)
{
    if (a.m <= 0 || a.max_n_summ <= 0) return cudaSuccess;
    const int G = a.Hq / a.Hkv;
    int64_t blocks = ((int64_t)a.max_n_summ * a.Hkv * ((G + 3) / 4) + 7) / 8;
    if (blocks > 148 * 32) blocks = 148 * 32;
    dim3 grid((unsigned)blocks, (unsigned)a.num_seqs, 1u);
    if (a.D == 128) ksa_summary_streams_kernel<128><<<grid, 256, 0, stream>>>(a, qs);
    else            ksa_summary_streams_kernel<64><<<grid, 256, 0, stream>>>(a, qs);
    return cudaGetLastError();
}

cudaError_t launch_text_ref(const KernelArgs& a, cudaStream_t stream)
{
    if (a.num_work <= 0) return cudaSuccess;
    if (a.D == 128) ksa_text_ref_kernel<128><<<a.num_work, 256, 0, stream>>>(a);
    else            ksa_text_ref_kernel<64><<<a.num_work, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace ksa
