// Summary rows of long chunks on the tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32).
//
// With many summary tokens per chunk and several query heads per KV head the summary rows of one (chunk, KV head)
// are a small dense problem: M = m G query rows (summary r of the chunk, query head g of the group), the chunk's
// k + m keys, head_dim D -- e.g. 64 x 72 x 128 twice over (Q K^T and P V) for the 64 + 8 layout with G = 8.
// Chunks with few query rows are stacked: a block takes an aligned group of consecutive chunks (up to 64 query rows), a
// row sees the keys of its own chunk only, and chunk j always sits at position j mod group size, so that a row's
// arithmetic is the same whichever row range a call covers.
// One block of four warps per (chunk or chunk group, KV head): the K and V rows and the M query rows are staged in shared
// memory (16-byte chunks XOR-swizzled by row, so that ldmatrix is conflict-free), each warp takes 16-row tiles of the
// M rows: S = Q K^T over all keys (at most 128, scores stay in registers), the visibility rule of Sec. 2.2.1 -- a
// summary sees the k text tokens of its chunk and the chunk's summaries up to itself (text only under
// KSA_FLAG_SUMMARY_TEXT_ONLY) -- a plain softmax over the row, then O = P V with the probabilities taken straight from
// the score registers as the A operand.  This is a legacy-tensor-path kernel on purpose: the tiles are far below a
// tcgen05 tile, and the step is 0.1 - 0.6 % of the forward pass's arithmetic.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "ksa_launch.h"

namespace ksa {

namespace {

constexpr int kMmaMaxKeys = 128;      // k + m, padded to a multiple of 16
constexpr int kMmaMaxRows = 128;      // m G, padded to a multiple of 16

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// rows of D bf16 in shared memory, 16-byte chunk c of row r stored at chunk position c ^ (r & 7)
template <int D>
__device__ __forceinline__ uint32_t sw_addr(uint32_t base, int row, int chunk)
{
    return base + (uint32_t)row * (uint32_t)(D * 2) + (uint32_t)(((chunk ^ (row & 7)) & (D / 8 - 1)) << 4);
}

template <int D>
__global__ void __launch_bounds__(128, 3) ksa_summary_mma_kernel(KernelArgs a, int s_pad, int m_pad, int cpb)
{
    constexpr int CH = D / 8;                     // 16-byte chunks per row
    constexpr int KT_MAX = kMmaMaxKeys / 16;
    extern __shared__ __align__(128) uint16_t smem[];
    const bool ranged = a.r_seq >= 0;
    const SeqInfo sq = a.seqs[ranged ? a.r_seq : (int)blockIdx.y];
    const int hk = blockIdx.z;
    const int G = a.Hq / a.Hkv;
    const int per_chunk = a.m * G, s = a.k + a.m;
    const int j_first = ranged ? a.r_summ0 / a.m : 0;
    const int j_end = ranged ? a.r_summq1 / a.m : sq.n_chunks;
    // The block takes the chunks of one aligned group [j, j + cpb) that lie in [j_first, j_end): their rows and keys are
    // stacked, chunk j + cc always at position cc, so that a row's arithmetic does not depend on where a row range starts.
    const int j = (j_first / cpb + (int)blockIdx.x) * cpb;
    const int cc_lo = max(0, j_first - j), cc_hi = min(cpb, j_end - j);
    if (cc_hi <= cc_lo) return;                                        // block-uniform
    const int tasks = cc_hi * per_chunk, keys = cc_hi * s;             // stacked rows / keys up to the last chunk present
    const int task_lo = cc_lo * per_chunk, key_lo = cc_lo * s;         // ... from the first chunk present
    const int own = (a.flags & 1u) ? 0 : 1;
    const int64_t row0 = sq.aug_off + (int64_t)j * s;                  // first row of the chunk
    const uint32_t sQ = s_u32(smem);
    const uint32_t sK = sQ + (uint32_t)m_pad * D * 2;
    const uint32_t sV = sK + (uint32_t)s_pad * D * 2;
    // ---- stage Q (row t = summary t / G of the chunk, query head hk G + t % G), K, V; padding rows are zeros.
    //      Asynchronous 16-byte copies: every load of the block is in flight before the first one is waited for. ----
    for (int idx = threadIdx.x; idx < (m_pad + 2 * s_pad) * CH; idx += blockDim.x) {
        const int rr = idx / CH, c = idx - rr * CH;
        const uint16_t* src = a.kx + row0 * a.k_st + (int64_t)hk * a.k_sh;   // a valid address for the zero-filled rows
        uint32_t bytes = 0, dst;
        if (rr < m_pad) {
            if (rr >= task_lo && rr < tasks) {
                const int cc = rr / per_chunk, tt = rr - cc * per_chunk;
                const int r = tt / G, g = tt - r * G;
                src = a.q + (row0 + (int64_t)cc * s + a.k + r) * a.q_st + (int64_t)(hk * G + g) * a.q_sh + c * 8;
                bytes = 16;
            }
            dst = sw_addr<D>(sQ, rr, c);
        } else if (rr < m_pad + s_pad) {
            const int kr = rr - m_pad;
            if (kr >= key_lo && kr < keys) { src = a.kx + (row0 + kr) * a.k_st + (int64_t)hk * a.k_sh + c * 8; bytes = 16; }
            dst = sw_addr<D>(sK, kr, c);
        } else {
            const int vr = rr - m_pad - s_pad;
            if (vr >= key_lo && vr < keys) { src = a.v + (row0 + vr) * a.v_st + (int64_t)hk * a.v_sh + c * 8; bytes = 16; }
            dst = sw_addr<D>(sV, vr, c);
        }
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mi = lane >> 3, r8 = lane & 7;      // ldmatrix: matrix index, row within the matrix
    const int g0 = lane >> 2, c2 = (lane & 3) * 2; // accumulator fragment: row (and row + 8), column pair
    const int kt_run = s_pad / 16;
    const float sl2 = a.scale * 1.4426950408889634f;
    for (int mt = warp; mt < m_pad / 16; mt += 4) {
        if (mt * 16 + 16 <= task_lo || mt * 16 >= tasks) continue;     // no row of this tile is present
        // ---- S = Q K^T: 16 rows x s_pad keys ----
        float sc[2 * KT_MAX][4];
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) { sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t qa[4];
            ldsm_x4(qa, sw_addr<D>(sQ, mt * 16 + r8 + 8 * (mi & 1), 2 * kk + (mi >> 1)));
#pragma unroll
            for (int kt = 0; kt < KT_MAX; ++kt) {
                if (kt < kt_run) {
                    uint32_t kb[4];
                    ldsm_x4(kb, sw_addr<D>(sK, kt * 16 + r8 + 8 * (mi >> 1), 2 * kk + (mi & 1)));
                    mma16816(sc[2 * kt], qa, kb[0], kb[1]);
                    mma16816(sc[2 * kt + 1], qa, kb[2], kb[3]);
                }
            }
        }
        // ---- visibility (Sec. 2.2.1) and softmax: rows t0 = 16 mt + g0 and t0 + 8 ----
        const int t0 = mt * 16 + g0, t1 = t0 + 8;
        // visible keys [lo, lo + nk) of the stacked keys: the row's own chunk (padding rows mimic the last row)
        int lo0, lo1;
        uint32_t nk0, nk1;
        {
            const int u0 = min(max(t0, task_lo), tasks - 1), u1 = min(max(t1, task_lo), tasks - 1);
            const int cc0 = u0 / per_chunk, cc1 = u1 / per_chunk;
            lo0 = cc0 * s; nk0 = (uint32_t)(a.k + own * ((u0 - cc0 * per_chunk) / G + 1));
            lo1 = cc1 * s; nk1 = (uint32_t)(a.k + own * ((u1 - cc1 * per_chunk) / G + 1));
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) {
            if (n < 2 * kt_run) {
                const int key = n * 8 + c2;
                sc[n][0] = (uint32_t)(key - lo0) < nk0 ? sc[n][0] * sl2 : -INFINITY;
                sc[n][1] = (uint32_t)(key + 1 - lo0) < nk0 ? sc[n][1] * sl2 : -INFINITY;
                sc[n][2] = (uint32_t)(key - lo1) < nk1 ? sc[n][2] * sl2 : -INFINITY;
                sc[n][3] = (uint32_t)(key + 1 - lo1) < nk1 ? sc[n][3] * sl2 : -INFINITY;
                mx0 = fmaxf(mx0, fmaxf(sc[n][0], sc[n][1]));
                mx1 = fmaxf(mx1, fmaxf(sc[n][2], sc[n][3]));
            }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        float l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) {
            if (n < 2 * kt_run) {
                sc[n][0] = ex2f(sc[n][0] - mx0); sc[n][1] = ex2f(sc[n][1] - mx0);
                sc[n][2] = ex2f(sc[n][2] - mx1); sc[n][3] = ex2f(sc[n][3] - mx1);
                l0 += sc[n][0] + sc[n][1];
                l1 += sc[n][2] + sc[n][3];
            }
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        // ---- O = P V (the probabilities as bf16 pairs first: half the registers while the output tile is live) ----
        uint32_t pp[KT_MAX][4];
#pragma unroll
        for (int kt = 0; kt < KT_MAX; ++kt) {
            if (kt < kt_run) {
                pp[kt][0] = pack_bf2(sc[2 * kt][0], sc[2 * kt][1]);         pp[kt][1] = pack_bf2(sc[2 * kt][2], sc[2 * kt][3]);
                pp[kt][2] = pack_bf2(sc[2 * kt + 1][0], sc[2 * kt + 1][1]); pp[kt][3] = pack_bf2(sc[2 * kt + 1][2], sc[2 * kt + 1][3]);
            }
        }
        float o[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
#pragma unroll
        for (int kt = 0; kt < KT_MAX; ++kt) {
            if (kt < kt_run) {
#pragma unroll
                for (int n2 = 0; n2 < D / 16; ++n2) {
                    uint32_t vb[4];
                    ldsm_x4_trans(vb, sw_addr<D>(sV, kt * 16 + r8 + 8 * (mi & 1), 2 * n2 + (mi >> 1)));
                    mma16816(o[2 * n2], pp[kt], vb[0], vb[1]);
                    mma16816(o[2 * n2 + 1], pp[kt], vb[2], vb[3]);
                }
            }
        }
        // ---- rows to their augmented positions (Eq. 1): the tile goes through the warp's own 16 Q rows of shared
        //      memory (no other warp reads them), so that a lane stores 16 bytes and a warp whole rows ----
        {
            const float inv0 = 1.f / l0, inv1 = 1.f / l1;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const uint32_t w0 = pack_bf2(o[i][0] * inv0, o[i][1] * inv0), w1 = pack_bf2(o[i][2] * inv1, o[i][3] * inv1);
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sw_addr<D>(sQ, t0, i) + (uint32_t)c2 * 2), "r"(w0) : "memory");
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sw_addr<D>(sQ, t1, i) + (uint32_t)c2 * 2), "r"(w1) : "memory");
            }
            if ((lane & 3) == 0) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int t = half ? t1 : t0;
                    if (t >= task_lo && t < tasks) {
                        const int cc = t / per_chunk, tt = t - cc * per_chunk;
                        const int r = tt / G, h = hk * G + (tt - r * G);
                        const int64_t aug = row0 + (int64_t)cc * s + a.k + r;
                        if (ksa_out_row_ok(a, aug, h))
                            a.lse[(int64_t)h * a.total_aug + aug] = ((half ? mx1 : mx0) + log2f(half ? l1 : l0)) * 0.6931471805599453f;
                    }
                }
            }
            __syncwarp();
#pragma unroll
            for (int it = 0; it < 16 * CH / 32; ++it) {
                const int idx = it * 32 + lane;
                const int rl = idx / CH, c = idx - rl * CH;
                const int t = mt * 16 + rl;
                if (t < task_lo || t >= tasks) continue;
                const int cc = t / per_chunk, tt = t - cc * per_chunk;
                const int r = tt / G, h = hk * G + (tt - r * G);
                const int64_t aug = row0 + (int64_t)cc * s + a.k + r;
                if (!ksa_out_row_ok(a, aug, h)) continue;
                uint4 val;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(sw_addr<D>(sQ, t, c)));
                *reinterpret_cast<uint4*>(a.out + aug * a.o_st + (int64_t)h * a.o_sh + c * 8) = val;
            }
        }
    }
}

std::mutex g_attr_mutex;
bool g_attr_done[64] = {};

}  // namespace

// Chunks per block: short chunks are stacked until the block has up to 64 query rows, within the row and key limits.
static int summ_chunks_per_block(const KernelArgs& a)
{
    const int G = a.Hq / a.Hkv, per_chunk = a.m * G, s = a.k + a.m;
    int c = 64 / per_chunk;
    c = std::min(c, std::min(kMmaMaxKeys / s, kMmaMaxRows / per_chunk));
    return std::max(c, 1);
}

// True if the kernel takes this shape (rows and keys within its register and shared-memory budget).
bool summary_mma_applies(const KernelArgs& a)
{
    const int G = a.Hq / a.Hkv;
    return a.m > 0 && a.k + a.m <= kMmaMaxKeys && a.m * G <= kMmaMaxRows;
}

cudaError_t launch_summary_mma(const KernelArgs& a, int max_chunks, unsigned ny, cudaStream_t stream)
{
    const int G = a.Hq / a.Hkv;
    const int cpb = summ_chunks_per_block(a);
    const int s_pad = (cpb * (a.k + a.m) + 15) / 16 * 16, m_pad = (cpb * a.m * G + 15) / 16 * 16;
    const size_t smem = (size_t)(m_pad + 2 * s_pad) * a.D * 2;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) {
        std::lock_guard<std::mutex> lock(g_attr_mutex);          // the shared-memory opt-in is a per-device setting
        if (!g_attr_done[dev]) {
            const int cap = (kMmaMaxRows + 2 * kMmaMaxKeys) * 128 * 2;
            if ((e = cudaFuncSetAttribute(ksa_summary_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap)) != cudaSuccess) return e;
            if ((e = cudaFuncSetAttribute(ksa_summary_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap / 2)) != cudaSuccess) return e;
            g_attr_done[dev] = true;
        }
    }
    // aligned groups of cpb chunks that the chunk range [j_first, j_first + max_chunks) touches
    const int j_first = a.r_seq >= 0 ? a.r_summ0 / a.m : 0;
    dim3 grid((unsigned)((j_first + max_chunks - 1) / cpb - j_first / cpb + 1), ny, (unsigned)a.Hkv);
    if (a.D == 128) ksa_summary_mma_kernel<128><<<grid, 128, smem, stream>>>(a, s_pad, m_pad, cpb);
    else            ksa_summary_mma_kernel<64><<<grid, 128, smem, stream>>>(a, s_pad, m_pad, cpb);
    return cudaGetLastError();
}

}  // namespace ksa
