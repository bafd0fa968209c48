// Gradients of the summary rows of long chunks on the tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32).
//
// Per (chunk, KV head) the summary rows are M = m G query rows (summary r, query head g of the group) over the chunk's
// k + m keys (Sec. 2.2.1): with P recomputed from q, k and the forward's lse,
//   dP = dO V^T,  delta = rowsum(P o dP) (= <dO, O>),  dS = P o (dP - delta),
//   dQ = scale dS K,  dV = P^T dO,  dK = scale dS^T Q.
// One block of four warps per (chunk, KV head) -- or per group of consecutive chunks where a chunk alone has fewer than 16
// query rows: their rows and keys are stacked, and a row sees keys of its own chunk only -- : Q, dO, K, V rows staged in shared memory (cp.async, 16-byte chunks
// XOR-swizzled by row for ldmatrix).  Phase 1, a warp per 16 query rows: S and dP on the tensor cores, P, delta and
// dS in registers, dQ = dS K with dS taken from the accumulator registers as the A operand; P and dS also go to shared
// memory as bf16.  Phase 2, a warp per 16 keys: dV and dK as products over the query rows, with P^T and dS^T read
// through ldmatrix.trans; one vector atomic per element and block into the fp32 accumulators of the key streams (the
// text keys of the chunk also collect from the text rows' kernels), instead of one per element and query row.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "ksa_bwd.h"

namespace ksa {

namespace {

constexpr int kBsMaxKeys = 128;       // k + m, padded to a multiple of 16
constexpr int kBsMaxRows = 128;       // m G, padded to a multiple of 16

__device__ __forceinline__ uint32_t bs_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bs_ldsm(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void bs_ldsm_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void bs_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t bs_pack(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bs_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// rows of D bf16, 16-byte chunk c of row r stored at chunk position c ^ (r & 7)
template <int D>
__device__ __forceinline__ uint32_t bs_sw(uint32_t base, int row, int chunk)
{
    return base + (uint32_t)row * (uint32_t)(D * 2) + (uint32_t)(((chunk ^ (row & 7)) & (D / 8 - 1)) << 4);
}

template <int D>
__global__ void __launch_bounds__(128, 2) ksa_bwd_summary_mma_kernel(BwdArgs a, int s_pad, int m_pad, int cpb)
{
    constexpr int CH = D / 8;
    constexpr int KT_MAX = kBsMaxKeys / 16;
    extern __shared__ __align__(128) uint16_t bs_smem[];
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int j = blockIdx.x * cpb, hk = blockIdx.z;                   // first chunk of the block
    const int here = min(cpb, sq.n_summ / a.m - j);                    // chunks of this block
    if (here <= 0) return;                                             // block-uniform
    const int G = a.Hq / a.Hkv, per_chunk = a.m * G, s = a.k + a.m;
    const int tasks = here * per_chunk, keys = here * s;               // stacked query rows and keys
    const int own = (a.flags & 1u) ? 0 : 1;
    const int64_t row0 = sq.aug_off + (int64_t)j * s;                  // first row of the chunk
    const int pstride = (s_pad + 8) * 2;                               // bytes per row of P / dS (conflict-free for ldmatrix)
    const uint32_t sQ = bs_u32(bs_smem);
    const uint32_t sG = sQ + (uint32_t)m_pad * D * 2;
    const uint32_t sK = sG + (uint32_t)m_pad * D * 2;
    const uint32_t sV = sK + (uint32_t)s_pad * D * 2;
    const uint32_t sP = sV + (uint32_t)s_pad * D * 2;
    const uint32_t sS = sP + (uint32_t)m_pad * pstride;
    const uint32_t sO = sS + (uint32_t)m_pad * pstride;                // per warp 16 rows of dQ on their way out
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- stage Q, dO (row t = summary t / G, query head hk G + t % G), K, V; padding rows are zeros ----
    for (int idx = threadIdx.x; idx < 2 * (m_pad + s_pad) * CH; idx += blockDim.x) {
        const int rr = idx / CH, c = idx - rr * CH;
        const uint16_t* src = a.kx + row0 * a.k_st + (int64_t)hk * a.k_sh;   // a valid address for the zero-filled rows
        uint32_t bytes = 0, dst;
        if (rr < 2 * m_pad) {
            const int t = rr < m_pad ? rr : rr - m_pad;
            if (t < tasks) {
                const int cc = t / per_chunk, tt = t - cc * per_chunk;
                const int r = tt / G, h = hk * G + (tt - r * G);
                const int64_t qrow = row0 + (int64_t)cc * s + a.k + r;
                src = rr < m_pad ? a.q + qrow * a.q_st + (int64_t)h * a.q_sh + c * 8
                                 : a.dout + qrow * a.do_st + (int64_t)h * a.do_sh + c * 8;
                bytes = 16;
            }
            dst = bs_sw<D>(rr < m_pad ? sQ : sG, t, c);
        } else {
            const int kr0 = rr - 2 * m_pad, kr = kr0 < s_pad ? kr0 : kr0 - s_pad;
            if (kr < keys) {
                src = kr0 < s_pad ? a.kx + (row0 + kr) * a.k_st + (int64_t)hk * a.k_sh + c * 8
                                  : a.v + (row0 + kr) * a.v_st + (int64_t)hk * a.v_sh + c * 8;
                bytes = 16;
            }
            dst = bs_sw<D>(kr0 < s_pad ? sK : sV, kr, c);
        }
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    const int mi = lane >> 3, r8 = lane & 7;      // ldmatrix: matrix index, row within the matrix
    const int g0 = lane >> 2, c2 = (lane & 3) * 2; // accumulator fragment: row (and row + 8), column pair
    const int kt_run = s_pad / 16;
    const float sl2 = a.scale * 1.4426950408889634f;

    // =============================== phase 1: a warp per 16 query rows ===============================
    for (int mt = warp; mt < m_pad / 16; mt += 4) {
        float sc[2 * KT_MAX][4], dp[2 * KT_MAX][4];
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) { sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f; dp[n][0] = dp[n][1] = dp[n][2] = dp[n][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t qa[4], ga[4];
            bs_ldsm(qa, bs_sw<D>(sQ, mt * 16 + r8 + 8 * (mi & 1), 2 * kk + (mi >> 1)));
            bs_ldsm(ga, bs_sw<D>(sG, mt * 16 + r8 + 8 * (mi & 1), 2 * kk + (mi >> 1)));
#pragma unroll
            for (int kt = 0; kt < KT_MAX; ++kt) {
                if (kt < kt_run) {
                    uint32_t kb[4], vb[4];
                    bs_ldsm(kb, bs_sw<D>(sK, kt * 16 + r8 + 8 * (mi >> 1), 2 * kk + (mi & 1)));
                    bs_ldsm(vb, bs_sw<D>(sV, kt * 16 + r8 + 8 * (mi >> 1), 2 * kk + (mi & 1)));
                    bs_mma(sc[2 * kt], qa, kb[0], kb[1]);
                    bs_mma(sc[2 * kt + 1], qa, kb[2], kb[3]);
                    bs_mma(dp[2 * kt], ga, vb[0], vb[1]);
                    bs_mma(dp[2 * kt + 1], ga, vb[2], vb[3]);
                }
            }
        }
        // rows t0 = 16 mt + g0 and t0 + 8: visible keys [lo, lo + nk) of the stacked keys -- the row's own chunk
        // (Sec. 2.2.1) --, lse of the forward pass in log2 units
        const int t0 = mt * 16 + g0, t1 = t0 + 8;
        int lo0 = 0, lo1 = 0;
        uint32_t nk0 = 0, nk1 = 0;
        float l0 = 0.f, l1 = 0.f;
        if (t0 < tasks) {
            const int cc = t0 / per_chunk, tt = t0 - cc * per_chunk;
            const int r = tt / G, h = hk * G + (tt - r * G);
            lo0 = cc * s; nk0 = (uint32_t)(a.k + own * (r + 1));
            l0 = a.lse[(int64_t)h * a.total_aug + row0 + (int64_t)cc * s + a.k + r] * 1.4426950408889634f;
        }
        if (t1 < tasks) {
            const int cc = t1 / per_chunk, tt = t1 - cc * per_chunk;
            const int r = tt / G, h = hk * G + (tt - r * G);
            lo1 = cc * s; nk1 = (uint32_t)(a.k + own * (r + 1));
            l1 = a.lse[(int64_t)h * a.total_aug + row0 + (int64_t)cc * s + a.k + r] * 1.4426950408889634f;
        }
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) {
            if (n < 2 * kt_run) {
                const int key = n * 8 + c2;
                sc[n][0] = (uint32_t)(key - lo0) < nk0 ? bs_ex2(fmaf(sc[n][0], sl2, -l0)) : 0.f;
                sc[n][1] = (uint32_t)(key + 1 - lo0) < nk0 ? bs_ex2(fmaf(sc[n][1], sl2, -l0)) : 0.f;
                sc[n][2] = (uint32_t)(key - lo1) < nk1 ? bs_ex2(fmaf(sc[n][2], sl2, -l1)) : 0.f;
                sc[n][3] = (uint32_t)(key + 1 - lo1) < nk1 ? bs_ex2(fmaf(sc[n][3], sl2, -l1)) : 0.f;
                d0 = fmaf(sc[n][0], dp[n][0], fmaf(sc[n][1], dp[n][1], d0));
                d1 = fmaf(sc[n][2], dp[n][2], fmaf(sc[n][3], dp[n][3], d1));
            }
        }
        d0 += __shfl_xor_sync(0xffffffffu, d0, 1); d0 += __shfl_xor_sync(0xffffffffu, d0, 2);
        d1 += __shfl_xor_sync(0xffffffffu, d1, 1); d1 += __shfl_xor_sync(0xffffffffu, d1, 2);
        // dS = P (dP - delta); P and dS as bf16 to shared memory (row-major, rows = query rows) for phase 2
        uint32_t da[KT_MAX][4];
#pragma unroll
        for (int n = 0; n < 2 * KT_MAX; ++n) {
            if (n < 2 * kt_run) {
                dp[n][0] = sc[n][0] * (dp[n][0] - d0); dp[n][1] = sc[n][1] * (dp[n][1] - d0);
                dp[n][2] = sc[n][2] * (dp[n][2] - d1); dp[n][3] = sc[n][3] * (dp[n][3] - d1);
                const uint32_t p_lo = bs_pack(sc[n][0], sc[n][1]), p_hi = bs_pack(sc[n][2], sc[n][3]);
                const uint32_t s_lo = bs_pack(dp[n][0], dp[n][1]), s_hi = bs_pack(dp[n][2], dp[n][3]);
                const uint32_t off0 = (uint32_t)t0 * pstride + (uint32_t)(n * 8 + c2) * 2, off1 = (uint32_t)t1 * pstride + (uint32_t)(n * 8 + c2) * 2;
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sP + off0), "r"(p_lo) : "memory");
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sP + off1), "r"(p_hi) : "memory");
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sS + off0), "r"(s_lo) : "memory");
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sS + off1), "r"(s_hi) : "memory");
                da[n >> 1][(n & 1) * 2] = s_lo;                            // A fragments of dS for dQ = dS K
                da[n >> 1][(n & 1) * 2 + 1] = s_hi;
            }
        }
        // ---- dQ = scale dS K ----
        float o[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
#pragma unroll
        for (int kt = 0; kt < KT_MAX; ++kt) {
            if (kt < kt_run) {
#pragma unroll
                for (int n2 = 0; n2 < D / 16; ++n2) {
                    uint32_t kb[4];
                    bs_ldsm_t(kb, bs_sw<D>(sK, kt * 16 + r8 + 8 * (mi & 1), 2 * n2 + (mi >> 1)));
                    bs_mma(o[2 * n2], da[kt], kb[0], kb[1]);
                    bs_mma(o[2 * n2 + 1], da[kt], kb[2], kb[3]);
                }
            }
        }
        // rows to their augmented positions (Eq. 1) through the warp's own staging rows: a lane stores 16 bytes
        {
            const uint32_t sOw = sO + (uint32_t)warp * 16 * D * 2;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const uint32_t w0 = bs_pack(o[i][0] * a.scale, o[i][1] * a.scale), w1 = bs_pack(o[i][2] * a.scale, o[i][3] * a.scale);
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(bs_sw<D>(sOw, g0, i) + (uint32_t)c2 * 2), "r"(w0) : "memory");
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(bs_sw<D>(sOw, g0 + 8, i) + (uint32_t)c2 * 2), "r"(w1) : "memory");
            }
            __syncwarp();
#pragma unroll
            for (int it = 0; it < 16 * CH / 32; ++it) {
                const int idx = it * 32 + lane;
                const int rl = idx / CH, c = idx - rl * CH;
                const int t = mt * 16 + rl;
                if (t >= tasks) continue;
                const int cc = t / per_chunk, tt = t - cc * per_chunk;
                const int r = tt / G, h = hk * G + (tt - r * G);
                uint4 val;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(bs_sw<D>(sOw, rl, c)));
                *reinterpret_cast<uint4*>(a.dq + (row0 + (int64_t)cc * s + a.k + r) * a.dq_st + (int64_t)h * a.dq_sh + c * 8) = val;
            }
        }
    }
    __syncthreads();

    // =============================== phase 2: a warp per 16 keys ===============================
    for (int kt = warp; kt < kt_run; kt += 4) {
        // the accumulator rows of keys kt 16 + g0 and + 8: text rows of the chunk, then the chunk's own summaries
        float* acc_k[2]; float* acc_v[2];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int kidx = kt * 16 + g0 + 8 * half;
            const int kc = kidx / s, key = kidx - kc * s;              // chunk within the block, key within the chunk
            if (kidx < keys && key < a.k) {
                const size_t row = (size_t)hk * a.text_rows + sq.text_off + (size_t)(j + kc) * a.k + key;
                acc_k[half] = a.dkt + row * D; acc_v[half] = a.dvt + row * D;
            } else if (kidx < keys) {
                const size_t row = (size_t)hk * a.summ_rows + sq.summ_off + (size_t)(j + kc) * a.m + (key - a.k);
                acc_k[half] = a.dks + row * D; acc_v[half] = a.dvs + row * D;
            } else {
                acc_k[half] = nullptr; acc_v[half] = nullptr;
            }
        }
#pragma unroll
        for (int which = 0; which < 2; ++which) {                     // 0: dV = P^T dO, 1: dK = scale dS^T Q
            const uint32_t sA = which ? sS : sP, sB = which ? sQ : sG;
            float o[D / 8][4];
#pragma unroll
            for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
            for (int rk = 0; rk < m_pad / 16; ++rk) {
                uint32_t pa[4];
                bs_ldsm_t(pa, sA + (uint32_t)(rk * 16 + r8 + 8 * (mi >> 1)) * pstride + (uint32_t)(kt * 16 + 8 * (mi & 1)) * 2);
#pragma unroll
                for (int n2 = 0; n2 < D / 16; ++n2) {
                    uint32_t gb[4];
                    bs_ldsm_t(gb, bs_sw<D>(sB, rk * 16 + r8 + 8 * (mi & 1), 2 * n2 + (mi >> 1)));
                    bs_mma(o[2 * n2], pa, gb[0], gb[1]);
                    bs_mma(o[2 * n2 + 1], pa, gb[2], gb[3]);
                }
            }
            const float mul = which ? a.scale : 1.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float* acc = which ? acc_k[half] : acc_v[half];
                if (acc == nullptr) continue;
#pragma unroll
                for (int i = 0; i < D / 8; ++i)
                    atomicAdd(reinterpret_cast<float2*>(acc + i * 8 + c2), make_float2(o[i][2 * half] * mul, o[i][2 * half + 1] * mul));
            }
        }
    }
}

std::mutex g_bs_mutex;
bool g_bs_done[64] = {};

size_t bs_smem_bytes(int D, int s_pad, int m_pad)
{
    return (size_t)2 * (m_pad + s_pad) * D * 2 + (size_t)2 * m_pad * (s_pad + 8) * 2 + (size_t)4 * 16 * D * 2;
}

}  // namespace

// Chunks per block: as many as it takes to fill a 16-row tile, within the kernel's row and key limits.
static int bs_chunks_per_block(const BwdArgs& a)
{
    const int G = a.Hq / a.Hkv, per_chunk = a.m * G, s = a.k + a.m;
    int c = (16 + per_chunk - 1) / per_chunk;
    c = std::min(c, std::min(kBsMaxKeys / s, kBsMaxRows / per_chunk));
    return std::max(c, 1);
}

bool bwd_summary_mma_applies(const BwdArgs& a)
{
    const int G = a.Hq / a.Hkv;
    return a.m > 0 && a.k + a.m <= kBsMaxKeys && a.m * G <= kBsMaxRows;
}

cudaError_t launch_bwd_summary_mma(const BwdArgs& a, cudaStream_t stream)
{
    const int G = a.Hq / a.Hkv;
    const int cpb = bs_chunks_per_block(a);
    const int s_pad = (cpb * (a.k + a.m) + 15) / 16 * 16, m_pad = (cpb * a.m * G + 15) / 16 * 16;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) {
        std::lock_guard<std::mutex> lock(g_bs_mutex);            // the shared-memory opt-in is a per-device setting
        if (!g_bs_done[dev]) {
            if ((e = cudaFuncSetAttribute(ksa_bwd_summary_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)bs_smem_bytes(128, kBsMaxKeys, kBsMaxRows))) != cudaSuccess) return e;
            if ((e = cudaFuncSetAttribute(ksa_bwd_summary_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)bs_smem_bytes(64, kBsMaxKeys, kBsMaxRows))) != cudaSuccess) return e;
            g_bs_done[dev] = true;
        }
    }
    const int max_chunks = a.max_n_summ / a.m;
    dim3 grid((unsigned)((max_chunks + cpb - 1) / cpb), (unsigned)a.num_seqs, (unsigned)a.Hkv);
    const size_t smem = bs_smem_bytes(a.D, s_pad, m_pad);
    if (a.D == 128) ksa_bwd_summary_mma_kernel<128><<<grid, 128, smem, stream>>>(a, s_pad, m_pad, cpb);
    else            ksa_bwd_summary_mma_kernel<64><<<grid, 128, smem, stream>>>(a, s_pad, m_pad, cpb);
    return cudaGetLastError();
}

}  // namespace ksa
