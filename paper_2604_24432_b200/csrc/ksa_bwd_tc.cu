// dK / dV of the backward pass on the sm_100a tensor cores (head_dim 128).
//
// Key-stationary and transposed, like the mma.sync kernel it replaces for D = 128: a CTA owns one
// tile of 128 keys of one KV head (text stream or summary stream) and walks a segment of the
// (query tile, query head) pairs that see it.  TMEM (512 columns): ST = K Q^T [0,128),
// DPT = V dO^T [128,256), dV [256,384), dK [384,512); lanes are the 128 keys.  Per pair:
//   MMA     ST = K Q^T, DPT = V dO^T (shared memory x shared memory)              -> s_full
//   warps   P^T = exp2(ST scale - lse_q) on visible pairs, dS^T = P^T (DPT - delta_q); both as
//           bf16 over the first 16 columns of each 32-column chunk of ST / DPT    -> p_full
//   MMA     dV += P^T dO, dK += dS^T Q (A from TMEM, B = the dO / Q tile read MN-major)
// The Q and dO tiles stream through two shared-memory stages filled by TMA; K and V stay.
// At the end each key row adds its dV and scale * dK to the fp32 accumulators of the stream
// (vector atomics: several segments and the summary-row kernel add to the same rows).
// Warps 0-7: one key row per thread, two warps per row quarter (warp w and w + 4 share the lanes
// 32 (w % 4) ..; each takes two of the four 32-column chunks of the query tile); warp 8: TMA
// producer; warp 9: MMA issuer.
// Every mbarrier wait is bounded (status word + CTA-wide abort flag, as in the forward kernel).
#include <cuda_bf16.h>

#include <algorithm>

#include "ksa_bwd.h"
#include "ksa_ptx.cuh"

namespace ksa {

using namespace ptx;

constexpr int kBwdTcThreads = 320;
constexpr int kBwdSegTiles = 8;                 // query tiles (of 128 rows) per segment
constexpr int kBwdTileBytes = 128 * 128 * 2;    // one 128 x 128 bf16 tile

// shared memory map (bytes from the 1024-aligned base)
constexpr int kOffK = 0, kOffV = kBwdTileBytes, kOffQ = 2 * kBwdTileBytes;            // Q stage s at kOffQ + s * 2 tiles, dO right after Q
constexpr int kOffBars = 6 * kBwdTileBytes;                                           // 8 barriers
constexpr int kOffMisc = kOffBars + 64;                                               // TMEM slot, abort flags
constexpr int kOffRow = kOffMisc + 64;                                                // [8 warps][3][64] per-query scalars
constexpr int kBwdTcSmem = kOffRow + 8 * 3 * 64 * 4 + 1024;
enum : int { BB_KVFULL = 0, BB_QFULL = 1, BB_QEMPTY = 3, BB_SFULL = 5, BB_PFULL = 6, BB_OFULL = 7 };

__device__ __forceinline__ uint32_t bt_ld_shared(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void bt_st_shared(uint32_t addr, uint32_t v)
{
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ bool bt_wait(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (bt_ld_shared(abort_addr) != 0u) return false;
            if (clock64() - t0 > (1ll << 31)) {
                atomicCAS(status, 0, code);
                bt_st_shared(abort_addr, 1u);
                return false;
            }
        }
    }
}

__global__ void __launch_bounds__(kBwdTcThreads, 1)
ksa_bwd_dkv_tc_kernel(const __grid_constant__ BwdArgs a, const __grid_constant__ BwdMaps maps, const int summ)
{
    extern __shared__ uint8_t bsm_raw[];
    const uint32_t base = (smem_u32(bsm_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = bsm_raw + (base - smem_u32(bsm_raw));
    const uint32_t sK = base + kOffK, sV = base + kOffV;
    auto sQ = [&](int st) -> uint32_t { return base + kOffQ + (uint32_t)st * 2u * kBwdTileBytes; };
    auto sG = [&](int st) -> uint32_t { return sQ(st) + kBwdTileBytes; };
    auto bar = [&](int i) -> uint32_t { return base + kOffBars + 8u * (uint32_t)i; };
    const uint32_t tmem_slot = base + kOffMisc, abort_addr = tmem_slot + 4;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- which keys, which queries (Eq. 3) ------------------------------------------------------
    const int G = a.Hq / a.Hkv;
    const int hk = blockIdx.z % a.Hkv, b = blockIdx.z / a.Hkv;
    const SeqInfo sq = a.seqs[b];
    const int kt = blockIdx.y;
    const int n_keys = summ ? sq.n_summ : sq.n_text;
    if (kt * 128 >= n_keys) return;
    const int n_qt = (sq.n_text + 127) / 128;
    int qt_lo, qt_hi;
    if (!summ) {
        const int key_last = min(n_keys, kt * 128 + 128) - 1;
        qt_lo = kt;
        const long long i_max = ((long long)(key_last / a.k) + a.C + 1) * a.k - 1;
        qt_hi = (int)min((long long)(n_qt - 1), i_max / 128);
    } else {
        const long long i_min = ((long long)(kt * 128) / a.m + 1 + a.C) * a.k;     // first row that sees summary kt*128
        if (i_min >= sq.n_text) return;
        qt_lo = (int)(i_min / 128);
        qt_hi = n_qt - 1;
    }
    const int seg0 = qt_lo + (int)blockIdx.x * kBwdSegTiles;
    if (seg0 > qt_hi) return;
    const int seg1 = min(qt_hi + 1, seg0 + kBwdSegTiles);
    const int iters = (seg1 - seg0) * G;
    const int krow0 = (summ ? sq.summ_off : sq.text_off) + kt * 128;      // first row of the tile in its packed stream

    if (tid == 0) {
        mbar_init(bar(BB_KVFULL), 1);
        for (int s = 0; s < 2; ++s) { mbar_init(bar(BB_QFULL + s), 1); mbar_init(bar(BB_QEMPTY + s), 1); }
        mbar_init(bar(BB_SFULL), 1);
        mbar_init(bar(BB_PFULL), 8);
        mbar_init(bar(BB_OFULL), 1);
        bt_st_shared(abort_addr, 0u);
        bt_st_shared(abort_addr + 4, 0u);
        fence_mbar_init();
    }
    if (warp == 8) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bt_ld_shared(tmem_slot);

    if (warp == 8) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.qt); prefetch_tensormap(&maps.dot);
            const CUtensorMap* mk = summ ? &maps.ks : &maps.kt;
            const CUtensorMap* mv = summ ? &maps.vs : &maps.vt;
            mbar_arrive_expect_tx(bar(BB_KVFULL), 2u * kBwdTileBytes);
            for (int h2 = 0; h2 < 2; ++h2) {
                tma_load_3d(sK + h2 * 16384, mk, bar(BB_KVFULL), h2 * 64, krow0, hk);
                tma_load_3d(sV + h2 * 16384, mv, bar(BB_KVFULL), h2 * 64, krow0, hk);
            }
            int last_it[2] = {-1, -1};
            for (int it = 0; it < iters; ++it) {
                const int st = it & 1;
                if (!bt_wait(bar(BB_QEMPTY + st), ((it >> 1) & 1) ^ 1u, abort_addr, a.status, kStatusWaitQEmpty)) break;
                const int qt = seg0 + it / G, h = hk * G + it % G;
                mbar_arrive_expect_tx(bar(BB_QFULL + st), 2u * kBwdTileBytes);
                last_it[st] = it;
                for (int h2 = 0; h2 < 2; ++h2) {
                    tma_load_3d(sQ(st) + h2 * 16384, &maps.qt, bar(BB_QFULL + st), h2 * 64, sq.text_off + qt * 128, h);
                    tma_load_3d(sG(st) + h2 * 16384, &maps.dot, bar(BB_QFULL + st), h2 * 64, sq.text_off + qt * 128, h);
                }
            }
            if (bt_ld_shared(abort_addr) != 0u) {
                // gave up: leave no copy in flight (bounded waits on what was issued last; the second flag is never set)
                bt_wait(bar(BB_KVFULL), 0, abort_addr + 4, a.status, kStatusWaitKvFull);
                for (int st = 0; st < 2; ++st)
                    if (last_it[st] >= 0) bt_wait(bar(BB_QFULL + st), (last_it[st] >> 1) & 1, abort_addr + 4, a.status, kStatusWaitQFull);
            }
        }
    } else if (warp == 9) {
        // =============================== MMA issuer =================================
        if (lane == 0) {
            constexpr uint32_t idesc_kmajor = make_idesc_bf16(128, 128, false);     // both operands K-major
            constexpr uint32_t idesc_mnb = make_idesc_bf16(128, 128, true);         // B read MN-major
            const uint64_t kd = make_smem_desc_sw128(sK, 16, 1024), vd = make_smem_desc_sw128(sV, 16, 1024);
            bool alive = bt_wait(bar(BB_KVFULL), 0, abort_addr, a.status, kStatusWaitKvFull);
            uint32_t pf_phase = 0;
            for (int it = 0; it < iters && alive; ++it) {
                const int st = it & 1;
                if (!bt_wait(bar(BB_QFULL + st), (it >> 1) & 1, abort_addr, a.status, kStatusWaitQFull)) break;
                tc_fence_after();
                const uint64_t qd = make_smem_desc_sw128(sQ(st), 16, 1024), gd = make_smem_desc_sw128(sG(st), 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    mma_ss(tmem + 0, kd + off, qd + off, idesc_kmajor, kk > 0 ? 1u : 0u);          // ST = K Q^T
                }
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    mma_ss(tmem + 128, vd + off, gd + off, idesc_kmajor, kk > 0 ? 1u : 0u);        // DPT = V dO^T
                }
                tc_commit(bar(BB_SFULL));
                if (!bt_wait(bar(BB_PFULL), pf_phase, abort_addr, a.status, kStatusWaitPFull)) break;
                pf_phase ^= 1u;
                tc_fence_after();
                const uint64_t gmn = make_smem_desc_sw128(sG(st), 16384, 1024), qmn = make_smem_desc_sw128(sQ(st), 16384, 1024);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)                                                       // dV += P^T dO
                    mma_ts(tmem + 256, tmem + 0 + (kk >> 1) * 32 + (kk & 1) * 8, gmn + (uint32_t)((kk * 2048) >> 4), idesc_mnb, (it > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)                                                       // dK += dS^T Q
                    mma_ts(tmem + 384, tmem + 128 + (kk >> 1) * 32 + (kk & 1) * 8, qmn + (uint32_t)((kk * 2048) >> 4), idesc_mnb, (it > 0 || kk > 0) ? 1u : 0u);
                tc_commit(bar(BB_QEMPTY + st));
            }
            tc_commit(bar(BB_OFULL));
        }
    } else {
        // =============================== key rows ===================================
        const int quarter = warp & 3, half = warp >> 2;                  // lanes 32 quarter ..; chunks half and half + 2
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t tST = tmem + lane_sel, tDP = tmem + lane_sel + 128u;
        const int key_raw = kt * 128 + quarter * 32 + lane;
        const int key = key_raw < n_keys ? key_raw : 0x7fffffff;        // rows past the stream never match
        float* rowf = reinterpret_cast<float*>(base_ptr + kOffRow) + warp * 3 * 64;      // this warp's lse / delta / bound
        int* rowi = reinterpret_cast<int*>(rowf + 2 * 64);
        uint32_t sf_phase = 0;
        bool alive = true;
        for (int it = 0; it < iters; ++it) {
            const int qt = seg0 + it / G, h = hk * G + it % G;
            const size_t r = (size_t)h * a.text_rows + sq.text_off + (size_t)qt * 128;
            __syncwarp();
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int slot = e * 32 + lane;                           // slot j of pass e <-> column (half + 2 e) * 32 + j
                const int col = (half + 2 * e) * 32 + lane, i = qt * 128 + col;
                rowf[slot] = a.lse_t[r + col];
                rowf[64 + slot] = a.delta_t[r + col];
                const int far = max(0, i / a.k - a.C);
                rowi[slot] = (i >= sq.n_text) ? (summ ? 0 : 0x7fffffff) : (summ ? min(sq.n_summ, far * a.m) : far * a.k);
            }
            __syncwarp();
            bool ok = bt_wait(bar(BB_SFULL), sf_phase, abort_addr, a.status, kStatusWaitSFull);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { alive = false; break; }
            sf_phase ^= 1u;
            tc_fence_after();
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int c = half + 2 * e;                               // 32-column chunk of the query tile
                const int i0 = qt * 128 + c * 32;
                uint32_t st_[32], dp_[32];
                tmem_ld32(tST + c * 32, st_);
                tmem_ld32(tDP + c * 32, dp_);
                tc_wait_ld();
                uint32_t pp[16], dd[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float pv[2], dv[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int slot = e * 32 + j + u;
                        const bool vis = summ ? (key < rowi[slot]) : (key <= i0 + j + u && key >= rowi[slot]);
                        const float p = vis ? ex2_approx(fmaf(__uint_as_float(st_[j + u]), a.scale_log2, -rowf[slot])) : 0.f;
                        pv[u] = p;
                        dv[u] = vis ? p * (__uint_as_float(dp_[j + u]) - rowf[64 + slot]) : 0.f;
                    }
                    pp[j >> 1] = pack_bf16x2(pv[0], pv[1]);
                    dd[j >> 1] = pack_bf16x2(dv[0], dv[1]);
                }
                // bf16 results over the first 16 columns of the chunk's own fp32 columns: no other warp reads those
                tmem_st16(tST + c * 32, pp);
                tmem_st16(tDP + c * 32, dd);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BB_PFULL));
        }
        if (alive) {
            bool ok = bt_wait(bar(BB_OFULL), 0, abort_addr, a.status, kStatusWaitOFull);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                // half 0 adds dV, half 1 adds scale * dK (tcgen05.ld is warp-collective: rows past the stream load, too)
                const size_t arow = (size_t)hk * (summ ? a.summ_rows : a.text_rows) + (size_t)krow0 + quarter * 32 + lane;
                float* acc = (half ? (summ ? a.dks : a.dkt) : (summ ? a.dvs : a.dvt)) + arow * 128;
                const float mul = half ? a.scale : 1.f;
                const uint32_t tacc = tmem + lane_sel + (half ? 384u : 256u);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tacc + c * 32, o);
                    tc_wait_ld();
                    if (key_raw < n_keys) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            atomicAdd(reinterpret_cast<float4*>(acc + c * 32 + e),
                                      make_float4(__uint_as_float(o[e]) * mul, __uint_as_float(o[e + 1]) * mul,
                                                  __uint_as_float(o[e + 2]) * mul, __uint_as_float(o[e + 3]) * mul));
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

cudaError_t setup_bwd_tc()
{
    return cudaFuncSetAttribute(ksa_bwd_dkv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdTcSmem);
}

cudaError_t launch_bwd_dkv_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream)
{
    const int n_qt = a.max_text_pad / 128;
    const long long text_span = std::min<long long>(n_qt, ((long long)a.C + 1) * a.k / 128 + 2);
    for (int summ = 0; summ < 2; ++summ) {
        if (summ && (a.m <= 0 || a.max_n_summ <= 0)) continue;
        const long long span = summ ? n_qt : text_span;
        const int tiles = summ ? (a.max_n_summ + 127) / 128 : n_qt;
        dim3 grid((unsigned)((span + kBwdSegTiles - 1) / kBwdSegTiles), (unsigned)tiles, (unsigned)(a.num_seqs * a.Hkv));
        ksa_bwd_dkv_tc_kernel<<<grid, kBwdTcThreads, kBwdTcSmem, stream>>>(a, maps, summ);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace ksa
