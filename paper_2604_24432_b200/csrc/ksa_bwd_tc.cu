// Backward pass of the text rows on the sm_100a tensor cores (head_dim 128): dK / dV and dQ.
//
// Both kernels keep two 128-row operand tiles resident in shared memory, stream 64-row half
// tiles of the other two operands through four TMA-filled slots, and run the same software
// pipeline over "half iterations" u = 0, 1, 2, ...:
//   MMA     X_u = A1 B1_u^T, Y_u = A2 B2_u^T   (128 x 64, shared memory x shared memory) -> s_full[u & 1]
//   warps   P = exp2(X scale - lse) on visible pairs, dS = P (Y - delta); as bf16 over the
//           first 8 columns of each 16-column chunk of X / Y                             -> p_full[u & 1]
//   MMA     accumulators += (bf16 from TMEM) x (the streamed half tile read MN-major)
// The tensor pipe works in order, so s_full of u + 2 also tells the producer that slot u & 3 is free again.
// The issuing thread pays a few hundred cycles per wait / fence / commit while the tensor pipe runs dry
// (its queue is short), so it waits once per half iteration: row warp 0 checks the slot of u + 2 before
// it arrives on p_full[u & 1].
// The two TMEM buffers (u even / odd) let the products of u + 1 and the accumulations of u - 1
// run while the warps work on u.  TMEM (512 columns): X0 [0,64) X1 [64,128) Y0 [128,192)
// Y1 [192,256), accumulators from 256.
//
//   dK / dV  key-stationary and transposed: A1 = K tile, A2 = V tile (text or summary stream),
//            B1 = Q half tile, B2 = dO half tile of the (query tile, query head) pairs that see
//            the keys; X = S^T, Y = dP^T; dV += P^T dO, dK += dS^T Q; at the end each key row
//            adds dV and scale * dK to the fp32 accumulators of its stream (vector atomics:
//            several segments and the summary-row kernel add to the same rows).
//   dQ       query-stationary: A1 = Q tile, A2 = dO tile, B1 = K half tile, B2 = V half tile over
//            the visible summary tiles, then the visible text tiles (Eq. 3); X = S, Y = dP;
//            dQ += dS K; at the end scale * dQ goes to the caller's tensor as bf16.
//
// Warps 0-15: one accumulator row per thread, four warps per row quarter (warps w, w + 4, w + 8, w + 12
// share the lanes 32 (w % 4) ..; each takes one 16-column chunk of a half tile: the element-wise work has
// no reduction across columns, and four warps per scheduler hide the TMEM load / store latencies);
// warp 16: TMA producer; warp 17: MMA issuer.  Every mbarrier wait is bounded (status word + CTA-wide
// abort flag).
#include <cuda_bf16.h>

#include <algorithm>

#include "ksa_bwd.h"
#include "ksa_ptx.cuh"

namespace ksa {

using namespace ptx;

constexpr int kBwdTcThreads = 576;
constexpr int kBwdTcRegs = 96;                  // 18 warps: five on a scheduler, 5 x 32 x 96 registers fit its file
constexpr int kBwdSegTiles = 16;                // dK / dV: query tiles (of 128 rows) per CTA
constexpr int kBwdTileBytes = 128 * 128 * 2;    // one 128 x 128 bf16 tile: [d half][128 rows][128 B]
constexpr int kBwdSlotBytes = 2 * 64 * 128 * 2; // two 64 x 128 half tiles, each [d half][64 rows][128 B]

// shared memory map (bytes from the 1024-aligned base)
constexpr int kOffA1 = 0, kOffA2 = kBwdTileBytes, kOffSlots = 2 * kBwdTileBytes;
constexpr int kOffBars = kOffSlots + 4 * kBwdSlotBytes;                               // 10 barriers
constexpr int kOffMisc = kOffBars + 128;                                              // TMEM slot, abort flags
constexpr int kOffRow = kOffMisc + 64;                                                // dK / dV: [16 warps][2][3][32] per-query scalars
constexpr int kBwdTcSmem = kOffRow + 16 * 2 * 3 * 32 * 4 + 1024;
// Optional event trace (compile with -DKSA_BWD_TRACE): one CTA of the dQ kernel records (event id, clock)
// pairs for the MMA issuer and lane 0 of every row warp; ksa_debug_read_bwd_trace() copies them out.
#ifdef KSA_BWD_TRACE
constexpr int kBtEvents = 4096;
__device__ uint2 g_btrace[17][kBtEvents];         // role 0: MMA issuer; 1 + w: row warp w
__device__ uint32_t g_btrace_cnt[17];
#define KSA_BT(role, id)                                                                         \
    do {                                                                                         \
        if (bt_on && bt_n < (uint32_t)kBtEvents) g_btrace[role][bt_n++] = make_uint2((uint32_t)(id), (uint32_t)clock()); \
    } while (0)
#else
#define KSA_BT(role, id) do { } while (0)
#endif

enum : int { BB_AFULL = 0, BB_QFULL = 1, BB_SFULL = 5, BB_PFULL = 7, BB_OFULL = 9 };

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

// The MMA issuer's wait: its time is the kernel's critical path, and a try_wait costs it a few hundred cycles
// even when the phase is already complete; test_wait returns at once, so it spins on that.
__device__ __forceinline__ bool bt_wait_spin(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status, int code)
{
    if (mbar_test_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (bt_ld_shared(abort_addr) != 0u) return false;
            if (clock64() - t0 > (1ll << 31)) {
                atomicCAS(status, 0, code);
                bt_st_shared(abort_addr, 1u);
                return false;
            }
        }
    }
}

// One lane polls for the warp (512 polling threads would crowd the barrier unit and slow the MMA issuer's waits).
__device__ __forceinline__ bool bt_wait_warp(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status, int code, int lane)
{
    bool ok = true;
    if (lane == 0) ok = bt_wait(bar, parity, abort_addr, status, code);
    return __shfl_sync(0xffffffffu, ok, 0);
}

// Shared-memory layout and barrier addresses of one CTA.
struct BtSmem {
    uint32_t base;
    __device__ __forceinline__ uint32_t a1() const { return base + kOffA1; }
    __device__ __forceinline__ uint32_t a2() const { return base + kOffA2; }
    __device__ __forceinline__ uint32_t b1(int slot) const { return base + kOffSlots + (uint32_t)slot * kBwdSlotBytes; }
    __device__ __forceinline__ uint32_t b2(int slot) const { return b1(slot) + kBwdSlotBytes / 2; }
    __device__ __forceinline__ uint32_t bar(int i) const { return base + kOffBars + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t tmem_slot() const { return base + kOffMisc; }
    __device__ __forceinline__ uint32_t abort_addr() const { return base + kOffMisc + 4; }
};

__device__ __forceinline__ void bt_init(const BtSmem& sm, int tid, int warp)
{
    if (tid == 0) {
        mbar_init(sm.bar(BB_AFULL), 1);
        for (int s = 0; s < 4; ++s) mbar_init(sm.bar(BB_QFULL + s), 1);
        for (int s = 0; s < 2; ++s) { mbar_init(sm.bar(BB_SFULL + s), 1); mbar_init(sm.bar(BB_PFULL + s), 16); }
        mbar_init(sm.bar(BB_OFULL), 1);
        bt_st_shared(sm.abort_addr(), 0u);
        bt_st_shared(sm.abort_addr() + 4, 0u);
        fence_mbar_init();
    }
    if (warp == 16) { tmem_alloc(sm.tmem_slot(), 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
}

// One MMA issuer's whole loop: the half iterations u = par, par + step, ...  kAcc = number of accumulators
// (2: dV from X and B2 at acc_col, dK from Y and B1 at acc_col + 128; 1: dQ from X and B1 at acc_col).
// acc_zeroed: the accumulators were cleared beforehand (issuers that share them cannot tell who is first).
template <int kAcc>
__device__ __forceinline__ void bt_mma_loop(const BtSmem& sm, uint32_t tmem, int U, int32_t* status, int par, int step,
                                            uint32_t acc_col, bool acc_zeroed, bool bt_on = false)
{
    uint32_t bt_n = 0;
    (void)bt_on; (void)bt_n;
#if defined(KSA_BWD_TRACE) && KSA_BWD_TRACE == 2
    uint32_t bt_wait_sum = 0;
    const uint32_t bt_t_begin = (uint32_t)clock();
    const bool bt_sum_on = bt_on;
    bt_on = false;
#endif
    constexpr uint32_t idesc_ss = make_idesc_bf16(128, 64, false);      // both operands K-major, N = 64
    constexpr uint32_t idesc_ts = make_idesc_bf16(128, 128, true);      // B read MN-major, N = 128
    const uint32_t abort_addr = sm.abort_addr();
    const uint64_t a1d = make_smem_desc_sw128(sm.a1(), 16, 1024), a2d = make_smem_desc_sw128(sm.a2(), 16, 1024);
    // wait_slot: only for the first ones; later slots were checked by row warp 0 before its p_full arrival
    auto products = [&](int u, bool wait_slot) -> bool {
        const int slot = u & 3, buf = u & 1;
        if (wait_slot && !bt_wait(sm.bar(BB_QFULL + slot), (u >> 2) & 1, abort_addr, status, kStatusWaitQFull)) return false;
        KSA_BT(0, 5);
        const uint64_t b1d = make_smem_desc_sw128(sm.b1(slot), 16, 1024), b2d = make_smem_desc_sw128(sm.b2(slot), 16, 1024);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
            mma_ss(tmem + buf * 64, a1d + (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4),
                   b1d + (uint32_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4), idesc_ss, kk > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
            mma_ss(tmem + 128 + buf * 64, a2d + (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4),
                   b2d + (uint32_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4), idesc_ss, kk > 0 ? 1u : 0u);
        KSA_BT(0, 6);
        tc_commit(sm.bar(BB_SFULL + buf));
        KSA_BT(0, 4);
#ifdef KSA_BWD_TRACE
        if (bt_on) { const uint32_t probe = bt_ld_shared(sm.abort_addr() + 4); if (probe == 12345u) bt_n = 0; KSA_BT(0, 30); }
#endif
        return true;
    };
    bool alive = bt_wait(sm.bar(BB_AFULL), 0, abort_addr, status, kStatusWaitKvFull);
    if (alive) alive = products(par, true);
    if (alive && step == 1 && U > 1) alive = products(1, true);
    for (int u = par; u < U && alive; u += step) {
        const int slot = u & 3, buf = u & 1;
#if defined(KSA_BWD_TRACE) && KSA_BWD_TRACE == 2
        const uint32_t tw0 = (uint32_t)clock();
#endif
        if (!bt_wait_spin(sm.bar(BB_PFULL + buf), (u >> 1) & 1, abort_addr, status, kStatusWaitPFull)) break;
#if defined(KSA_BWD_TRACE) && KSA_BWD_TRACE == 2
        bt_wait_sum += (uint32_t)clock() - tw0;
#endif
        KSA_BT(0, 1);
        tc_fence_after();
        KSA_BT(0, 7);
        // half tile read MN-major: 64-element atoms of d are 8192 bytes apart, 8-row groups 1024 bytes
        const uint64_t b1m = make_smem_desc_sw128(sm.b1(slot), 8192, 1024), b2m = make_smem_desc_sw128(sm.b2(slot), 8192, 1024);
        const bool later = acc_zeroed || u > par;
        if (kAcc == 2) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                mma_ts(tmem + acc_col, tmem + buf * 64 + kk * 16, b2m + (uint32_t)((kk * 2048) >> 4), idesc_ts,
                       (later || kk > 0) ? 1u : 0u);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                mma_ts(tmem + acc_col + 128, tmem + 128 + buf * 64 + kk * 16, b1m + (uint32_t)((kk * 2048) >> 4), idesc_ts,
                       (later || kk > 0) ? 1u : 0u);
        } else {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                mma_ts(tmem + acc_col, tmem + buf * 64 + kk * 16, b1m + (uint32_t)((kk * 2048) >> 4), idesc_ts,
                       (later || kk > 0) ? 1u : 0u);
        }
        KSA_BT(0, 2);
        if (u + 2 < U) alive = products(u + 2, false);
    }
    tc_commit(sm.bar(BB_OFULL));
#ifdef KSA_BWD_TRACE
    if (bt_on) g_btrace_cnt[0] = bt_n;
#if KSA_BWD_TRACE == 2
    if (bt_sum_on) { g_btrace[0][0] = make_uint2(bt_wait_sum, (uint32_t)clock() - bt_t_begin); g_btrace[0][1] = make_uint2((uint32_t)U, 0u); g_btrace_cnt[0] = 2; }
#endif
#endif
}

// Producer: slot u & 3 was last read by the accumulations of u - 4, and the products of u - 2 were issued after
// those, so their s_full completion frees the slot.  A parity wait only tells neighbouring phases apart:
// the first time round (u = 4, 5) the phase before is waited for as well.
__device__ __forceinline__ bool bt_slot_free(const BtSmem& sm, int u, int32_t* status)
{
    const uint32_t bar = sm.bar(BB_SFULL + (u & 1));
    if (u < 6 && !bt_wait(bar, 0, sm.abort_addr(), status, kStatusWaitQEmpty)) return false;
    return bt_wait(bar, ((u - 2) >> 1) & 1, sm.abort_addr(), status, kStatusWaitQEmpty);
}

// One TMA-filled slot: the 64 x 128 half tiles of two tensors (rows row .. row + 63 of head `head`).
__device__ __forceinline__ void bt_load_slot(const BtSmem& sm, int slot, const CUtensorMap* m1, const CUtensorMap* m2, int row, int head)
{
    const uint32_t bar = sm.bar(BB_QFULL + slot);
    mbar_arrive_expect_tx(bar, (uint32_t)kBwdSlotBytes);
    for (int h2 = 0; h2 < 2; ++h2) {
        tma_load_3d(sm.b1(slot) + h2 * 8192, m1, bar, h2 * 64, row, head);
        tma_load_3d(sm.b2(slot) + h2 * 8192, m2, bar, h2 * 64, row, head);
    }
}
// The two resident 128 x 128 tiles.
__device__ __forceinline__ void bt_load_resident(const BtSmem& sm, const CUtensorMap* m1, const CUtensorMap* m2, int row, int head)
{
    const uint32_t bar = sm.bar(BB_AFULL);
    mbar_arrive_expect_tx(bar, 2u * kBwdTileBytes);
    for (int h2 = 0; h2 < 2; ++h2) {
        tma_load_3d(sm.a1() + h2 * 16384, m1, bar, h2 * 64, row, head);
        tma_load_3d(sm.a2() + h2 * 16384, m2, bar, h2 * 64, row, head);
    }
}
// After an abort: leave no copy in flight (bounded waits on what was issued last; the second flag is never set).
__device__ __forceinline__ void bt_drain(const BtSmem& sm, const int (&last_u)[4], int32_t* status)
{
    bt_wait(sm.bar(BB_AFULL), 0, sm.abort_addr() + 4, status, kStatusWaitKvFull);
    for (int s = 0; s < 4; ++s)
        if (last_u[s] >= 0) bt_wait(sm.bar(BB_QFULL + s), (last_u[s] >> 2) & 1, sm.abort_addr() + 4, status, kStatusWaitQFull);
}

__global__ void __maxnreg__(kBwdTcRegs)
ksa_bwd_dkv_tc_kernel(const __grid_constant__ BwdArgs a, const __grid_constant__ BwdMaps maps, const int summ)
{
    extern __shared__ uint8_t bsm_raw[];
    BtSmem sm;
    sm.base = (smem_u32(bsm_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = bsm_raw + (sm.base - smem_u32(bsm_raw));
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
    const int iters = (seg1 - seg0) * G;                                  // (query tile, query head) pairs
    const int U = 2 * iters;                                              // half iterations
    const int krow0 = (summ ? sq.summ_off : sq.text_off) + kt * 128;      // first row of the tile in its packed stream

    bt_init(sm, tid, warp);
    const uint32_t tmem = bt_ld_shared(sm.tmem_slot());

    if (warp == 16) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.qt64); prefetch_tensormap(&maps.dot64);
            bt_load_resident(sm, summ ? &maps.ks : &maps.kt, summ ? &maps.vs : &maps.vt, krow0, hk);
            int last_u[4] = {-1, -1, -1, -1};
            for (int u = 0; u < U; ++u) {
                const int slot = u & 3, it = u >> 1;
                if (u >= 4 && !bt_slot_free(sm, u, a.status)) break;
                const int qt = seg0 + it / G, h = hk * G + it % G;
                bt_load_slot(sm, slot, &maps.qt64, &maps.dot64, sq.text_off + qt * 128 + (u & 1) * 64, h);
                last_u[slot] = u;
            }
            if (bt_ld_shared(sm.abort_addr()) != 0u) bt_drain(sm, last_u, a.status);
        }
    } else if (warp == 17) {
        // =============================== MMA issuer =================================
        if (lane == 0) bt_mma_loop<2>(sm, tmem, U, a.status, 0, 1, 256u, false);
    } else {
        // =============================== key rows ===================================
        const int quarter = warp & 3, cc = warp >> 2;                    // lanes 32 quarter ..; columns 16 cc .. of each half tile
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const int key_raw = kt * 128 + quarter * 32 + lane;
        const int key = key_raw < n_keys ? key_raw : 0x7fffffff;        // rows past the stream never match
        const int key_first = kt * 128, key_last_pad = kt * 128 + 127;
        // per-query scalars of this warp's columns, double-buffered by iteration: [buf][lse, delta, bound][32];
        // entry x * 16 + j belongs to query column 64 x + 16 cc + j of the tile
        float* rows = reinterpret_cast<float*>(base_ptr + kOffRow) + warp * 2 * 3 * 32;
        const int my_col = 64 * (lane >> 4) + 16 * cc + (lane & 15);     // the column whose scalars this lane fetches
        float n_lse, n_dl;
        int n_bnd;
        auto fetch = [&](int it) {
            const int qt = seg0 + it / G, h = hk * G + it % G;
            const size_t r = (size_t)h * a.text_rows + sq.text_off + (size_t)qt * 128 + my_col;
            const int i = qt * 128 + my_col;
            n_lse = a.lse_t[r];
            n_dl = a.delta_t[r];
            const int far = max(0, i / a.k - a.C);
            n_bnd = (i >= sq.n_text) ? (summ ? 0 : 0x7fffffff) : (summ ? min(sq.n_summ, far * a.m) : far * a.k);
        };
        auto stash = [&](int it) {
            float* rb = rows + (it & 1) * 3 * 32;
            rb[lane] = n_lse;
            rb[32 + lane] = n_dl;
            reinterpret_cast<int*>(rb)[64 + lane] = n_bnd;
        };
        fetch(0);
        stash(0);
        __syncwarp();
        bool alive = true;
        for (int it = 0; it < iters && alive; ++it) {
            if (it + 1 < iters) fetch(it + 1);                            // lands while this iteration is worked on
            const float* rowf = rows + (it & 1) * 3 * 32;
            const int* rowi = reinterpret_cast<const int*>(rowf) + 64;
            const int qt = seg0 + it / G;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (!bt_wait_warp(sm.bar(BB_SFULL + x), it & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
                tc_fence_after();
                const uint32_t tX = tmem + lane_sel + x * 64 + cc * 16, tY = tX + 128u;
                const int i0 = qt * 128 + 64 * x + 16 * cc;               // first query of the chunk
                uint32_t xs[16], ys[16];
                tmem_ld16(tX, xs);
                tmem_ld16(tY, ys);
                // every pair of the chunk visible (rows past the streams drop out by themselves: zero K / V
                // rows are discarded below, padding queries have lse = +inf)?
                bool full;
                if (!summ) {
                    const int far_last = max(0, (i0 + 15) / a.k - a.C);
                    full = key_last_pad <= i0 && far_last * a.k <= key_first;
                } else {
                    const int far_first = max(0, i0 / a.k - a.C);
                    full = key_last_pad < far_first * a.m;
                }
                tc_wait_ld();
                uint32_t pp[8], dd[8];
                if (full) {
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        const float p0 = ex2_approx(fmaf(__uint_as_float(xs[j]), a.scale_log2, -rowf[x * 16 + j]));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(xs[j + 1]), a.scale_log2, -rowf[x * 16 + j + 1]));
                        pp[j >> 1] = pack_bf16x2(p0, p1);
                        dd[j >> 1] = pack_bf16x2(p0 * (__uint_as_float(ys[j]) - rowf[32 + x * 16 + j]),
                                                 p1 * (__uint_as_float(ys[j + 1]) - rowf[32 + x * 16 + j + 1]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        float pv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int slot = x * 16 + j + e;
                            const bool vis = summ ? (key < rowi[slot]) : (key <= i0 + j + e && key >= rowi[slot]);
                            const float t = fmaf(__uint_as_float(xs[j + e]), a.scale_log2, -rowf[slot]);
                            pv[e] = ex2_approx(vis ? t : -INFINITY);
                        }
                        pp[j >> 1] = pack_bf16x2(pv[0], pv[1]);
                        dd[j >> 1] = pack_bf16x2(pv[0] * (__uint_as_float(ys[j]) - rowf[32 + x * 16 + j]),
                                                 pv[1] * (__uint_as_float(ys[j + 1]) - rowf[32 + x * 16 + j + 1]));
                    }
                }
                // bf16 results over the first 8 columns of the chunk's own fp32 columns: no other warp reads those
                tmem_st8(tX, pp);
                tmem_st8(tY, dd);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    const int u2 = 2 * it + x + 2;                        // warp 0 vouches for the slot of u + 2
                    if (warp == 0 && u2 < U) bt_wait(sm.bar(BB_QFULL + (u2 & 3)), (u2 >> 2) & 1, sm.abort_addr(), a.status, kStatusWaitQFull);
                    mbar_arrive(sm.bar(BB_PFULL + x));
                }
            }
            if (it + 1 < iters) { stash(it + 1); __syncwarp(); }
        }
        if (alive) {
            if (bt_wait_warp(sm.bar(BB_OFULL), 0, sm.abort_addr(), a.status, kStatusWaitOFull, lane)) {
                tc_fence_after();
                // odd cc: scale * dK, even cc: dV; cc / 2 picks the 64-element half of the row
                // (tcgen05.ld is warp-collective: rows past the stream load, too)
                const bool is_dk = (cc & 1) != 0;
                const int d0 = (cc >> 1) * 64;
                const size_t arow = (size_t)hk * (summ ? a.summ_rows : a.text_rows) + (size_t)krow0 + quarter * 32 + lane;
                float* acc = (is_dk ? (summ ? a.dks : a.dkt) : (summ ? a.dvs : a.dvt)) + arow * 128 + d0;
                const float mul = is_dk ? a.scale : 1.f;
                const uint32_t tacc = tmem + lane_sel + (is_dk ? 384u : 256u) + d0;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
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
    if (warp == 16) tmem_dealloc(tmem, 512);
}

__global__ void __maxnreg__(kBwdTcRegs)
ksa_bwd_dq_tc_kernel(const __grid_constant__ BwdArgs a, const __grid_constant__ BwdMaps maps)
{
    extern __shared__ uint8_t bsm_raw[];
    BtSmem sm;
    sm.base = (smem_u32(bsm_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- which queries, which keys (Eq. 3) ------------------------------------------------------
    const int h = blockIdx.y, hk = h / (a.Hq / a.Hkv);
    const SeqInfo sq = a.seqs[blockIdx.z];
    const int n_qt = (sq.n_text + 127) / 128;
    if ((int)blockIdx.x >= n_qt) return;
    const int qt = n_qt - 1 - (int)blockIdx.x;                            // long rows first
    const int i_first = qt * 128, i_last = min(sq.n_text, i_first + 128) - 1;
    const int far_first = max(0, i_first / a.k - a.C), far_last = max(0, i_last / a.k - a.C);
    const int n_s = a.m > 0 ? (min(sq.n_summ, far_last * a.m) + 127) / 128 : 0;     // summary tiles seen by the last row
    const int t_lo = (int)(((long long)far_first * a.k) / 128);                      // first text tile seen by the first row
    const int U = 2 * (n_s + qt - t_lo + 1);
    // half iteration u: summary tile u/2 while u/2 < n_s, then text tile t_lo + u/2 - n_s; rows 64 (u & 1) .. of it
    auto half_of = [&](int u, bool& is_summ, int& key0) {
        const int j = u >> 1;
        is_summ = j < n_s;
        key0 = (is_summ ? j : t_lo + j - n_s) * 128 + (u & 1) * 64;
    };

    bt_init(sm, tid, warp);
    const uint32_t tmem = bt_ld_shared(sm.tmem_slot());

    if (warp == 16) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.kt64); prefetch_tensormap(&maps.vt64);
            bt_load_resident(sm, &maps.qt, &maps.dot, sq.text_off + qt * 128, h);
            int last_u[4] = {-1, -1, -1, -1};
            for (int u = 0; u < U; ++u) {
                const int slot = u & 3;
                if (u >= 4 && !bt_slot_free(sm, u, a.status)) break;
                bool is_summ; int key0;
                half_of(u, is_summ, key0);
                if (is_summ) bt_load_slot(sm, slot, &maps.ks64, &maps.vs64, sq.summ_off + key0, hk);
                else         bt_load_slot(sm, slot, &maps.kt64, &maps.vt64, sq.text_off + key0, hk);
                last_u[slot] = u;
            }
            if (bt_ld_shared(sm.abort_addr()) != 0u) bt_drain(sm, last_u, a.status);
        }
    } else if (warp == 17) {
        // =============================== MMA issuer =================================
#ifdef KSA_BWD_TRACE
        if (lane == 0) bt_mma_loop<1>(sm, tmem, U, a.status, 0, 1, 256u, false, blockIdx.x == 8 && blockIdx.y == 0 && blockIdx.z == 0);
#else
        if (lane == 0) bt_mma_loop<1>(sm, tmem, U, a.status, 0, 1, 256u, false);
#endif
    } else {
        // =============================== query rows =================================
        const int quarter = warp & 3, cc = warp >> 2;                    // lanes 32 quarter ..; columns 16 cc .. of each half tile
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const int i_w0 = i_first + quarter * 32, i = i_w0 + lane;         // this thread's query row
        const size_t r = (size_t)h * a.text_rows + sq.text_off + i;
        const float lse2 = a.lse_t[r], dl = a.delta_t[r];                 // +inf / 0 on padding rows: P = 0 there
        const int far_i = max(0, i / a.k - a.C);
        const int lo_i = far_i * a.k, cnt_i = min(sq.n_summ, far_i * a.m);
        const int far_w0 = max(0, i_w0 / a.k - a.C), far_w1 = max(0, (i_w0 + 31) / a.k - a.C);
        bool alive = true;
#ifdef KSA_BWD_TRACE
        const bool bt_on = blockIdx.x == 8 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0;
        const int bt_role = 1 + warp;
        uint32_t bt_n = 0;
#endif
        for (int u = 0; u < U; ++u) {
            const int x = u & 1;
            if (!bt_wait_warp(sm.bar(BB_SFULL + x), (u >> 1) & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
            KSA_BT(bt_role, 10);
            tc_fence_after();
            bool is_summ; int key0;
            half_of(u, is_summ, key0);
            const int kc0 = key0 + 16 * cc;                               // first key of this warp's chunk
            const uint32_t tX = tmem + lane_sel + x * 64 + cc * 16, tY = tX + 128u;
            // the warp's 32 x 16 block: all visible, none, or mixed (rows of zeros past a stream add nothing to dQ)
            bool full, none;
            if (is_summ) {
                full = kc0 + 15 < min(sq.n_summ, far_w0 * a.m);
                none = kc0 >= far_w1 * a.m;
            } else {
                full = kc0 + 15 <= i_w0 && far_w1 * a.k <= kc0;
                none = kc0 > i_w0 + 31 || kc0 + 15 < far_w0 * a.k;
            }
            uint32_t dd[8];
            if (none) {
#pragma unroll
                for (int j = 0; j < 8; ++j) dd[j] = 0u;
            } else {
                uint32_t xs[16], ys[16];
                tmem_ld16(tX, xs);
                tmem_ld16(tY, ys);
                tc_wait_ld();
                KSA_BT(bt_role, 11);
                if (full) {
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        const float p0 = ex2_approx(fmaf(__uint_as_float(xs[j]), a.scale_log2, -lse2));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(xs[j + 1]), a.scale_log2, -lse2));
                        dd[j >> 1] = pack_bf16x2(p0 * (__uint_as_float(ys[j]) - dl), p1 * (__uint_as_float(ys[j + 1]) - dl));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        float pv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int key = kc0 + j + e;
                            const bool vis = is_summ ? (key < cnt_i) : (key <= i && key >= lo_i);
                            const float t = fmaf(__uint_as_float(xs[j + e]), a.scale_log2, -lse2);
                            pv[e] = ex2_approx(vis ? t : -INFINITY);
                        }
                        dd[j >> 1] = pack_bf16x2(pv[0] * (__uint_as_float(ys[j]) - dl), pv[1] * (__uint_as_float(ys[j + 1]) - dl));
                    }
                }
            }
            KSA_BT(bt_role, 12);
            tmem_st8(tX, dd);                                             // dS as bf16 over the chunk's own first 8 columns
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                const int u2 = u + 2;                                     // warp 0 vouches for the slot of u + 2
                if (warp == 0 && u2 < U) bt_wait(sm.bar(BB_QFULL + (u2 & 3)), (u2 >> 2) & 1, sm.abort_addr(), a.status, kStatusWaitQFull);
                mbar_arrive(sm.bar(BB_PFULL + x));
            }
            KSA_BT(bt_role, 13);
        }
#ifdef KSA_BWD_TRACE
        if (bt_on) g_btrace_cnt[bt_role] = bt_n;
#endif
        if (alive) {
            if (bt_wait_warp(sm.bar(BB_OFULL), 0, sm.abort_addr(), a.status, kStatusWaitOFull, lane)) {
                tc_fence_after();
                // scale * dQ as bf16 to the row's augmented position (Eq. 1); warp group cc writes elements 32 cc ..
                const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * (a.k + a.m) + (i % a.k);
                uint16_t* dst = a.dq + aug * a.dq_st + (int64_t)h * a.dq_sh + cc * 32;
                uint32_t o0[32];
                tmem_ld32(tmem + lane_sel + 256u + cc * 32, o0);
                tc_wait_ld();
                if (i < sq.n_text) {
                    float o[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __uint_as_float(o0[e]) * a.scale;
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(o[e], o[e + 1]);
                        w.y = pack_bf16x2(o[e + 2], o[e + 3]);
                        w.z = pack_bf16x2(o[e + 4], o[e + 5]);
                        w.w = pack_bf16x2(o[e + 6], o[e + 7]);
                        *reinterpret_cast<uint4*>(dst + e) = w;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 16) tmem_dealloc(tmem, 512);
}

#ifdef KSA_BWD_TRACE
extern "C" __attribute__((visibility("default"))) int ksa_debug_read_bwd_trace(void* events, void* counts)
{
    cudaDeviceSynchronize();
    cudaError_t e = cudaMemcpyFromSymbol(events, g_btrace, sizeof(g_btrace));
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(counts, g_btrace_cnt, sizeof(g_btrace_cnt));
    return (int)e;
}
#endif

cudaError_t setup_bwd_tc()
{
    cudaError_t e = cudaFuncSetAttribute(ksa_bwd_dkv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdTcSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(ksa_bwd_dq_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdTcSmem);
}

cudaError_t launch_bwd_dq_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream)
{
    dim3 grid((unsigned)(a.max_text_pad / 128), (unsigned)a.Hq, (unsigned)a.num_seqs);
    ksa_bwd_dq_tc_kernel<<<grid, kBwdTcThreads, kBwdTcSmem, stream>>>(a, maps);
    return cudaGetLastError();
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
