// Backward pass of the text rows on the sm_100a tensor cores (head_dim D = 128 or 64): dK / dV and dQ.
//
// Both kernels keep two 128 x D operand tiles resident in shared memory (A1, A2) and stream the tiles
// of the other two operands (B1: three TMA-filled stages, B2: two) past them.  Per streamed tile j the
// tensor pipe computes two products into TMEM, X_j = A1 B1_j^T and Y_j = A2 B2_j^T (128 x 128, fp32),
// and the row warps turn them into bf16 operands for the accumulating MMAs in two phases:
//   phase A (after X_j)   P = exp2(X scale - lse) on the visible pairs, kept in registers
//   phase B (after Y_j)   dS = P (Y - delta), written as bf16 over the first half of Y's own columns
// TMEM (512 columns): X [0,128), Y [128,256), accumulators from 256.
//
//   dK / dV  key-stationary and transposed: A1 = K tile, A2 = V tile (text or summary stream), B1 = Q tile,
//            B2 = dO tile of the (query tile, query head) pairs that see the keys; X = S^T, Y = dP^T.
//            The warps hand X back as soon as it is in their registers, so X_{j+1} runs beside the
//            exponentials of tile j; phase B goes through each warp's 32-column block of Y in two halves of
//            16 queries and writes dS^T over the first 8 and P^T over the other 8 columns of the half just
//            read, with one arrival per half: the accumulations over the first halves (k-steps 0, 2, 4, 6)
//            run beside the arithmetic of the second.  Pipe order per j: X_{j+1}, dV += P^T dO_j and
//            dK += dS^T Q_j (even k-steps, then odd), Y_{j+1}.  At the end each key row adds dV and
//            scale * dK to the fp32 accumulators of its stream (vector atomics: several segments and the
//            summary-row kernel add to the same rows).
//   dQ       query-stationary: A1 = Q tile, A2 = dO tile, B1 = K tile, B2 = V tile over the visible
//            summary tiles, then the visible text tiles (Eq. 3); X = S, Y = dP.  One accumulator leaves
//            room for a second Y buffer (columns from 384), so both products of tile j + 1 are issued
//            as soon as the warps have read X_j, and the warps never wait for the pipe: order per j:
//            X_{j+1}, Y_{j+1}, dQ += dS K_j.  At the end scale * dQ goes to the caller's tensor as bf16.
//
// Warps 0-15: one accumulator row per thread, four warps per row quarter (warps w, w + 4, w + 8, w + 12
// share the lanes 32 (w % 4) ..; each takes 32 of the 128 columns: the element-wise work has no reduction
// across columns, and four warps per scheduler hide the TMEM load / store latencies); warp 16: TMA
// producer; warp 17: MMA issuer.  The issuer's time is the critical path, so it waits only for the row
// warps: row warp 0 checks that the next B1 / B2 stage has landed before it arrives.  The tensor pipe
// works in order, so the completion of a product also tells which stage the accumulation before it has
// finished with: in the dQ kernel row warp 0, which sees every completion of X and Y, passes that on to
// the producer through one "empty" barrier per stage (the issuer is spared the extra commits -- except
// for the K stages, which the early products would otherwise release too late); in the dK / dV kernel the
// issuer commits to the "empty" barriers right behind each accumulation.  (The producer itself may fall
// several completions behind, which a parity wait on a shared barrier cannot follow: hence one barrier
// per stage.)  Every mbarrier wait is bounded (status word + CTA-wide abort flag).
#include <cuda_bf16.h>

#include <algorithm>

#include "ksa_bwd.h"
#include "ksa_ptx.cuh"

namespace ksa {

using namespace ptx;

constexpr int kBwdTcThreads = 576;
constexpr int kBwdTcRegs = 96;                  // 18 warps: five on a scheduler, 5 x 32 x 96 registers fit its file
constexpr int kBwdSegPairs = 64;                // dK / dV: (query tile, query head) pairs per CTA, at least 16 query tiles
constexpr int kB1Stages = 3, kB2Stages = 2;

// shared memory map (bytes from the 1024-aligned base) for head_dim D
template <int D>
struct BtMap {
    static constexpr int kTile = 128 * D * 2;   // one 128 x D bf16 tile: [64-element half of d][128 rows][128 B]
    static constexpr int kOffA1 = 0, kOffA2 = kTile, kOffB1 = 2 * kTile, kOffB2 = kOffB1 + kB1Stages * kTile;
    static constexpr int kOffBars = kOffB2 + kB2Stages * kTile;                        // 18 barriers
    static constexpr int kOffMisc = kOffBars + 192;                                    // TMEM slot, abort flags
    static constexpr int kOffRow = kOffMisc + 64;                                      // dK / dV: [2][lse, delta][128] per-query scalars
    static constexpr int kLayoutBytes = kOffRow + 2 * 2 * 128 * 4;
    // head_dim 128: the whole opt-in window (the layout needs all but 768 bytes of it); 64: the layout and the slack
    // for its 1024-byte alignment
    static constexpr int kSmem = D == 128 ? 232448 : kLayoutBytes + 1024;
    static_assert(kLayoutBytes <= kSmem, "shared memory layout");
};
enum : int { BB_AFULL = 0, BB_B1FULL = 1, BB_B2FULL = 4, BB_XFULL = 6, BB_YFULL = 7, BB_PA = 8, BB_PB = 9, BB_OFULL = 10,
             BB_B1EMPTY = 11, BB_B2EMPTY = 14, BB_YFULL2 = 16, BB_PB2 = 17 };

// Optional event trace (compile with -DKSA_BWD_TRACE=1 for the dQ kernel, =3 for the dK / dV kernel over summary
// keys): one CTA records (event id, clock) pairs for lane 0 of every row warp; ksa_debug_read_bwd_trace() copies
// them out.  =2 / =4: no stamps, only the MMA issuer's waiting times (below).
#ifdef KSA_BWD_TRACE
constexpr int kBtEvents = 4096;
__device__ uint2 g_btrace[17][kBtEvents];         // role 0: MMA issuer (sums only); 1 + w: row warp w
__device__ uint32_t g_btrace_cnt[17];
#define KSA_BT(role, id)                                                                         \
    do {                                                                                         \
        if (bt_on && bt_n < (uint32_t)kBtEvents) g_btrace[role][bt_n++] = make_uint2((uint32_t)(id), (uint32_t)clock()); \
    } while (0)
#else
#define KSA_BT(role, id) do { } while (0)
#endif
// KSA_BWD_TRACE == 2 / 4: the MMA issuer of one CTA of the dQ / the dK/dV (summary keys) kernel sums the cycles it
// spends waiting for the row warps (registers only, written once at the end: stamps in memory disturb the waits).
#if defined(KSA_BWD_TRACE) && (KSA_BWD_TRACE == 2 || KSA_BWD_TRACE == 4)
#define KSA_BT_WAIT_BEGIN() const uint32_t bt_w0 = (uint32_t)clock()
#define KSA_BT_WAIT_END(acc) acc += (uint32_t)clock() - bt_w0
#else
#define KSA_BT_WAIT_BEGIN() do { } while (0)
#define KSA_BT_WAIT_END(acc) do { } while (0)
#endif

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
// One lane polls for the warp (hundreds of polling threads would crowd the barrier unit).
__device__ __forceinline__ bool bt_wait_warp(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status, int code, int lane)
{
    bool ok = true;
    if (lane == 0) ok = bt_wait(bar, parity, abort_addr, status, code);
    return __shfl_sync(0xffffffffu, ok, 0);
}

// Shared-memory layout and barrier addresses of one CTA.
template <int D>
struct BtSmem {
    using M = BtMap<D>;
    uint32_t base;
    __device__ __forceinline__ uint32_t a1() const { return base + M::kOffA1; }
    __device__ __forceinline__ uint32_t a2() const { return base + M::kOffA2; }
    __device__ __forceinline__ uint32_t b1(int stage) const { return base + M::kOffB1 + (uint32_t)stage * M::kTile; }
    __device__ __forceinline__ uint32_t b2(int stage) const { return base + M::kOffB2 + (uint32_t)stage * M::kTile; }
    __device__ __forceinline__ uint32_t bar(int i) const { return base + M::kOffBars + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t tmem_slot() const { return base + M::kOffMisc; }
    __device__ __forceinline__ uint32_t abort_addr() const { return base + M::kOffMisc + 4; }
};

// The layout starts on the first 1024-byte boundary of the dynamic window; false (and a status code) if it
// does not fit behind it.  Uniform over the CTA: everybody returns before any barrier is touched.
template <int D>
__device__ __forceinline__ bool bt_layout(BtSmem<D>& sm, const uint8_t* raw, int32_t* status)
{
    const uint32_t raw_addr = smem_u32(raw);
    sm.base = (raw_addr + 1023u) & ~1023u;
    if (sm.base - raw_addr + (uint32_t)BtMap<D>::kLayoutBytes > (uint32_t)BtMap<D>::kSmem) {
        if (threadIdx.x == 0) atomicCAS(status, 0, (int)kStatusSmemLayout);
        return false;
    }
    return true;
}

template <int D>
__device__ __forceinline__ void bt_init(const BtSmem<D>& sm, int tid, int warp)
{
    if (tid == 0) {
        mbar_init(sm.bar(BB_AFULL), 1);
        for (int s = 0; s < kB1Stages; ++s) { mbar_init(sm.bar(BB_B1FULL + s), 1); mbar_init(sm.bar(BB_B1EMPTY + s), 1); }
        for (int s = 0; s < kB2Stages; ++s) { mbar_init(sm.bar(BB_B2FULL + s), 1); mbar_init(sm.bar(BB_B2EMPTY + s), 1); }
        mbar_init(sm.bar(BB_XFULL), 1);
        mbar_init(sm.bar(BB_YFULL), 1);
        mbar_init(sm.bar(BB_YFULL2), 1);
        mbar_init(sm.bar(BB_PA), 16);
        mbar_init(sm.bar(BB_PB), 16);
        mbar_init(sm.bar(BB_PB2), 16);
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

// ---- MMA issue helpers (one thread) ---------------------------------------------------------------
// D[tmem_d] = A B^T, both 128 x D tiles K-major in shared memory ([64-element half of d][128 rows][128 B]).
template <int D>
__device__ __forceinline__ void bt_product(uint32_t tmem_d, uint32_t a_tile, uint32_t b_tile)
{
    constexpr uint32_t idesc = make_idesc_bf16(128, 128, false);
    const uint64_t ad = make_smem_desc_sw128(a_tile, 16, 1024), bd = make_smem_desc_sw128(b_tile, 16, 1024);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
        mma_ss(tmem_d, ad + off, bd + off, idesc, kk > 0 ? 1u : 0u);
    }
}
// D[tmem_d] (+)= A B: A = 128 x 128 bf16 in TMEM (16 packed columns at the start of every 32-column chunk of
// tmem_a), B = a 128 x D tile in shared memory read MN-major (64-element atoms of d 16384 bytes apart,
// 8-row groups 1024 bytes apart): D accumulator columns.
template <int D>
__device__ __forceinline__ void bt_accumulate(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_tile, bool first)
{
    constexpr uint32_t idesc = make_idesc_bf16(128, D, true);
    const uint64_t bd = make_smem_desc_sw128(b_tile, 16384, 1024);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk)
        mma_ts(tmem_d, tmem_a + (kk >> 1) * 32 + (kk & 1) * 8, bd + (uint32_t)((kk * 2048) >> 4), idesc, (!first || kk > 0) ? 1u : 0u);
}

// Half of such an accumulation for the dK / dV kernel, whose row warps hand their 32-column blocks over in two
// halves of 16 query columns: the four k-steps 2 c + odd, whose 16 x bf16 operand stands in the 8 columns at
// tmem_a + 32 c + 16 odd (tmem_a already points at dS^T, or 8 columns further at P^T).
template <int D>
__device__ __forceinline__ void bt_accumulate_half(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_tile, int odd, bool first)
{
    constexpr uint32_t idesc = make_idesc_bf16(128, D, true);
    const uint64_t bd = make_smem_desc_sw128(b_tile, 16384, 1024);
#pragma unroll
    for (int c = 0; c < 4; ++c)
        mma_ts(tmem_d, tmem_a + c * 32 + odd * 16, bd + (uint32_t)(((2 * c + odd) * 2048) >> 4), idesc, (!first || c > 0) ? 1u : 0u);
}

// ---- producer helpers (one thread) ----------------------------------------------------------------
// The two 64-column halves of a 128-row tile.  Packed streams: rows pos .. pos + 127 of a 3-D map.  Direct mode
// (no packed copies: every sequence a whole number of chunks): chunks pos .. of a 4-D view [D, rows per chunk,
// chunk, head] of the caller's interleaved tensor, whose box lands in shared memory as the same dense tile.
template <int D>
__device__ __forceinline__ void bt_issue_tile(uint32_t dst, uint32_t bar, const CUtensorMap* map, int pos, int head, bool direct)
{
    if (direct) {
        tma_load_4d(dst, map, bar, 0, 0, pos, head);
        if (D == 128) tma_load_4d(dst + 16384, map, bar, 64, 0, pos, head);
    } else {
        tma_load_3d(dst, map, bar, 0, pos, head);
        if (D == 128) tma_load_3d(dst + 16384, map, bar, 64, pos, head);
    }
}
template <int D>
__device__ __forceinline__ void bt_load_tile(uint32_t dst, uint32_t bar, const CUtensorMap* map, int pos, int head, bool direct)
{
    mbar_arrive_expect_tx(bar, (uint32_t)BtMap<D>::kTile);
    bt_issue_tile<D>(dst, bar, map, pos, head, direct);
}
// After an abort: leave no copy in flight.  Bounded waits (the second flag is never set) for the last fill of
// every stage; filled1 / filled2 = B1 / B2 tiles whose load was issued.
template <int D>
__device__ __forceinline__ void bt_drain(const BtSmem<D>& sm, int filled1, int filled2, int32_t* status)
{
    const uint32_t never = sm.abort_addr() + 4;
    bt_wait(sm.bar(BB_AFULL), 0, never, status, kStatusWaitKvFull);
    for (int s = 0; s < kB1Stages; ++s) {
        const int fills = (filled1 + kB1Stages - 1 - s) / kB1Stages;     // tiles j < filled1 with j % 3 == s
        if (fills > 0) bt_wait(sm.bar(BB_B1FULL + s), (uint32_t)((fills - 1) & 1), never, status, kStatusWaitQFull);
    }
    for (int s = 0; s < kB2Stages; ++s) {
        const int fills = (filled2 + kB2Stages - 1 - s) / kB2Stages;
        if (fills > 0) bt_wait(sm.bar(BB_B2FULL + s), (uint32_t)((fills - 1) & 1), never, status, kStatusWaitQFull);
    }
}

// Stage `stage` (of `stages`) is about to take tile j: wait until its previous tile (j - stages) was released.
template <int D>
__device__ __forceinline__ bool bt_stage_free(const BtSmem<D>& sm, int empty0, int stages, int j, int32_t* status)
{
    if (j < stages) return true;
    return bt_wait(sm.bar(empty0 + j % stages), (uint32_t)((j / stages - 1) & 1), sm.abort_addr(), status, kStatusWaitQEmpty);
}

// =====================================================================================================
// dK / dV
// =====================================================================================================
template <int D>
__global__ void __maxnreg__(kBwdTcRegs)
ksa_bwd_dkv_tc_kernel(const __grid_constant__ BwdArgs a, const __grid_constant__ BwdMaps maps, const int summ, const int seg_tiles, const int store)
{
    extern __shared__ uint8_t bsm_raw[];
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
    const int seg0 = qt_lo + (int)blockIdx.x * seg_tiles;
    if (seg0 > qt_hi) return;
    const int seg1 = min(qt_hi + 1, seg0 + seg_tiles);
    const int J = (seg1 - seg0) * G;                                      // streamed tiles: (query tile, query head) pairs
    const int krow0 = (summ ? sq.summ_off : sq.text_off) + kt * 128;      // first row of the key tile in its packed stream
    auto pair_of = [&](int j, int& qt, int& h) { qt = seg0 + j / G; h = hk * G + j % G; };

    BtSmem<D> sm;
    if (!bt_layout(sm, bsm_raw, a.status)) return;
    uint8_t* base_ptr = bsm_raw + (sm.base - smem_u32(bsm_raw));
    // per-query scalars of the streamed tile, double-buffered by j: [j & 1][lse, delta][128 columns]; every row
    // warp writes the 32 columns it reads itself, one tile ahead (the four warps of a column group write the same
    // values, and each relies on its own writes only), see below
    float* rows = reinterpret_cast<float*>(base_ptr + BtMap<D>::kOffRow);
    const int quarter = warp & 3, cg = warp >> 2;                        // row warps: lanes 32 quarter ..; columns 32 cg ..
    const bool scalar_writer = warp < 16 && quarter == 0;
    float n_lse = 0.f, n_dl = 0.f;                                        // the writer lane's values for the next tile
    auto fetch = [&](int qt, int g) {                                     // pair (query tile qt, head g of the group)
        const int h = hk * G + g;
        const size_t r = (size_t)h * a.text_rows + sq.text_off + (size_t)qt * 128 + 32 * cg + lane;
        n_lse = a.lse_t[r];                                               // +inf on padding rows: P = 0 there
        n_dl = a.delta_t[r];
    };
    if (scalar_writer) {                                                  // tile 0: visible to all after the first barrier
        fetch(seg0, 0);
        rows[32 * cg + lane] = n_lse;
        rows[128 + 32 * cg + lane] = n_dl;
    }
    bt_init(sm, tid, warp);
    const uint32_t tmem = bt_ld_shared(sm.tmem_slot());
    const uint32_t tX = tmem, tY = tmem + 128u, tDV = tmem + 256u, tDK = tmem + 384u;

    if (warp == 16) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.qt); prefetch_tensormap(&maps.dot);
            const bool direct = a.direct != 0;
            const int q_step = direct ? 128 / a.k : 128, q_base = direct ? sq.chunk0 : sq.text_off;   // position of a query tile
            mbar_arrive_expect_tx(sm.bar(BB_AFULL), 2u * BtMap<D>::kTile);
            {
                const int kpos = direct ? sq.chunk0 + kt * (128 / (summ ? a.m : a.k)) : krow0;
                bt_issue_tile<D>(sm.a1(), sm.bar(BB_AFULL), summ ? &maps.ks : &maps.kt, kpos, hk, direct);
                bt_issue_tile<D>(sm.a2(), sm.bar(BB_AFULL), summ ? &maps.vs : &maps.vt, kpos, hk, direct);
            }
            int filled1 = 0, filled2 = 0;
            bool ok = true;
            for (int j = 0; j < J && ok; ++j) {
                int qt, h;
                pair_of(j, qt, h);
                const int pos = q_base + qt * q_step;
                if (!(ok = bt_stage_free(sm, BB_B1EMPTY, kB1Stages, j, a.status))) break;
                bt_load_tile<D>(sm.b1(j % kB1Stages), sm.bar(BB_B1FULL + j % kB1Stages), &maps.qt, pos, h, direct);
                ++filled1;
                if (!(ok = bt_stage_free(sm, BB_B2EMPTY, kB2Stages, j, a.status))) break;
                bt_load_tile<D>(sm.b2(j & 1), sm.bar(BB_B2FULL + (j & 1)), &maps.dot, pos, h, direct);
                ++filled2;
            }
            if (bt_ld_shared(sm.abort_addr()) != 0u) bt_drain(sm, filled1, filled2, a.status);
        }
    } else if (warp == 17) {
        // =============================== MMA issuer =================================
        if (lane == 0) {
            const uint32_t abort_addr = sm.abort_addr();
            bool alive = bt_wait(sm.bar(BB_AFULL), 0, abort_addr, a.status, kStatusWaitKvFull);
            if (alive) alive = bt_wait(sm.bar(BB_B1FULL), 0, abort_addr, a.status, kStatusWaitQFull);
            if (alive) { bt_product<D>(tX, sm.a1(), sm.b1(0)); tc_commit(sm.bar(BB_XFULL)); }
            if (alive) alive = bt_wait(sm.bar(BB_B2FULL), 0, abort_addr, a.status, kStatusWaitQFull);
            if (alive) { bt_product<D>(tY, sm.a2(), sm.b2(0)); tc_commit(sm.bar(BB_YFULL)); }
            uint32_t bt_wait_a = 0, bt_wait_b = 0, bt_wait_c = 0, bt_iss_x = 0, bt_iss_acc = 0;
            const uint32_t bt_loop0 = (uint32_t)clock();
            (void)bt_wait_a; (void)bt_wait_b; (void)bt_loop0; (void)bt_wait_c; (void)bt_iss_x; (void)bt_iss_acc;
            for (int j = 0; j < J && alive; ++j) {
                // the warps hold X_j in registers: the next S^T product may overwrite it while they exponentiate
                { KSA_BT_WAIT_BEGIN();
                  if (!bt_wait(sm.bar(BB_PA), j & 1, abort_addr, a.status, kStatusWaitPFull)) break;
                  KSA_BT_WAIT_END(bt_wait_a); }
                tc_fence_after();
                if (j + 1 < J) {
                    const int s1 = (j + 1) % kB1Stages;
                    { KSA_BT_WAIT_BEGIN();
                    if (!bt_wait(sm.bar(BB_B1FULL + s1), ((j + 1) / kB1Stages) & 1, abort_addr, a.status, kStatusWaitQFull)) break;
                    KSA_BT_WAIT_END(bt_wait_c); }
                    { KSA_BT_WAIT_BEGIN();
                    bt_product<D>(tX, sm.a1(), sm.b1(s1));
                    tc_commit(sm.bar(BB_XFULL));
                    KSA_BT_WAIT_END(bt_iss_x); }
                }
                // dS^T and P^T of the first 16 queries of every block stand in Y's columns: the even k-steps
                { KSA_BT_WAIT_BEGIN();
                  if (!bt_wait(sm.bar(BB_PB), j & 1, abort_addr, a.status, kStatusWaitPFull)) break;
                  KSA_BT_WAIT_END(bt_wait_b); }
                tc_fence_after();
                KSA_BT_WAIT_BEGIN();
                bt_accumulate_half<D>(tDV, tY + 8, sm.b2(j & 1), 0, j == 0);                   // dV += P^T dO_j
                bt_accumulate_half<D>(tDK, tY, sm.b1(j % kB1Stages), 0, j == 0);               // dK += dS^T Q_j
                // ... the other 16 (row warp 0 checked the stage of Y_{j+1} before it arrived): the odd k-steps
                if (!bt_wait(sm.bar(BB_PB2), j & 1, abort_addr, a.status, kStatusWaitPFull)) break;
                tc_fence_after();
                bt_accumulate_half<D>(tDV, tY + 8, sm.b2(j & 1), 1, false);
                tc_commit(sm.bar(BB_B2EMPTY + (j & 1)));                                    // ... then its dO stage is free
                bt_accumulate_half<D>(tDK, tY, sm.b1(j % kB1Stages), 1, false);
                tc_commit(sm.bar(BB_B1EMPTY + j % kB1Stages));                              // ... then its Q stage is free
                if (j + 1 < J) { bt_product<D>(tY, sm.a2(), sm.b2((j + 1) & 1)); tc_commit(sm.bar(BB_YFULL)); }
                KSA_BT_WAIT_END(bt_iss_acc);
            }
            tc_commit(sm.bar(BB_OFULL));
#if defined(KSA_BWD_TRACE) && KSA_BWD_TRACE == 4
            if (summ && blockIdx.x == 1 && blockIdx.y == 4 && blockIdx.z == 0) {
                g_btrace[0][0] = make_uint2(bt_wait_a, bt_wait_b);
                g_btrace[0][1] = make_uint2((uint32_t)clock() - bt_loop0, (uint32_t)J);
                g_btrace[0][2] = make_uint2(bt_wait_c, bt_iss_x);
                g_btrace[0][3] = make_uint2(bt_iss_acc, 0u);
                g_btrace_cnt[0] = 4;
            }
#endif
        }
    } else {
        // =============================== key rows ===================================
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t tXc = tX + lane_sel + cg * 32, tYc = tY + lane_sel + cg * 32;    // this warp's 32 x 32 block
        const int key_raw = kt * 128 + quarter * 32 + lane;
        const int key = key_raw < n_keys ? key_raw : 0x3fffffff;        // rows past the stream: never visible
        const int kq = key / (summ ? a.m : a.k);                          // the key's chunk
        const int kq_first = (kt * 128) / (summ ? a.m : a.k), kq_last = (kt * 128 + 127) / (summ ? a.m : a.k);
        bool alive = true;
        // The streamed tiles walk the pairs (query tile, head of the group) in order; the chunk of the block's first
        // query, i0 = 128 qt + 32 cg, is kept as quotient and remainder by k and advanced by 128 per query tile
        // (integer divisions are slow, and this loop is the warps' critical path).
        const int step_q = 128 / a.k, step_r = 128 - step_q * a.k, q31 = 31 / a.k, r31 = 31 - q31 * a.k;
#ifdef KSA_BWD_TRACE
        const bool bt_on = KSA_BWD_TRACE == 3 && summ && blockIdx.x == 1 && blockIdx.y == 4 && blockIdx.z == 0 && lane == 0;
        const int bt_role = 1 + warp;
        uint32_t bt_n = 0;
#endif
        int qt = seg0, g = 0;
        int iq0 = (seg0 * 128 + 32 * cg) / a.k, ir0 = (seg0 * 128 + 32 * cg) - iq0 * a.k;
        for (int j = 0; j < J && alive; ++j) {
            if (j + 1 < J) fetch(g + 1 == G ? qt + 1 : qt, g + 1 == G ? 0 : g + 1);   // lands while this tile is worked on
            const float* lse_c = rows + (j & 1) * 256 + 32 * cg;          // this warp's 32 columns
            const float* dl_c = lse_c + 128;
            const int i0 = qt * 128 + 32 * cg;                            // first query of the block
            const int iq1 = iq0 + q31 + (ir0 + r31 >= a.k ? 1 : 0);       // chunk of the block's last query
            // ---------------- phase A: P^T = exp2(S^T scale - lse), kept in registers ----------------
            if (!bt_wait_warp(sm.bar(BB_XFULL), j & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
            KSA_BT(bt_role, 10);
            tc_fence_after();
            // all pairs of the block visible / none (rows past the streams drop out by themselves: zero K / V
            // rows are discarded at the end, padding queries have lse = +inf)
            bool full, none;
            if (!summ) {
                full = kt * 128 + 127 <= i0 && iq1 - kq_first <= a.C;
                none = kt * 128 > i0 + 31 || iq0 - kq_last > a.C;
            } else {
                full = iq0 - kq_last > a.C;
                none = iq1 - kq_first <= a.C;
            }
            uint32_t x0[16], x1[16];                                      // S^T, then P^T in place (fp32 bits), kept for phase B
            if (none) {
#pragma unroll
                for (int c = 0; c < 16; ++c) x0[c] = x1[c] = 0u;
            } else {
                tmem_ld16(tXc, x0);
                tmem_ld16(tXc + 16, x1);
                tc_wait_ld();
            }
            // X_j is in registers: the issuer may start X_{j+1} while the exponentials run
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.bar(BB_PA));
            KSA_BT(bt_role, 11);
            if (!none) {
                if (full) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        x0[c] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(x0[c]), a.scale_log2, -lse_c[c])));
                        x1[c] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(x1[c]), a.scale_log2, -lse_c[16 + c])));
                    }
                } else {
                    int iq = iq0, ir = ir0;                               // chunk of query i0 + c, counted up from i0's
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        uint32_t& xc = c < 16 ? x0[c & 15] : x1[c & 15];
                        const bool vis = summ ? (iq - kq > a.C) : (key <= i0 + c && iq - kq <= a.C);
                        const float t = fmaf(__uint_as_float(xc), a.scale_log2, -lse_c[c]);
                        xc = __float_as_uint(ex2_approx(vis ? t : -INFINITY));
                        if (++ir == a.k) { ir = 0; ++iq; }
                    }
                }
            }
            KSA_BT(bt_role, 12);
            // ---------------- phase B: dS^T = P^T (dP^T - delta); both as bf16 over Y's own columns ----------------
            if (!bt_wait_warp(sm.bar(BB_YFULL), j & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
            KSA_BT(bt_role, 13);
            tc_fence_after();
            // Y_j was issued after every warp's arrival for tile j - 1: that tile's scalars may be overwritten
            if (j + 1 < J) {
                rows[((j + 1) & 1) * 256 + 32 * cg + lane] = n_lse;
                rows[((j + 1) & 1) * 256 + 128 + 32 * cg + lane] = n_dl;
            }
            // handed over in two halves of 16 queries, so that the accumulations of the first run beside the
            // arithmetic of the second: columns 16 half + 0 .. 7 take dS^T, 16 half + 8 .. 15 take P^T
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t o[16];
                if (none) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) o[c] = 0u;
                } else {
                    uint32_t ys[16];
                    tmem_ld16(tYc + half * 16, ys);
                    tc_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; c += 2) {
                        const float p0 = __uint_as_float(half ? x1[c] : x0[c]), p1 = __uint_as_float(half ? x1[c + 1] : x0[c + 1]);
                        o[c >> 1] = pack_bf16x2(p0 * (__uint_as_float(ys[c]) - dl_c[half * 16 + c]),
                                                p1 * (__uint_as_float(ys[c + 1]) - dl_c[half * 16 + c + 1]));
                        o[8 + (c >> 1)] = pack_bf16x2(p0, p1);
                    }
                }
                tmem_st16(tYc + half * 16, o);                            // over the 16 columns of dP^T just read
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (half == 1 && warp == 0 && j + 1 < J)               // warp 0 vouches for the stage of Y_{j+1}
                        bt_wait(sm.bar(BB_B2FULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, sm.abort_addr(), a.status, kStatusWaitQFull);
                    mbar_arrive(sm.bar(half ? BB_PB2 : BB_PB));
                }
            }
            KSA_BT(bt_role, 14);
            if (++g == G) {                                               // next query tile
                g = 0; ++qt;
                iq0 += step_q; ir0 += step_r;
                if (ir0 >= a.k) { ir0 -= a.k; ++iq0; }
            }
        }
#ifdef KSA_BWD_TRACE
        if (bt_on) g_btrace_cnt[bt_role] = bt_n;
#endif
        if (alive && bt_wait_warp(sm.bar(BB_OFULL), 0, sm.abort_addr(), a.status, kStatusWaitOFull, lane)) {
            tc_fence_after();
            // odd cg: scale * dK, even cg: dV; cg / 2 picks the half of the row (D / 2 elements)
            // (tcgen05.ld is warp-collective: rows past the stream load, too)
            const bool is_dk = (cg & 1) != 0;
            const int d0 = (cg >> 1) * (D / 2);
            const size_t arow = (size_t)hk * (summ ? a.summ_rows : a.text_rows) + (size_t)krow0 + quarter * 32 + lane;
            float* acc = (is_dk ? (summ ? a.dks : a.dkt) : (summ ? a.dvs : a.dvt)) + arow * D + d0;
            const float mul = is_dk ? a.scale : 1.f;
            const uint32_t tacc = (is_dk ? tDK : tDV) + lane_sel + d0;
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                uint32_t o[32];
                tmem_ld32(tacc + c * 32, o);
                tc_wait_ld();
                if (key_raw < n_keys) {
                    // store: this CTA is the only one of its launch for these keys and the first writer of their rows
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float4 val = make_float4(__uint_as_float(o[e]) * mul, __uint_as_float(o[e + 1]) * mul,
                                                       __uint_as_float(o[e + 2]) * mul, __uint_as_float(o[e + 3]) * mul);
                        if (store) *reinterpret_cast<float4*>(acc + c * 32 + e) = val;
                        else atomicAdd(reinterpret_cast<float4*>(acc + c * 32 + e), val);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 16) tmem_dealloc(tmem, 512);
}

// =====================================================================================================
// dQ
// =====================================================================================================
template <int D>
__global__ void __maxnreg__(kBwdTcRegs)
ksa_bwd_dq_tc_kernel(const __grid_constant__ BwdArgs a, const __grid_constant__ BwdMaps maps)
{
    extern __shared__ uint8_t bsm_raw[];
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
    const int J = n_s + qt - t_lo + 1;
    // streamed tile j: summary tile j while j < n_s, then text tile t_lo + j - n_s
    auto tile_of = [&](int j, bool& is_summ, int& key0) {
        is_summ = j < n_s;
        key0 = (is_summ ? j : t_lo + j - n_s) * 128;
    };

    BtSmem<D> sm;
    if (!bt_layout(sm, bsm_raw, a.status)) return;
    bt_init(sm, tid, warp);
    const uint32_t tmem = bt_ld_shared(sm.tmem_slot());
    const uint32_t tX = tmem, tDQ = tmem + 256u;
    auto tY = [&](int j) -> uint32_t { return tmem + ((j & 1) ? 384u : 128u); };   // dP of tile j, then dS in place
    auto y_full = [&](int j) -> uint32_t { return sm.bar((j & 1) ? BB_YFULL2 : BB_YFULL); };
    // likewise one phase B barrier per Y buffer: with both products of tile j + 1 issued early, a warp may finish
    // tile j + 1 before another has finished tile j, and must not arrive in its phase
    auto p_b = [&](int j) -> uint32_t { return sm.bar((j & 1) ? BB_PB2 : BB_PB); };

    if (warp == 16) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.kt); prefetch_tensormap(&maps.vt);
            const bool direct = a.direct != 0;
            mbar_arrive_expect_tx(sm.bar(BB_AFULL), 2u * BtMap<D>::kTile);
            {
                const int qpos = direct ? sq.chunk0 + qt * (128 / a.k) : sq.text_off + qt * 128;
                bt_issue_tile<D>(sm.a1(), sm.bar(BB_AFULL), &maps.qt, qpos, h, direct);
                bt_issue_tile<D>(sm.a2(), sm.bar(BB_AFULL), &maps.dot, qpos, h, direct);
            }
            int filled1 = 0, filled2 = 0;
            bool ok = true;
            for (int j = 0; j < J && ok; ++j) {
                bool is_summ; int key0;
                tile_of(j, is_summ, key0);
                // key0 / 128 tiles into its stream: rows of the packed stream, or chunks of the caller's tensor
                const int pos = direct ? sq.chunk0 + (key0 >> 7) * (128 / (is_summ ? a.m : a.k))
                                       : (is_summ ? sq.summ_off : sq.text_off) + key0;
                if (!(ok = bt_stage_free(sm, BB_B1EMPTY, kB1Stages, j, a.status))) break;
                bt_load_tile<D>(sm.b1(j % kB1Stages), sm.bar(BB_B1FULL + j % kB1Stages), is_summ ? &maps.ks : &maps.kt, pos, hk, direct);
                ++filled1;
                if (!(ok = bt_stage_free(sm, BB_B2EMPTY, kB2Stages, j, a.status))) break;
                bt_load_tile<D>(sm.b2(j & 1), sm.bar(BB_B2FULL + (j & 1)), is_summ ? &maps.vs : &maps.vt, pos, hk, direct);
                ++filled2;
            }
            if (bt_ld_shared(sm.abort_addr()) != 0u) bt_drain(sm, filled1, filled2, a.status);
        }
    } else if (warp == 17) {
        // =============================== MMA issuer =================================
        if (lane == 0) {
            const uint32_t abort_addr = sm.abort_addr();
            bool alive = bt_wait(sm.bar(BB_AFULL), 0, abort_addr, a.status, kStatusWaitKvFull);
            if (alive) alive = bt_wait(sm.bar(BB_B1FULL), 0, abort_addr, a.status, kStatusWaitQFull);
            if (alive) { bt_product<D>(tX, sm.a1(), sm.b1(0)); tc_commit(sm.bar(BB_XFULL)); }
            if (alive) alive = bt_wait(sm.bar(BB_B2FULL), 0, abort_addr, a.status, kStatusWaitQFull);
            if (alive) { bt_product<D>(tY(0), sm.a2(), sm.b2(0)); tc_commit(y_full(0)); }
            uint32_t bt_wait_a = 0, bt_wait_b = 0;
            const uint32_t bt_loop0 = (uint32_t)clock();
            (void)bt_wait_a; (void)bt_wait_b; (void)bt_loop0;
            for (int j = 0; j < J && alive; ++j) {
                // later stages were checked by row warp 0 before its arrival
                if (j + 1 < J) {
                    // phase A of tile j has read X into registers; the other Y buffer was read by dQ += dS K_{j-1}
                    KSA_BT_WAIT_BEGIN();
                    if (!bt_wait(sm.bar(BB_PA), j & 1, abort_addr, a.status, kStatusWaitPFull)) break;
                    KSA_BT_WAIT_END(bt_wait_a);
                    tc_fence_after();
                    bt_product<D>(tX, sm.a1(), sm.b1((j + 1) % kB1Stages));
                    tc_commit(sm.bar(BB_XFULL));
                    bt_product<D>(tY(j + 1), sm.a2(), sm.b2((j + 1) & 1));
                    tc_commit(y_full(j + 1));
                }
                { KSA_BT_WAIT_BEGIN();
                  if (!bt_wait(p_b(j), (j >> 1) & 1, abort_addr, a.status, kStatusWaitPFull)) break;
                  KSA_BT_WAIT_END(bt_wait_b); }
                tc_fence_after();
                bt_accumulate<D>(tDQ, tY(j), sm.b1(j % kB1Stages), j == 0);                    // dQ += dS K_j
                tc_commit(sm.bar(BB_B1EMPTY + j % kB1Stages));                              // K_j is free after that
            }
            tc_commit(sm.bar(BB_OFULL));
#if defined(KSA_BWD_TRACE) && KSA_BWD_TRACE == 2
            if (blockIdx.x == 8 && blockIdx.y == 0 && blockIdx.z == 0) {
                g_btrace[0][0] = make_uint2(bt_wait_a, bt_wait_b);
                g_btrace[0][1] = make_uint2((uint32_t)clock() - bt_loop0, (uint32_t)J);
                g_btrace_cnt[0] = 2;
            }
#endif
        }
    } else {
        // =============================== query rows =================================
        const int quarter = warp & 3, cg = warp >> 2;                    // lanes 32 quarter ..; columns 32 cg ..
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t tXc = tX + lane_sel + cg * 32;                     // this warp's 32 x 32 block
        const int i_w0 = i_first + quarter * 32, i = i_w0 + lane;         // this thread's query row
        const size_t r = (size_t)h * a.text_rows + sq.text_off + i;
        const float lse2 = a.lse_t[r], dl = a.delta_t[r];                 // +inf / 0 on padding rows: P = 0 there
        const int iq = i / a.k, iq_w0 = i_w0 / a.k, iq_w1 = (i_w0 + 31) / a.k;
#ifdef KSA_BWD_TRACE
        const bool bt_on = KSA_BWD_TRACE == 1 && blockIdx.x == 8 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0;
        const int bt_role = 1 + warp;
        uint32_t bt_n = 0;
#endif
        bool alive = true;
        // The chunk of the block's first key, kc0 = key0 + 32 cg, is kept as quotient and remainder by the keys per
        // chunk of its stream and advanced by 128 per tile; divisions only where the stream starts (integer
        // divisions are slow, and this loop is the warps' critical path).
        int cdiv = 1, kq0 = 0, kr0 = 0, step_q = 0, step_r = 0, q31 = 0, r31 = 0;
        for (int j = 0; j < J; ++j) {
            bool is_summ; int key0;
            tile_of(j, is_summ, key0);
            const int kc0 = key0 + 32 * cg;                               // first key of this warp's block
            if (j == 0 || j == n_s) {                                     // first tile of the summary / the text stream
                cdiv = is_summ ? a.m : a.k;                               // keys per chunk in this stream
                kq0 = kc0 / cdiv; kr0 = kc0 - kq0 * cdiv;
                step_q = 128 / cdiv; step_r = 128 - step_q * cdiv;
                q31 = 31 / cdiv; r31 = 31 - q31 * cdiv;
            } else {
                kq0 += step_q; kr0 += step_r;
                if (kr0 >= cdiv) { kr0 -= cdiv; ++kq0; }
            }
            const int kq1 = kq0 + q31 + (kr0 + r31 >= cdiv ? 1 : 0);      // chunk of the block's last key
            // the warp's 32 x 32 block: all visible, none, or mixed (zero rows past a stream add nothing to dQ).
            // Text key t is visible to row i iff t <= i and chunk(i) - chunk(t) <= C; summary key s iff
            // chunk(i) - chunk(s) > C (Eq. 3)
            bool full, none;
            if (is_summ) {
                full = iq_w0 - kq1 > a.C;
                none = iq_w1 - kq0 <= a.C;
            } else {
                full = kc0 + 31 <= i_w0 && iq_w1 - kq0 <= a.C;
                none = kc0 > i_w0 + 31 || iq_w0 - kq1 > a.C;
            }
            // ---------------- phase A: P = exp2(S scale - lse) ----------------
            if (!bt_wait_warp(sm.bar(BB_XFULL), j & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
            KSA_BT(bt_role, 10);
            tc_fence_after();
            uint32_t x0[16], x1[16];                                      // S, then P in place (fp32 bits)
            if (!none) {
                tmem_ld16(tXc, x0);
                tmem_ld16(tXc + 16, x1);
                tc_wait_ld();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {                                              // X may be overwritten from here on
                if (warp == 0 && j + 1 < J) {                              // warp 0 vouches for the stages of X_{j+1} and Y_{j+1}
                    bt_wait(sm.bar(BB_B1FULL + (j + 1) % kB1Stages), ((j + 1) / kB1Stages) & 1, sm.abort_addr(), a.status, kStatusWaitQFull);
                    bt_wait(sm.bar(BB_B2FULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, sm.abort_addr(), a.status, kStatusWaitQFull);
                }
                mbar_arrive(sm.bar(BB_PA));
            }
            KSA_BT(bt_role, 11);
            if (!none) {
                if (full) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        x0[c] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(x0[c]), a.scale_log2, -lse2)));
                        x1[c] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(x1[c]), a.scale_log2, -lse2)));
                    }
                } else {
                    int kq = kq0, kr = kr0;                               // chunk of key kc0 + c, counted up from kc0's
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        uint32_t& xc = c < 16 ? x0[c & 15] : x1[c & 15];
                        const bool vis = is_summ ? (iq - kq > a.C) : (kc0 + c <= i && iq - kq <= a.C);
                        const float t = fmaf(__uint_as_float(xc), a.scale_log2, -lse2);
                        xc = __float_as_uint(ex2_approx(vis ? t : -INFINITY));
                        if (++kr == cdiv) { kr = 0; ++kq; }
                    }
                }
            }
            KSA_BT(bt_role, 12);
            // ---------------- phase B: dS = P (dP - delta) ----------------
            // one barrier per Y buffer: Y_{j+1} may be complete before a warp gets here for Y_j
            if (!bt_wait_warp(y_full(j), (j >> 1) & 1, sm.abort_addr(), a.status, kStatusWaitSFull, lane)) { alive = false; break; }
            KSA_BT(bt_role, 13);
            tc_fence_after();
            if (warp == 0 && lane == 0) mbar_arrive(sm.bar(BB_B2EMPTY + (j & 1)));          // Y_j is complete: its V stage is free
            const uint32_t tYc = tY(j) + lane_sel + cg * 32;
            uint32_t dd[16];
            if (none) {
#pragma unroll
                for (int c = 0; c < 16; ++c) dd[c] = 0u;
            } else {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t ys[16];
                    tmem_ld16(tYc + half * 16, ys);
                    tc_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; c += 2) {
                        const float p0 = __uint_as_float(half ? x1[c] : x0[c]), p1 = __uint_as_float(half ? x1[c + 1] : x0[c + 1]);
                        dd[half * 8 + (c >> 1)] = pack_bf16x2(p0 * (__uint_as_float(ys[c]) - dl), p1 * (__uint_as_float(ys[c + 1]) - dl));
                    }
                }
            }
            tmem_st16(tYc, dd);                                           // over the block's own first 16 columns
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_b(j));
            KSA_BT(bt_role, 14);
        }
#ifdef KSA_BWD_TRACE
        if (bt_on) g_btrace_cnt[bt_role] = bt_n;
#endif
        if (alive && bt_wait_warp(sm.bar(BB_OFULL), 0, sm.abort_addr(), a.status, kStatusWaitOFull, lane)) {
            tc_fence_after();
            // scale * dQ as bf16 to the row's augmented position (Eq. 1); warp group cg writes elements 32 cg ..
            const int64_t aug = sq.aug_off + (int64_t)iq * (a.k + a.m) + (i - iq * a.k);
            uint16_t* dst = a.dq + aug * a.dq_st + (int64_t)h * a.dq_sh + cg * 32;
            uint32_t o[32];
            if (cg * 32 < D) {                                            // warp-uniform: the row has D elements
                tmem_ld32(tDQ + lane_sel + cg * 32, o);
                tc_wait_ld();
            }
            if (cg * 32 < D && i < sq.n_text) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(o[e]) * a.scale, __uint_as_float(o[e + 1]) * a.scale);
                    w.y = pack_bf16x2(__uint_as_float(o[e + 2]) * a.scale, __uint_as_float(o[e + 3]) * a.scale);
                    w.z = pack_bf16x2(__uint_as_float(o[e + 4]) * a.scale, __uint_as_float(o[e + 5]) * a.scale);
                    w.w = pack_bf16x2(__uint_as_float(o[e + 6]) * a.scale, __uint_as_float(o[e + 7]) * a.scale);
                    *reinterpret_cast<uint4*>(dst + e) = w;
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
    cudaError_t e = cudaFuncSetAttribute(ksa_bwd_dkv_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BtMap<128>::kSmem);
    if (e != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(ksa_bwd_dq_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BtMap<128>::kSmem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(ksa_bwd_dkv_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BtMap<64>::kSmem)) != cudaSuccess) return e;
    return cudaFuncSetAttribute(ksa_bwd_dq_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BtMap<64>::kSmem);
}

cudaError_t launch_bwd_dq_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream)
{
    dim3 grid((unsigned)(a.max_text_pad / 128), (unsigned)a.Hq, (unsigned)a.num_seqs);
    if (a.D == 128) ksa_bwd_dq_tc_kernel<128><<<grid, kBwdTcThreads, BtMap<128>::kSmem, stream>>>(a, maps);
    else            ksa_bwd_dq_tc_kernel<64><<<grid, kBwdTcThreads, BtMap<64>::kSmem, stream>>>(a, maps);
    return cudaGetLastError();
}

// Query tiles that see a text key tile (an upper bound), and the query tiles a CTA of the dK / dV kernel walks.
static long long bwd_text_span(const BwdArgs& a)
{
    return std::min<long long>(a.max_text_pad / 128, ((long long)a.C + 1) * a.k / 128 + 2);
}
static int bwd_seg_tiles(const BwdArgs& a) { return std::max(16, kBwdSegPairs / (a.Hq / a.Hkv)); }

// True if one CTA covers every query tile that sees a text key tile: then the text-key launch writes its rows of the
// accumulators with plain stores -- it must be their first writer (no clear needed; the summary rows' kernel adds later).
bool bwd_text_keys_stored(const BwdArgs& a) { return bwd_text_span(a) <= bwd_seg_tiles(a); }

cudaError_t launch_bwd_dkv_tc(const BwdArgs& a, const BwdMaps& maps, cudaStream_t stream)
{
    const int n_qt = a.max_text_pad / 128;
    const long long text_span = bwd_text_span(a);
    for (int summ = 0; summ < 2; ++summ) {
        if (summ && (a.m <= 0 || a.max_n_summ <= 0)) continue;
        const long long span = summ ? n_qt : text_span;
        const int tiles = summ ? (a.max_n_summ + 127) / 128 : n_qt;
        // a CTA walks seg query tiles x G heads: 16 tiles with four or more heads per KV head, more with fewer (the
        // start-up and the final atomics of a CTA are spread over about 64 streamed tiles either way)
        const int seg = bwd_seg_tiles(a);
        const int store = (!summ && bwd_text_keys_stored(a)) ? 1 : 0;
        dim3 grid((unsigned)((span + seg - 1) / seg), (unsigned)tiles, (unsigned)(a.num_seqs * a.Hkv));
        if (a.D == 128) ksa_bwd_dkv_tc_kernel<128><<<grid, kBwdTcThreads, BtMap<128>::kSmem, stream>>>(a, maps, summ, seg, store);
        else            ksa_bwd_dkv_tc_kernel<64><<<grid, kBwdTcThreads, BtMap<64>::kSmem, stream>>>(a, maps, summ, seg, store);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace ksa
