// Text-row KSA attention on CTA pairs (tcgen05 cta_group::2), head_dim 128, work items of two query heads.
//
// A cluster of two CTAs (two SMs) takes one work item at a time: 128 text query rows for the two query
// heads of one KV head, and the key/value tiles Eq. 3 makes visible to them.  CTA r of the pair owns query
// head head0 + r: its Q tile sits in its shared memory, its scores and its output accumulator in its TMEM.
// Every key/value tile is split between the two CTAs -- CTA r loads keys [64 r, 64 r + 64) of the K tile and
// head dimensions [64 r, 64 r + 64) of the V tile, each with its own plain TMA loads -- and threads of the
// pair's first CTA issue M = 256 MMAs that read both halves: S = Q K^T (both operands from shared memory)
// and O += P V (P from TMEM).  With one query tile per CTA the TMEM holds the scores and the probabilities
// in separate columns, so a score buffer is handed back as soon as its softmax warps hold it in registers:
// Q K^T of the next key tile never waits for a softmax to finish, only P V does.
//
// TMEM (512 columns per CTA): S0 [0,128), S1 [128,256), P0 [256,320), P1 [320,384) (bf16 pairs), O [384,512).
// Key tile g of the pair's tile stream uses S and P buffer g mod 2 and softmax group g mod 2.
//
// Warp roles in each CTA (384 threads):
//   warps 0-3   softmax group 0, warps 4-7 softmax group 1: one query row per thread, alternate key tiles
//   warp  8     TMA producer: this CTA's Q tile (double buffered) and K halves (ring of 16 KB stages)
//   warp 10     TMA producer: this CTA's V halves (ring of 16 KB stages)
//   warp  9     first CTA: issues O += P V.        second CTA: forwards "my V half has landed" to the first
//   warp 11     first CTA: issues S = Q K^T.       second CTA: forwards "my Q tile / K half has landed"
// The two issuing threads are independent streams: tcgen05 operations of ONE thread execute in issue order,
// across the two nothing is assumed -- every hand-over between them goes through an mbarrier
// (Q K^T into a score buffer: after its previous contents were read; P V: after the probabilities were
// written; a probability buffer is rewritten after the product that read it has completed).
//
// Online softmax across the two groups.  The rows' reference maximum m (log2 units, moves only when a row
// outgrows it by 2^8, row by row) lives in shared memory: the group that takes tile g reads the value the other group
// published after tile g - 1, decides, publishes, and only then takes its exponentials, so the hand-over is
// off the critical path.  Each group keeps the row sum of its own tiles relative to the m it last saw; the
// epilogue adds the two.  When m moves, the deciding group rescales O in TMEM after the product of tile
// g - 1 has completed and before it releases P(g).
//
// The tile stream is continuous across work items: Q K^T of the next item's first tiles is issued while the
// last tiles of the current item are still in their softmax.
//
// Every mbarrier wait is bounded: on timeout the thread records which wait gave up in the status word and
// raises the abort flag of both CTAs; all roles leave their loops, the producers wait (bounded) for their
// copies in flight, the pair meets at a cluster barrier, TMEM is freed and the kernel returns.
#include <cuda_bf16.h>

#include "ksa_launch.h"
#include "ksa_ptx.cuh"

namespace ksa {

using namespace ptx;

namespace pairk {

constexpr int kThreads = 384;
constexpr int kRegsSoftmax = 216;
constexpr int kRegsOther = 72;
static_assert(8 * kRegsSoftmax + 4 * kRegsOther <= 12 * ((65536 / kThreads) / 8 * 8), "register hand-over exceeds the CTA's allocation");
constexpr int kQkWarp = 11, kPvWarp = 9, kKProdWarp = 8, kVProdWarp = 10;
#ifndef KSA_RESCALE_T
#define KSA_RESCALE_T 8.0f
#endif
constexpr float kRescaleThreshold = KSA_RESCALE_T;
constexpr int D = 128;
constexpr int kKStages = 5;                   // ring of K halves (64 keys x 128 dims, 16 KB each)
constexpr int kVStages = 4;                   // ring of V halves (128 keys x 64 dims, 16 KB each)
constexpr int kStageBytes = 16384;
constexpr int kQBytes = 32768;
constexpr uint32_t kColP = 256, kColO = 384;

enum : int {
    B_QFULL = 0,                  // [2] this CTA's Q tile has landed (second CTA; the first CTA's lands on B_QPAIR)
    B_QPAIR = 2,                  // [2] first CTA: both Q tiles have landed
    B_QEMPTY = 4,                 // [2] every Q K^T of the item that used the buffer has completed
    B_SFULL = 6,                  // [2] scores of a tile are in TMEM
    B_SFREE = 8,                  // [2] first CTA: the scores are in registers (4 warps x 2 CTAs)
    B_PFULL = 10,                 // [2] first CTA: probabilities written (4 warps x 2 CTAs)
    B_PVDONE = 12,                // [2] O += P V of a tile has completed
    B_OEMPTY = 14,                // first CTA: the epilogue has read O (8 warps x 2 CTAs)
    B_DRAIN = 15,                 // [2] one per issuing thread
    B_UNUSED = 17,                // [8]
    B_LBAR = 25,                  // [4] row sums exchanged (2 arrivals)
    B_KFULL = 29,                 // [kKStages] second CTA: its K half has landed
    B_KPAIR = B_KFULL + kKStages, // first CTA: both K halves have landed
    B_KEMPTY = B_KPAIR + kKStages,
    B_VFULL = B_KEMPTY + kKStages,
    B_VPAIR = B_VFULL + kVStages,
    B_VEMPTY = B_VPAIR + kVStages,
    B_COUNT = B_VEMPTY + kVStages
};
static_assert(B_COUNT <= 64, "barrier area");
constexpr int kQOff = 0;
constexpr int kKRingOff = 2 * kQBytes;
constexpr int kVRingOff = kKRingOff + kKStages * kStageBytes;
constexpr int kBarOff = kVRingOff + kVStages * kStageBytes;
constexpr int kMiscOff = kBarOff + 8 * 64;
constexpr int kMshOff = kMiscOff + 64;                   // {float m, uint32 tag}[2 tile parities][128]: published reference maximum
constexpr int kLshOff = kMshOff + 2048;                  // float[2 item parities][2 groups][128]: row sums
constexpr int kMs2Off = kLshOff + 2048;                  // same shape: the maximum each sum is relative to
constexpr int kSmemBytes = kMs2Off + 2048 + 1024;        // + slack for 1024-byte alignment
static_assert(kSmemBytes <= 232448, "shared memory window");

// Optional cycle accounting (compile with -DKSA_PAIR_TRACE): per role, the first CTA of pair 0 adds up the cycles
// it spends in each kind of wait (in registers) and writes the sums once at the end; ksa_debug_pair_trace() copies
// them out.  Compiled out by default.
#ifdef KSA_PAIR_TRACE
__device__ unsigned long long g_pair_trace[64];
#define KSA_PT_DECL uint32_t pt_acc_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}; long long pt_t0_ = 0; const long long pt_start_ = clock64()
#define KSA_PT_BEGIN() do { pt_t0_ = clock64(); } while (0)
#define KSA_PT_END(slot) do { pt_acc_[slot] += (uint32_t)(clock64() - pt_t0_); } while (0)
#define KSA_PT_COUNT(slot) do { pt_acc_[slot] += 1u; } while (0)
#define KSA_PT_FLUSH(base, on) do { if (on) { pt_acc_[7] = (uint32_t)(clock64() - pt_start_); \
    for (int i_ = 0; i_ < 12; ++i_) atomicAdd(&g_pair_trace[(base) + i_], (unsigned long long)pt_acc_[i_]); } } while (0)
#else
#define KSA_PT_DECL do { } while (0)
#define KSA_PT_BEGIN() do { } while (0)
#define KSA_PT_END(slot) do { } while (0)
#define KSA_PT_COUNT(slot) do { } while (0)
#define KSA_PT_FLUSH(base, on) do { } while (0)
#endif

struct Ctl {
    uint32_t abort_addr;        // this CTA's abort flag
    uint32_t abort_peer;        // the other CTA's abort flag (shared::cluster address)
    int32_t* status;
};

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ float lds_f32(uint32_t addr) { return __uint_as_float(lds_u32(addr)); }
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) { sts_u32(addr, __float_as_uint(v)); }

#ifndef KSA_WAIT_HINT_NS
#define KSA_WAIT_HINT_NS 100000
#endif
constexpr uint32_t kWaitHintNs = KSA_WAIT_HINT_NS;     // per try_wait; the abort flag is looked at between them

// Bounded wait.  Returns false if the wait gave up or the pair is aborting.
__device__ __forceinline__ bool bwait_slow(uint32_t bar, uint32_t parity, uint32_t abort_addr, uint32_t abort_peer, int32_t* status, int code)
{
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
#if defined(KSA_SLEEP_NS) && KSA_SLEEP_NS > 0
        if (mbar_test_wait(bar, parity)) return true;
        __nanosleep(KSA_SLEEP_NS);
#else
        if (mbar_try_wait_hint(bar, parity, kWaitHintNs)) return true;
#endif
        if ((it & 15u) == 0u) {
            if (lds_u32(abort_addr) != 0u) return false;
            if (clock64() - t0 > (1ll << 31)) {
                atomicCAS(status, 0, code);
                sts_u32(abort_addr, 1u);
                st_shared_cluster_u32(abort_peer, 1u);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool bwait(uint32_t bar, uint32_t parity, const Ctl& c, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (mbar_try_wait(bar, parity)) return true;
    return bwait_slow(bar, parity, c.abort_addr, c.abort_peer, c.status, code);
}
// One 8-byte shared-memory word {value, tag}: written and read whole.
__device__ __forceinline__ void sts_tagged(uint32_t addr, float v, uint32_t tag)
{
    asm volatile("st.volatile.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(__float_as_uint(v)), "r"(tag) : "memory");
}
// Reads the word until its tag is `tag` (bounded like every other wait).
__device__ __forceinline__ bool wait_tagged(uint32_t addr, uint32_t tag, float& v, const Ctl& c, int code)
{
    uint32_t a, b;
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(a), "=r"(b) : "r"(addr) : "memory");
        if (b == tag) { v = __uint_as_float(a); return true; }
#if !defined(KSA_TAG_SLEEP_NS) || KSA_TAG_SLEEP_NS > 0
#ifndef KSA_TAG_SLEEP_NS
#define KSA_TAG_SLEEP_NS 32
#endif
        __nanosleep(KSA_TAG_SLEEP_NS);        // a tight read loop only burns issue slots and power next to the working warps
#endif
        if (it == 0) t0 = clock64();
        if ((it & 63u) == 63u) {
            if (lds_u32(c.abort_addr) != 0u) return false;
            if (clock64() - t0 > (1ll << 31)) {
                atomicCAS(c.status, 0, code);
                sts_u32(c.abort_addr, 1u);
                st_shared_cluster_u32(c.abort_peer, 1u);
                return false;
            }
        }
    }
}
// Teardown form: ignores the abort flags (the copies it waits for are in flight whatever else happened).
__device__ __noinline__ bool bwait_teardown(uint32_t bar, uint32_t parity, int32_t* status, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u && clock64() - t0 > (1ll << 31)) { atomicCAS(status, 0, code); return false; }
    }
}

// Walks the tile stream of a CTA pair: its work items in snake order over the longest-first list
// (round r gives pair c item r * pairs + c, or r * pairs + pairs - 1 - c in odd rounds), tile by tile.
struct Walk {
    const WorkItem* work;
    int num_work, pairs, cid;
    int r;            // ordinal of the current item for this pair
    int j, T;         // tile within the item, tiles of the item
    int ns;           // summary tiles come first: tiles [0, ns)
    int band_lo;
    int seq, q_tile, head0;
    bool done;
    __device__ __forceinline__ int index_of(int rr) const { return rr * pairs + ((rr & 1) ? (pairs - 1 - cid) : cid); }
    __device__ __forceinline__ void load()
    {
        const int idx = index_of(r);
        done = idx >= num_work;
        j = 0;
        if (!done) {
            const WorkItem w = work[idx];
            ns = w.ns_tiles; band_lo = w.band_lo; T = w.ns_tiles + (w.band_hi - w.band_lo + 1);
            seq = w.seq; q_tile = w.q_tile; head0 = w.head0;
        }
    }
    __device__ __forceinline__ void init(const KernelArgs& a, int pairs_, int cid_)
    {
        work = a.work; num_work = a.num_work; pairs = pairs_; cid = cid_; r = 0;
        load();
    }
    __device__ __forceinline__ void advance() { if (++j == T) { ++r; load(); } }
};
// The same walk for roles that only count tiles.
struct WalkLite {
    const WorkItem* work;
    int num_work, pairs, cid, r, j, T;
    bool done;
    __device__ __forceinline__ void load()
    {
        const int idx = r * pairs + ((r & 1) ? (pairs - 1 - cid) : cid);
        done = idx >= num_work;
        j = 0;
        if (!done) { const WorkItem* w = work + idx; T = w->ns_tiles + (w->band_hi - w->band_lo + 1); }
    }
    __device__ __forceinline__ void init(const KernelArgs& a, int pairs_, int cid_)
    {
        work = a.work; num_work = a.num_work; pairs = pairs_; cid = cid_; r = 0;
        load();
    }
    __device__ __forceinline__ void advance() { if (++j == T) { ++r; load(); } }
};

// descriptor with a 32-bit low word (start address field) and a fixed high word
__device__ __forceinline__ uint64_t desc_from(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
ksa_text_pair_kernel(const __grid_constant__ KernelArgs a, const __grid_constant__ PairMaps maps)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offsets in both CTAs of the pair: the MMA descriptors and the multicast commits rely on it
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + kQOff;
    const uint32_t sK = smem_base + kKRingOff;
    const uint32_t sV = smem_base + kVRingOff;
    const uint32_t bars = smem_base + kBarOff;
    const uint32_t tmem_slot = smem_base + kMiscOff;
    const uint32_t abort_addr = tmem_slot + 4;
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const int pairs = (int)gridDim.x >> 1;
    const int cid = (int)blockIdx.x >> 1;
    Ctl ctl;
    ctl.abort_addr = abort_addr;
    ctl.abort_peer = mapa_shared(abort_addr, rank ^ 1u);
    ctl.status = a.status;
    auto lead = [&](uint32_t local_addr) -> uint32_t { return mapa_shared(local_addr, 0u); };   // the first CTA's copy

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(B_QFULL + b), 1); mbar_init(bar(B_QPAIR + b), 2); mbar_init(bar(B_QEMPTY + b), 1);
            mbar_init(bar(B_SFULL + b), 1); mbar_init(bar(B_SFREE + b), 8); mbar_init(bar(B_PFULL + b), 8);
            mbar_init(bar(B_PVDONE + b), 1); mbar_init(bar(B_DRAIN + b), 1);
        }
        mbar_init(bar(B_OEMPTY), 16);
        for (int i = 0; i < 4; ++i) mbar_init(bar(B_LBAR + i), 2);
        for (int s = 0; s < kKStages; ++s) { mbar_init(bar(B_KFULL + s), 1); mbar_init(bar(B_KPAIR + s), 2); mbar_init(bar(B_KEMPTY + s), 1); }
        for (int s = 0; s < kVStages; ++s) { mbar_init(bar(B_VFULL + s), 1); mbar_init(bar(B_VPAIR + s), 2); mbar_init(bar(B_VEMPTY + s), 1); }
        sts_u32(abort_addr, 0u);
        fence_mbar_init();
    }
    if (tid < 256) { sts_u32(smem_base + kMshOff + 8u * (uint32_t)tid, 0u); sts_u32(smem_base + kMshOff + 8u * (uint32_t)tid + 4u, 0u); }
    if (warp == kQkWarp) {                  // one warp of each CTA: all 512 columns of both (1 CTA per SM)
        tmem_alloc_pair(tmem_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    // the other CTA's barriers exist before anything here signals them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem = lds_u32(tmem_slot);

    if (warp >= 8) {
    setmaxnreg_dec<kRegsOther>();
    if (lane == 0) {
    if (warp == kKProdWarp) {
        // =============================== TMA producer: Q tiles and K halves ==============================
        // First CTA: the loads complete on the pair barriers directly.  Second CTA: on its own barriers; its
        // forwarding warps pass the news on.
        prefetch_tensormap(&maps.qt); prefetch_tensormap(&maps.kt); prefetch_tensormap(&maps.ks);
        Walk wk;
        wk.init(a, pairs, cid);
        const int G = a.Hq / a.Hkv;
        const int q_bar = rank == 0 ? B_QPAIR : B_QFULL, k_bar = rank == 0 ? B_KPAIR : B_KFULL;
        int stage = 0; uint32_t phase = 0;
        uint32_t armed = 0, armed_par = 0, q_armed = 0, q_par = 0;
        bool alive = true;
        SeqInfo sq;
        int hk = 0;
        while (!wk.done && alive) {
            if (wk.j == 0) {
                const int b = wk.r & 1;
                if (wk.r >= 2 && !bwait(bar(B_QEMPTY + b), (uint32_t)(((wk.r >> 1) - 1) & 1), ctl, kStatusWaitQEmpty)) { alive = false; break; }
                sq = a.seqs[wk.seq];
                hk = wk.head0 / G;
                mbar_arrive_expect_tx(bar(q_bar + b), (uint32_t)kQBytes);
                q_armed |= 1u << b; q_par = (q_par & ~(1u << b)) | ((uint32_t)((wk.r >> 1) & 1) << b);
                for (int h = 0; h < 2; ++h)
                    if (a.direct)
                        tma_load_4d(sQ + b * kQBytes + h * 16384, &maps.qt, bar(q_bar + b), h * 64, 0,
                                    sq.chunk0 + wk.q_tile * (kTileM / a.k), wk.head0 + (int)rank);
                    else
                        tma_load_3d(sQ + b * kQBytes + h * 16384, &maps.qt, bar(q_bar + b), h * 64,
                                    sq.text_off + wk.q_tile * kTileM, wk.head0 + (int)rank);
            }
            if (!bwait(bar(B_KEMPTY + stage), phase ^ 1u, ctl, kStatusWaitKvEmpty)) { alive = false; break; }
            const bool summ = wk.j < wk.ns;
            const int bt = wk.band_lo + (wk.j - wk.ns);
            const uint32_t dst = sK + stage * kStageBytes;
            mbar_arrive_expect_tx(bar(k_bar + stage), (uint32_t)kStageBytes);
            armed |= 1u << stage; armed_par = (armed_par & ~(1u << stage)) | (phase << stage);
            // key rows [64 rank, +64) of the tile, both 64-dimension panels
            if (a.direct) {
                const int per = summ ? (kTileN / max(a.m, 1)) : (kTileN / a.k);      // chunks per 128-row tile
                const int zc = sq.chunk0 + (summ ? wk.j : bt) * per + (int)rank * (per >> 1);
                for (int h = 0; h < 2; ++h)
                    tma_load_4d(dst + h * 8192, summ ? &maps.ks : &maps.kt, bar(k_bar + stage), h * 64, 0, zc, hk);
            } else {
                const int y = (summ ? (sq.summ_off + wk.j * kTileN) : (sq.text_off + bt * kTileN)) + (int)rank * 64;
                for (int h = 0; h < 2; ++h)
                    tma_load_3d(dst + h * 8192, summ ? &maps.ks : &maps.kt, bar(k_bar + stage), h * 64, y, hk);
            }
            if (++stage == kKStages) { stage = 0; phase ^= 1u; }
            wk.advance();
        }
        if (lds_u32(abort_addr) != 0u) {
            // leave no copy in flight behind.  Second CTA: wait (bounded) for every load that was issued.  First CTA: its
            // loads complete on barriers that also need the other CTA's arrival, so it waits out a fixed 2^20 cycles.
            if (rank != 0) {
                for (int b = 0; b < 2; ++b)
                    if (q_armed & (1u << b)) bwait_teardown(bar(B_QFULL + b), (q_par >> b) & 1u, a.status, kStatusWaitQFull);
                for (int s = 0; s < kKStages; ++s)
                    if (armed & (1u << s)) bwait_teardown(bar(B_KFULL + s), (armed_par >> s) & 1u, a.status, kStatusWaitKvFull);
            } else {
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 20)) { }
            }
        }
    } else if (warp == kVProdWarp) {
        // =============================== TMA producer: V halves ==========================================
        prefetch_tensormap(&maps.vt); prefetch_tensormap(&maps.vs);
        Walk wk;
        wk.init(a, pairs, cid);
        const int G = a.Hq / a.Hkv;
        const int v_bar = rank == 0 ? B_VPAIR : B_VFULL;
        int stage = 0; uint32_t phase = 0;
        uint32_t armed = 0, armed_par = 0;
        bool alive = true;
        SeqInfo sq;
        int hk = 0;
        while (!wk.done && alive) {
            if (wk.j == 0) { sq = a.seqs[wk.seq]; hk = wk.head0 / G; }
            if (!bwait(bar(B_VEMPTY + stage), phase ^ 1u, ctl, kStatusWaitKvEmpty)) { alive = false; break; }
            const bool summ = wk.j < wk.ns;
            const int bt = wk.band_lo + (wk.j - wk.ns);
            const uint32_t dst = sV + stage * kStageBytes;
            mbar_arrive_expect_tx(bar(v_bar + stage), (uint32_t)kStageBytes);
            armed |= 1u << stage; armed_par = (armed_par & ~(1u << stage)) | (phase << stage);
            // head dimensions [64 rank, +64) of all 128 keys of the tile
            if (a.direct) {
                const int zc = sq.chunk0 + (summ ? (kTileN / max(a.m, 1)) * wk.j : (kTileN / a.k) * bt);
                tma_load_4d(dst, summ ? &maps.vs : &maps.vt, bar(v_bar + stage), (int)rank * 64, 0, zc, hk);
            } else {
                const int y = summ ? (sq.summ_off + wk.j * kTileN) : (sq.text_off + bt * kTileN);
                tma_load_3d(dst, summ ? &maps.vs : &maps.vt, bar(v_bar + stage), (int)rank * 64, y, hk);
            }
            if (++stage == kVStages) { stage = 0; phase ^= 1u; }
            wk.advance();
        }
        if (lds_u32(abort_addr) != 0u) {
            if (rank != 0) {
                for (int s = 0; s < kVStages; ++s)
                    if (armed & (1u << s)) bwait_teardown(bar(B_VFULL + s), (armed_par >> s) & 1u, a.status, kStatusWaitKvFull);
            } else {
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 20)) { }
            }
        }
    } else if (warp == kQkWarp && rank == 0) {
        // =============================== issuer of S = Q K^T (first CTA) ================================
        constexpr uint32_t idesc_qk = make_idesc_bf16(256, 128, false);
        constexpr uint16_t both = 3;
        WalkLite wk;
        wk.init(a, pairs, cid);
        int stage = 0; uint32_t phase = 0;
        uint32_t g = 0;                                       // tiles issued so far
        const uint64_t d0 = make_smem_desc_sw128(0, 16, 1024);
        const uint32_t dhi = (uint32_t)(d0 >> 32), dlo = (uint32_t)d0;
        KSA_PT_DECL;
        while (!wk.done) {
            const int qb = wk.r & 1;
            const uint32_t sb = g & 1u;
            KSA_PT_BEGIN();
            if (wk.j == 0 && !bwait(bar(B_QPAIR + qb), (uint32_t)((wk.r >> 1) & 1), ctl, kStatusWaitQFull)) break;
            if (!bwait(bar(B_KPAIR + stage), phase, ctl, kStatusWaitKvFull)) break;
            KSA_PT_END(0);
            KSA_PT_BEGIN();
            // the score buffer's previous tile (g - 2) is in its softmax warps' registers
            if (g >= 2 && !bwait(bar(B_SFREE + sb), ((g >> 1) - 1u) & 1u, ctl, kStatusWaitSFull)) break;
            KSA_PT_END(1);
            KSA_PT_BEGIN();
            tc_fence_after();
            const uint32_t qlo = dlo + ((sQ + qb * kQBytes) >> 4);
            const uint32_t klo = dlo + ((sK + stage * kStageBytes) >> 4);
            const uint32_t dS = tmem + sb * 128u;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t qoff = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                const uint32_t koff = (uint32_t)((kk >> 2) * 8192 + (kk & 3) * 32) >> 4;
                mma_ss_pair(dS, desc_from(qlo + qoff, dhi), desc_from(klo + koff, dhi), idesc_qk, kk > 0 ? 1u : 0u);
            }
            tc_commit_pair(bar(B_SFULL + sb), both);
            tc_commit_pair(bar(B_KEMPTY + stage), both);
            if (wk.j == wk.T - 1) tc_commit_pair(bar(B_QEMPTY + qb), both);
            KSA_PT_END(2);
            KSA_PT_COUNT(6);
            if (++stage == kKStages) { stage = 0; phase ^= 1u; }
            ++g;
            wk.advance();
        }
        // drain this thread's products before the pair tears down
        tc_commit_pair(bar(B_DRAIN + 0), (uint16_t)1);
        bwait_teardown(bar(B_DRAIN + 0), 0, a.status, kStatusWaitOFull);
        KSA_PT_FLUSH(0, blockIdx.x == 0);
    } else if (warp == kPvWarp && rank == 0) {
        // =============================== issuer of O += P V (first CTA) =================================
        constexpr uint32_t idesc_pv = make_idesc_bf16(256, D, true);
        constexpr uint16_t both = 3;
        WalkLite wk;
        wk.init(a, pairs, cid);
        int stage = 0; uint32_t phase = 0;
        uint32_t g = 0;
        const uint64_t d0 = make_smem_desc_sw128(0, 16384, 1024);
        const uint32_t dhi = (uint32_t)(d0 >> 32), dlo = (uint32_t)d0;
        KSA_PT_DECL;
        while (!wk.done) {
            const uint32_t sb = g & 1u;
            KSA_PT_BEGIN();
            if (!bwait(bar(B_VPAIR + stage), phase, ctl, kStatusWaitKvFull)) break;
            KSA_PT_END(0);
            KSA_PT_BEGIN();
            if (!bwait(bar(B_PFULL + sb), (g >> 1) & 1u, ctl, kStatusWaitPFull)) break;
            KSA_PT_END(1);
            KSA_PT_BEGIN();
            // the epilogue of the item before has read O
            if (wk.j == 0 && wk.r > 0 && !bwait(bar(B_OEMPTY), (uint32_t)((wk.r - 1) & 1), ctl, kStatusWaitOEmpty)) break;
            KSA_PT_END(3);
            KSA_PT_BEGIN();
            tc_fence_after();
            const uint32_t vlo = dlo + ((sV + stage * kStageBytes) >> 4);
            const uint32_t aP = tmem + kColP + sb * 64u;
#pragma unroll
            for (int kk = 0; kk < kTileN / 16; ++kk)
                mma_ts_pair(tmem + kColO, aP + kk * 8, desc_from(vlo + (uint32_t)((kk * 2048) >> 4), dhi), idesc_pv,
                            (wk.j > 0 || kk > 0) ? 1u : 0u);
            tc_commit_pair(bar(B_PVDONE + sb), both);
            tc_commit_pair(bar(B_VEMPTY + stage), both);
            KSA_PT_END(2);
            KSA_PT_COUNT(6);
            if (++stage == kVStages) { stage = 0; phase ^= 1u; }
            ++g;
            wk.advance();
        }
        tc_commit_pair(bar(B_DRAIN + 1), (uint16_t)1);
        bwait_teardown(bar(B_DRAIN + 1), 0, a.status, kStatusWaitOFull);
        KSA_PT_FLUSH(48, blockIdx.x == 0);
    } else if (warp == kQkWarp) {
        // =============================== second CTA: forward "Q tile / K half landed" ====================
        WalkLite wk;
        wk.init(a, pairs, cid);
        int stage = 0; uint32_t phase = 0;
        while (!wk.done) {
            if (wk.j == 0) {
                const int b = wk.r & 1;
                if (!bwait(bar(B_QFULL + b), (uint32_t)((wk.r >> 1) & 1), ctl, kStatusWaitQFull)) break;
                mbar_arrive_cluster(lead(bar(B_QPAIR + b)));
            }
            if (!bwait(bar(B_KFULL + stage), phase, ctl, kStatusWaitKvFull)) break;
            mbar_arrive_cluster(lead(bar(B_KPAIR + stage)));
            if (++stage == kKStages) { stage = 0; phase ^= 1u; }
            wk.advance();
        }
    } else if (warp == kPvWarp) {
        // =============================== second CTA: forward "V half landed" =============================
        WalkLite wk;
        wk.init(a, pairs, cid);
        int stage = 0; uint32_t phase = 0;
        while (!wk.done) {
            if (!bwait(bar(B_VFULL + stage), phase, ctl, kStatusWaitKvFull)) break;
            mbar_arrive_cluster(lead(bar(B_VPAIR + stage)));
            if (++stage == kVStages) { stage = 0; phase ^= 1u; }
            wk.advance();
        }
    }
    }
    } else {
        setmaxnreg_inc<kRegsSoftmax>();
        // =============================== softmax groups ==================================================
        const int wg = warp >> 2;                       // takes the tiles g with g mod 2 == wg: S and P buffer wg
        const int w4 = warp & 3;                        // row quarter = TMEM lane quarter
        const int row = tid & 127;
        const uint32_t lane_sel = (uint32_t)(w4 * 32) << 16;
        const uint32_t tS = tmem + lane_sel + (uint32_t)wg * 128u;
        const uint32_t tP = tmem + lane_sel + kColP + (uint32_t)wg * 64u;
        const uint32_t tO = tmem + lane_sel + kColO;
        const float scale_log2 = a.scale_log2;
        const int s_len = a.k + a.m;
        // Publication of the reference maximum, row by row: the thread that takes tile g writes {m, g + 1} as ONE 8-byte
        // word into slot g mod 2 of its row; the thread of the other group that takes tile g + 1 reads that word until
        // the tag is g + 1.  Value and tag travel together, so no barrier and no fence is involved.  The slot is rewritten
        // at tile g + 2, which its writer starts only after it has seen the tag of tile g + 1 -- written after this read.
        const uint32_t msh_mine = smem_base + kMshOff + 8u * ((uint32_t)wg * 128u + (uint32_t)row);
        const uint32_t msh_other = smem_base + kMshOff + 8u * ((uint32_t)(wg ^ 1) * 128u + (uint32_t)row);
        bool alive = true;
        WalkLite wk;
        wk.init(a, pairs, cid);
        uint32_t gbase = 0;                              // stream index of the item's first tile
#ifdef KSA_PAIR_TRACE
        const bool pt_on_ = blockIdx.x == 0 && row == 0;
#endif
        KSA_PT_DECL;
        for (; !wk.done && alive; ) {
            const WorkItem w = a.work[wk.r * pairs + ((wk.r & 1) ? (pairs - 1 - cid) : cid)];
            const SeqInfo sq = a.seqs[w.seq];
            const int T = wk.T;
            const int i_raw = w.q_tile * kTileM + row;
            const bool valid = i_raw < sq.n_text;
            const int i = valid ? i_raw : sq.n_text - 1;     // padding rows mimic the last row; never stored
            const int chunk = i / a.k;
            const int far = max(0, chunk - a.C);
            const int lo_i = far * a.k;                      // Eq. 3: first visible text token
            const int cnt_i = far * a.m;                     // Eq. 3: summaries [0, cnt_i) visible
            float m_seen = -INFINITY, l_own = 0.f;           // my tiles' row sum, relative to m_seen

            for (int j = (int)((gbase ^ (uint32_t)wg) & 1u); j < T; j += 2) {
                const uint32_t g = gbase + (uint32_t)j;
                const uint32_t kown = g >> 1;                 // my tiles before this one
                KSA_PT_BEGIN();
                bool ok = bwait(bar(B_SFULL + wg), kown & 1u, ctl, kStatusWaitSFull);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { alive = false; break; }
                KSA_PT_END(0);
                KSA_PT_COUNT(6);
                KSA_PT_BEGIN();
                tc_fence_after();
                uint32_t s[128];
                {
                    uint32_t (&c0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[0]);
                    uint32_t (&c1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[32]);
                    uint32_t (&c2)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[64]);
                    uint32_t (&c3)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[96]);
                    tmem_ld32(tS + 0, c0); tmem_ld32(tS + 32, c1); tmem_ld32(tS + 64, c2); tmem_ld32(tS + 96, c3);
                }
                tc_wait_ld();
                KSA_PT_END(1);
                KSA_PT_BEGIN();
                // the scores are in registers: the buffer can take Q K^T of tile g + 2
                tc_fence_before();
                KSA_PT_END(11);
                KSA_PT_BEGIN();
                if (lane == 0) mbar_arrive_cluster_relaxed(lead(bar(B_SFREE + wg)));
                KSA_PT_END(5);
                KSA_PT_BEGIN();
                // in-tile mask, only where the schedule says the tile is partial
                bool masked;
                int ca, cb;                                   // visible columns [ca, cb)
                if (j < w.ns_tiles) {
                    masked = j >= w.ns_nomask;
                    ca = 0; cb = cnt_i - j * kTileN;
                } else {
                    const int bt = w.band_lo + (j - w.ns_tiles);
                    masked = !(bt >= w.band_nomask_lo && bt < w.band_nomask_hi);
                    ca = lo_i - bt * kTileN; cb = i + 1 - bt * kTileN;
                }
                if (masked) {
                    const uint32_t width = (uint32_t)max(cb - ca, 0);
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if ((uint32_t)(c - ca) >= width) s[c] = 0xff800000u;   // -inf
                }
                KSA_PT_END(8);
                KSA_PT_BEGIN();
                // row maximum: eight independent chains of 3-input maxima (the instruction's latency, not its issue
                // rate, is what a lone warp on a sub-partition feels)
                float mx[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) mx[c] = fmaxf(__uint_as_float(s[2 * c]), __uint_as_float(s[2 * c + 1]));
#pragma unroll
                for (int c = 16; c < 128; c += 16)
#pragma unroll
                    for (int e = 0; e < 8; ++e) mx[e] = fmax3(mx[e], __uint_as_float(s[c + 2 * e]), __uint_as_float(s[c + 2 * e + 1]));
                const float mx_sc = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]))) * scale_log2;
                KSA_PT_END(9);
                KSA_PT_BEGIN();
                // the reference maximum as the other group left it after tile g - 1
                float m_pub = -INFINITY;
                if (g > 0) {
                    ok = wait_tagged(msh_other, g, m_pub, ctl, kStatusWaitMaxPub);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) { alive = false; break; }
                }
                KSA_PT_END(2);
                KSA_PT_BEGIN();
                const float m_prev = (j == 0) ? -INFINITY : m_pub;
                // lazy rescale: a row's reference only moves when the row outgrew it by 2^8
                const bool need = mx_sc > m_prev + kRescaleThreshold;
                const float m_used = need ? mx_sc : m_prev;
                sts_tagged(msh_mine, m_used, g + 1u);
                if (m_seen != m_used) {
                    l_own = (m_seen == -INFINITY) ? 0.f : l_own * ex2_approx(m_seen - m_used);
                    m_seen = m_used;
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                KSA_PT_END(10);
                KSA_PT_BEGIN();
                const float2 sc2 = make_float2(scale_log2, scale_log2);
                const float2 nm2 = make_float2(neg_m, neg_m);
                float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
                for (int q = 0; q < 64; ++q) {
                    const float2 x = ffma2(make_float2(__uint_as_float(s[2 * q]), __uint_as_float(s[2 * q + 1])), sc2, nm2);
                    float2 pr;
                    pr.x = ex2_approx(x.x); pr.y = ex2_approx(x.y);
                    if (q & 1) lb = fadd2(lb, pr); else la = fadd2(la, pr);
                    s[q] = pack_bf16x2(pr.x, pr.y);
                }
                l_own += (la.x + la.y) + (lb.x + lb.y);
                KSA_PT_END(3);
                KSA_PT_BEGIN();
                // my probability buffer was last read by the product of my previous tile (g - 2)
                if (kown > 0) {
                    ok = bwait(bar(B_PVDONE + wg), (kown - 1u) & 1u, ctl, kStatusWaitPvDone);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) { alive = false; break; }
                    tc_fence_after();
                }
                {
                    uint32_t (&p0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[0]);
                    uint32_t (&p1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[32]);
                    tmem_st32(tP + 0, p0); tmem_st32(tP + 32, p1);
                }
                if (j > 0 && __any_sync(0xffffffffu, need)) {
                    // O holds the products up to tile g - 1 once that product has completed; the product of tile g
                    // cannot start before this warp releases P(g) below.  Rows whose reference stayed scale by 1.
                    const float alpha = (need && m_prev != -INFINITY) ? ex2_approx(m_prev - m_used) : 1.f;
                    const uint32_t gm = g - 1u;
                    ok = bwait(bar(B_PVDONE + (wg ^ 1)), (gm >> 1) & 1u, ctl, kStatusWaitPvDone);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) { alive = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + c * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tmem_st32(tO + c * 32, o);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_relaxed(lead(bar(B_PFULL + wg)));
                KSA_PT_END(4);
            }
            if (!alive) break;
            KSA_PT_BEGIN();
            // ---- epilogue: the two groups add their row sums; group wg writes head dimensions [64 wg, +64) ----
            const uint32_t par = (uint32_t)(wk.r & 1);
            const uint32_t l_mine = smem_base + kLshOff + 4u * ((par * 2u + (uint32_t)wg) * 128u + (uint32_t)row);
            const uint32_t l_oth = smem_base + kLshOff + 4u * ((par * 2u + (uint32_t)(wg ^ 1)) * 128u + (uint32_t)row);
            sts_f32(l_mine, l_own);
            sts_f32(l_mine + (kMs2Off - kLshOff), m_seen);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_LBAR + w4));
            bool ok = bwait(bar(B_LBAR + w4), par, ctl, kStatusWaitRowSums);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const float l_o = lds_f32(l_oth), m_o = lds_f32(l_oth + (kMs2Off - kLshOff));
            const float m_fin = fmaxf(m_seen, m_o);
            const float l_tot = ((m_seen == -INFINITY) ? 0.f : l_own * ex2_approx(m_seen - m_fin)) +
                                ((m_o == -INFINITY) ? 0.f : l_o * ex2_approx(m_o - m_fin));
            const uint32_t gl = gbase + (uint32_t)T - 1u;
            ok = bwait(bar(B_PVDONE + (int)(gl & 1u)), (gl >> 1) & 1u, ctl, kStatusWaitPvDone);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float inv_l = 1.f / l_tot;
            const int h = w.head0 + (int)rank;
            const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * s_len + (i % a.k);
            uint16_t* orow = a.out + aug * a.o_st + (int64_t)h * a.o_sh + wg * 64;
            const bool store = valid && ksa_out_row_ok(a, aug, h);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + wg * 64 + c * 32, o);
                tc_wait_ld();
                if (store) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 pk;
                        pk.x = pack_bf16x2(__uint_as_float(o[e]) * inv_l, __uint_as_float(o[e + 1]) * inv_l);
                        pk.y = pack_bf16x2(__uint_as_float(o[e + 2]) * inv_l, __uint_as_float(o[e + 3]) * inv_l);
                        pk.z = pack_bf16x2(__uint_as_float(o[e + 4]) * inv_l, __uint_as_float(o[e + 5]) * inv_l);
                        pk.w = pack_bf16x2(__uint_as_float(o[e + 6]) * inv_l, __uint_as_float(o[e + 7]) * inv_l);
                        *reinterpret_cast<uint4*>(orow + c * 32 + e) = pk;
                    }
                }
            }
            if (store && wg == 0) a.lse[(int64_t)h * a.total_aug + aug] = (m_fin + log2f(l_tot)) * 0.6931471805599453f;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_relaxed(lead(bar(B_OEMPTY)));
            KSA_PT_END(5);
            gbase += (uint32_t)T;
            ++wk.r;
            wk.load();
        }
        KSA_PT_FLUSH(16 + wg * 16, pt_on_);
    }

    // Neither CTA leaves (or frees its TMEM) while the other may still read its shared memory or signal its barriers.
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (warp == kQkWarp) tmem_dealloc_pair(tmem, 512);
}

}  // namespace pairk

#ifdef KSA_PAIR_TRACE
extern "C" __attribute__((visibility("default"))) int ksa_debug_pair_trace(void* sums, int reset)
{
    cudaDeviceSynchronize();
    if (sums) cudaMemcpyFromSymbol(sums, pairk::g_pair_trace, sizeof(pairk::g_pair_trace));
    if (reset) { static unsigned long long z[64] = {0}; cudaMemcpyToSymbol(pairk::g_pair_trace, z, sizeof(z)); }
    return (int)cudaGetLastError();
}
#endif

cudaError_t setup_text_pair(int* max_pairs)
{
    cudaError_t e = cudaFuncSetAttribute(pairk::ksa_text_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pairk::kSmemBytes);
    if (e != cudaSuccess) return e;
    // how many pairs the device runs at once (one CTA per SM, two SMs of one cluster per pair)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(pairk::kThreads, 1, 1);
    cfg.dynamicSmemBytes = pairk::kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, pairk::ksa_text_pair_kernel, &cfg);
    if (e != cudaSuccess) return e;
    *max_pairs = n;
    return cudaSuccess;
}

cudaError_t launch_text_pair(const KernelArgs& a, const PairMaps& maps, int max_pairs, cudaStream_t stream)
{
    if (a.num_work <= 0) return cudaSuccess;
    const int npairs = a.num_work < max_pairs ? a.num_work : max_pairs;
    pairk::ksa_text_pair_kernel<<<2 * npairs, pairk::kThreads, pairk::kSmemBytes, stream>>>(a, maps);
    return cudaGetLastError();
}

}  // namespace ksa
