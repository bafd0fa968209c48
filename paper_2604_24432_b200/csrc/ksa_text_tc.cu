// Text-row KSA attention on the sm_100a tensor cores.
//
// One persistent CTA per SM walks its share of the work list.  A work item is one tile of
// 128 text query rows for one or two query heads that share a KV head, plus the key/value
// tiles Eq. 3 makes visible to it: tiles of the packed summary stream first, then tiles of
// the packed text stream (the sliding-chunk band up to the diagonal).
//
// Warp roles (384 threads = three warpgroups; warps 10-11 idle, they complete the third one):
//   warps 0-3   softmax of query tile 0 (one row per thread), O rescale, epilogue
//   warps 4-7   softmax of query tile 1
//   warp  8     TMA producer: Q tiles, then K and V tiles through a ring of smem stages
//   warp  9     MMA issuer: S = Q K^T (smem x smem) and O += P V (P from TMEM) via tcgen05.mma
// TMEM (512 columns): S0 [0,128), S1 [128,256), O0 [256,256+D), O1 [384,384+D); the bf16
// probabilities P_t overwrite the first 64 columns of S_t.
//
// Pipeline per key/value tile j and query tile t:
//   MMA:     S_t(j) = Q_t K(j)^T                                   -> s_full[t]
//   softmax: load S_t, mask (only on tiles flagged partial), running max with lazy rescale,
//            p = 2^(s*scale*log2e - m), row sum, write P_t, rescale O_t if the max moved -> p_full[t]
//   MMA:     O_t += P_t V(j), then at once S_t(j+1) = Q_t K(j+1)^T -> s_full[t]
// so that while one query tile is in its softmax the tensor pipe works for the other.
// tcgen05.mma operations of one thread execute in issue order, which is what lets S_t(j+1)
// overwrite P_t(j) right after O_t += P_t(j) V(j) was issued, and what makes s_full[t] of
// tile j imply that O_t += P_t V(j-1) has completed (so the softmax warps may rescale O_t).
//
// Every mbarrier wait is bounded: on timeout the thread records which wait gave up in the
// status word, raises a CTA-wide abort flag, all roles leave their loops, the producer
// waits (bounded) for its copies in flight, TMEM is freed and the kernel returns.
#include <cuda_bf16.h>

#include "ksa_launch.h"
#include "ksa_ptx.cuh"
#include "ksa_wait.cuh"

namespace ksa {

using namespace ptx;

// Optional event trace (compile with -DKSA_TRACE): CTAs 0 and 100 record (event id, clock) pairs
// per role into a device buffer that ksa_debug_read_trace() copies out.  Compiled out by default.
#ifdef KSA_TRACE
constexpr int kTraceEvents = 8192;
constexpr int kTraceRoles = 12;             // 0 MMA issuer, 1-2 softmax row 0 of tile 0/1, 3 producer, 4-11 per-warp arrivals
__device__ uint2 g_trace[2][kTraceRoles][kTraceEvents];
__device__ uint32_t g_trace_cnt[2][kTraceRoles];
__device__ unsigned long long g_cta_span[2][256];   // start / end of every CTA (globaltimer, ns)
#define KSA_TR(role, id)                                                                           \
    do {                                                                                           \
        if (tr_slot >= 0 && tr_n < (uint32_t)kTraceEvents) {                                       \
            g_trace[tr_slot][role][tr_n] = make_uint2((uint32_t)(id), (uint32_t)clock64());        \
            g_trace_cnt[tr_slot][role] = ++tr_n;                                                   \
        }                                                                                          \
    } while (0)
#else
#define KSA_TR(role, id) do { } while (0)
#endif

constexpr int kThreadsTc = 384;           // three warpgroups; warps 10 and 11 only take part in the register hand-over
constexpr int kRegsSoftmax = 216;         // registers per thread of the softmax warpgroups after the hand-over
constexpr int kRegsOther = 72;            // ... of the producer / MMA warpgroup
// The CTA's register allocation is fixed at launch (65,536 / 384 threads = 170 -> 168 per thread): the softmax warps
// can only gain what the third warpgroup gives up; a larger setmaxnreg.inc would wait forever.
static_assert(8 * kRegsSoftmax + 4 * kRegsOther <= 12 * ((65536 / 384) / 8 * 8), "register hand-over exceeds the CTA's allocation");
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
// log2 units: P stays below 2^12.  A small threshold costs rescales of O: with 1 % of the keys four times larger (the 128k
// workload) some row of nearly every warp outgrew 2^8 once or twice per work item.  Measured at 128k: 8 -> 1,032,
// 12 -> 1,047, 20 -> 1,058 TFLOP/s, but the error against the fp64 oracle grows with it (mean |err| 5.6e-4, 5.9e-4,
// 6.2e-4; at 20 one sampled element of the 64 + 8 layout left the 2e-2 bound), so 12 it is.
constexpr float kRescaleThreshold = 12.0f;

template <int D>
struct TcCfg {
    static constexpr int kTileBytes = 128 * D * 2;
    static constexpr int kHalves = D / 64;                       // 64-column (128-byte) swizzle panels
    static constexpr int kStages = (D == 128) ? 5 : 10;          // K/V ring depth (tiles)
    static constexpr int kQOff = 0;
    static constexpr int kRingOff = 2 * kTileBytes;
    static constexpr int kBarOff = kRingOff + kStages * kTileBytes;
    static constexpr int kNumBars = 9 + 2 * kStages;
    static constexpr int kSmemBytes = kBarOff + 8 * kNumBars + 64 + 1024;   // + slack for 1024-byte alignment
    // MN-major V operand: the two 64-column panels of a D = 128 tile are 16 KB apart,
    // groups of 8 keys are 1 KB apart.
    static constexpr uint32_t kVLbo = 16384;
    static constexpr uint32_t kVSbo = 1024;
};

// barrier slots
enum : int { BAR_QFULL = 0, BAR_QEMPTY = 1, BAR_SFULL = 2, BAR_PFULL = 4, BAR_OFULL = 6, BAR_DRAIN = 8, BAR_KV = 9 };

struct TcShared {
    uint32_t bars;        // smem address of barrier 0
    uint32_t abort_addr;  // smem address of the abort flag
};

template <int D>
__global__ void __launch_bounds__(kThreadsTc, 1)
ksa_text_tc_kernel(const __grid_constant__ KernelArgs a, const __grid_constant__ TextMaps maps)
{
    using Cfg = TcCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + Cfg::kQOff;
    const uint32_t sRing = smem_base + Cfg::kRingOff;
    const uint32_t bars = smem_base + Cfg::kBarOff;
    const uint32_t tmem_slot = bars + 8 * Cfg::kNumBars;
    const uint32_t abort_addr = tmem_slot + 4;
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    auto kv_full = [&](int s) -> uint32_t { return bars + 8u * (uint32_t)(BAR_KV + s); };
    auto kv_empty = [&](int s) -> uint32_t { return bars + 8u * (uint32_t)(BAR_KV + Cfg::kStages + s); };

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
#ifdef KSA_TRACE
    const int tr_slot = (blockIdx.x == 0) ? 0 : ((blockIdx.x == 100) ? 1 : -1);
    uint32_t tr_n = 0;
    if (tid == 0 && blockIdx.x < 256) { unsigned long long t_; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_)); g_cta_span[0][blockIdx.x] = t_; }
#endif

    if (tid == 0) {
        mbar_init(bar(BAR_QFULL), 1);
        mbar_init(bar(BAR_QEMPTY), 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(BAR_SFULL + t), 1);
            mbar_init(bar(BAR_PFULL + t), 4);      // one arrival per softmax warp
            mbar_init(bar(BAR_OFULL + t), 1);
        }
        mbar_init(bar(BAR_DRAIN), 1);
        for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), 1); }
        st_shared_u32(abort_addr, 0u);
        st_shared_u32(abort_addr + 4, 0u);     // never raised: lets the teardown waits run while aborting
        fence_mbar_init();
    }
    if (warp == kProducerWarp) {            // one warp allocates all 512 TMEM columns (1 CTA per SM)
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ld_shared_u32(tmem_slot);

    const int G = a.Hq / a.Hkv;
    const int grid = (int)gridDim.x;
    const int cta = (int)blockIdx.x;
    // items are taken in snake order over the longest-first list: round r gives this CTA
    // item r*grid + cta (even r) or r*grid + grid-1-cta (odd r)
    auto item_index = [&](int r) -> int { return r * grid + ((r & 1) ? (grid - 1 - cta) : cta); };

    if (warp >= 8) {
    // register hand-over: this warpgroup gives most of its registers to the softmax warpgroups,
    // which keep a whole 128-column score row per thread
    setmaxnreg_dec<kRegsOther>();
    if (warp == kProducerWarp) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            prefetch_tensormap(&maps.qt); prefetch_tensormap(&maps.kt); prefetch_tensormap(&maps.vt);
            prefetch_tensormap(&maps.ks); prefetch_tensormap(&maps.vs);
            uint32_t q_phase = 0, ring_phase = 0;
            int stage = 0;
            uint32_t armed_mask = 0, armed_parity = 0;   // per stage: a load was issued / with which parity
            bool q_armed = false;
            bool alive = true;
            for (int r = 0; alive; ++r) {
                const int idx = item_index(r);
                if (idx >= a.num_work) break;
                const WorkItem w = a.work[idx];
                const SeqInfo sq = a.seqs[w.seq];
                // the two query heads of an item share a KV head (one K and one V tile per key tile) or, where a pair
                // straddles two KV heads (multi-head attention, odd group sizes), each has its own: then every key tile
                // takes four ring stages, K for head 0, K for head 1, V for head 0, V for head 1
                const int hk = w.head0 / G;
                const int nsplit = ((w.head0 + w.n_heads - 1) / G != hk) ? 2 : 1;
                const int T = w.ns_tiles + (w.band_hi - w.band_lo + 1);
                if (!bounded_wait(bar(BAR_QEMPTY), q_phase ^ 1u, abort_addr, a.status, kStatusWaitQEmpty)) break;
                mbar_arrive_expect_tx(bar(BAR_QFULL), (uint32_t)(w.n_heads * Cfg::kTileBytes));
                q_armed = true;
                for (int t = 0; t < w.n_heads; ++t)
                    for (int h = 0; h < Cfg::kHalves; ++h)
                        if (a.direct)
                            tma_load_4d(sQ + t * Cfg::kTileBytes + h * 16384, &maps.qt, bar(BAR_QFULL),
                                        h * 64, 0, sq.chunk0 + w.q_tile * (kTileM / a.k), w.head0 + t);
                        else
                            tma_load_3d(sQ + t * Cfg::kTileBytes + h * 16384, &maps.qt, bar(BAR_QFULL),
                                        h * 64, sq.text_off + w.q_tile * kTileM, w.head0 + t);
                q_phase ^= 1u;
                for (int j = 0; j < T && alive; ++j) {
                    const bool summ = j < w.ns_tiles;
                    const int y = summ ? (sq.summ_off + j * kTileN) : (sq.text_off + (w.band_lo + j - w.ns_tiles) * kTileN);
                    // direct views: a tile is 128/m chunks of the summary view or 128/k chunks of the text view
                    const int zc = sq.chunk0 + (summ ? j * (kTileN / max(a.m, 1)) : (w.band_lo + j - w.ns_tiles) * (kTileN / a.k));
                    const CUtensorMap* mk = summ ? &maps.ks : &maps.kt;
                    const CUtensorMap* mv = summ ? &maps.vs : &maps.vt;
                    for (int kvt = 0; kvt < 2 * nsplit && alive; ++kvt) {
                        const int kv = kvt / nsplit, hkt = hk + kvt % nsplit;
                        if (!bounded_wait(kv_empty(stage), ring_phase ^ 1u, abort_addr, a.status, kStatusWaitKvEmpty)) { alive = false; break; }
                        mbar_arrive_expect_tx(kv_full(stage), (uint32_t)Cfg::kTileBytes);
                        armed_mask |= 1u << stage;
                        armed_parity = (armed_parity & ~(1u << stage)) | (ring_phase << stage);
                        for (int h = 0; h < Cfg::kHalves; ++h)
                            if (a.direct)
                                tma_load_4d(sRing + stage * Cfg::kTileBytes + h * 16384, kv ? mv : mk, kv_full(stage), h * 64, 0, zc, hkt);
                            else
                                tma_load_3d(sRing + stage * Cfg::kTileBytes + h * 16384, kv ? mv : mk, kv_full(stage), h * 64, y, hkt);
                        if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                    }
                }
            }
            if (ld_shared_u32(abort_addr) != 0u) {
                // leave no copy in flight behind: wait (bounded) for every load that was issued
                if (q_armed) bounded_wait(bar(BAR_QFULL), q_phase ^ 1u, abort_addr + 4, a.status, kStatusWaitQFull);
                for (int s = 0; s < Cfg::kStages; ++s)
                    if (armed_mask & (1u << s))
                        bounded_wait(kv_full(s), (armed_parity >> s) & 1u, abort_addr + 4, a.status, kStatusWaitKvFull);
            }
        }
    } else if (warp == kMmaWarp) {
        // =============================== MMA issuer =================================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
            uint32_t qf_phase = 0, pf_phase[2] = {0, 0}, ring_phase = 0;
            int stage = 0;
            bool alive = true;
            auto issue_qk = [&](int t, int st) {
                const uint64_t qd = make_smem_desc_sw128(sQ + t * Cfg::kTileBytes, 16, 1024);
                const uint64_t kd = make_smem_desc_sw128(sRing + st * Cfg::kTileBytes, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    mma_ss(tmem + t * 128, qd + off, kd + off, idesc_qk, kk > 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, int st, bool acc) {
                const uint64_t vd = make_smem_desc_sw128(sRing + st * Cfg::kTileBytes, Cfg::kVLbo, Cfg::kVSbo);
#pragma unroll
                for (int kk = 0; kk < kTileN / 16; ++kk)
                    mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, vd + (uint32_t)((kk * 2048) >> 4), idesc_pv,
                           (acc || kk > 0) ? 1u : 0u);
            };
            for (int r = 0; alive; ++r) {
                const int idx = item_index(r);
                if (idx >= a.num_work) break;
                const WorkItem w = a.work[idx];
                const int T = w.ns_tiles + (w.band_hi - w.band_lo + 1);
                const int nh = w.n_heads;
                // one K and one V stage per key tile, or one per query head where the pair straddles two KV heads
                const int nsplit = ((w.head0 + nh - 1) / G != w.head0 / G) ? 2 : 1;
                if (nsplit == 1) {
                // ---- one K and one V stage per key tile (the two heads share a KV head, or a single head) ----
                    if (!bounded_wait(bar(BAR_QFULL), qf_phase, abort_addr, a.status, kStatusWaitQFull)) break;
                    qf_phase ^= 1u;
                    if (!bounded_wait(kv_full(stage), ring_phase, abort_addr, a.status, kStatusWaitKvFull)) break;
                    tc_fence_after();
                    for (int t = 0; t < nh; ++t) { issue_qk(t, stage); tc_commit(bar(BAR_SFULL + t)); }
                    if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                    for (int j = 0; j < T && alive; ++j) {
                        const int vstage = stage; const uint32_t vphase = ring_phase;
                        if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                        int kstage = -1; uint32_t kphase = 0;
                        if (j + 1 < T) {
                            kstage = stage; kphase = ring_phase;
                            if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                        }
                        KSA_TR(0, 39);
                        // both stages of this iteration are checked here, while the softmax warps still work on P_0: the ring
                        // runs two tiles ahead, so neither wait depends on anything this iteration does
                        if (!bounded_wait(kv_full(vstage), vphase, abort_addr, a.status, kStatusWaitKvFull)) { alive = false; break; }
                        if (kstage >= 0 && !bounded_wait(kv_full(kstage), kphase, abort_addr, a.status, kStatusWaitKvFull)) { alive = false; break; }
                        KSA_TR(0, 40);
                        for (int t = 0; t < nh; ++t) {
                            if (!bounded_wait(bar(BAR_PFULL + t), pf_phase[t], abort_addr, a.status, kStatusWaitPFull)) { alive = false; break; }
                            pf_phase[t] ^= 1u;
                            KSA_TR(0, 20 + t);
                            tc_fence_after();
                            issue_pv(t, vstage, j > 0);
                            KSA_TR(0, 25 + t);
                            if (j == T - 1) tc_commit(bar(BAR_OFULL + t));
                            if (j + 1 < T) {
                                issue_qk(t, kstage);
                                tc_commit(bar(BAR_SFULL + t));
                                KSA_TR(0, 30 + t);
                            }
                        }
                        if (!alive) break;
                    }
                } else {
                // ---- a pair that straddles two KV heads: every head has its own K and V stage ----
                    if (!bounded_wait(bar(BAR_QFULL), qf_phase, abort_addr, a.status, kStatusWaitQFull)) break;
                    qf_phase ^= 1u;
                    // stage and phase of the K and the V tile of query tile 0 / 1 (scalars: no indexed local arrays)
                    int kst0, kst1, vst0 = 0, vst1 = 0;
                    uint32_t kph0, kph1, vph0 = 0, vph1 = 0;
                    auto take = [&](int& st0, uint32_t& ph0, int& st1, uint32_t& ph1) {   // the next nsplit stages of the ring (not waited for yet)
                        st0 = stage; ph0 = ring_phase;
                        if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                        st1 = st0; ph1 = ph0;
                        if (nsplit == 2) {
                            st1 = stage; ph1 = ring_phase;
                            if (++stage == Cfg::kStages) { stage = 0; ring_phase ^= 1u; }
                        }
                    };
                    auto full = [&](int st, uint32_t ph) -> bool { return bounded_wait(kv_full(st), ph, abort_addr, a.status, kStatusWaitKvFull); };
                    take(kst0, kph0, kst1, kph1);
                    if (!full(kst0, kph0) || !full(kst1, kph1)) break;
                    tc_fence_after();
                    for (int t = 0; t < nh; ++t) { issue_qk(t, t ? kst1 : kst0); tc_commit(bar(BAR_SFULL + t)); }
                    for (int j = 0; j < T && alive; ++j) {
                        KSA_TR(0, 39);
                        take(vst0, vph0, vst1, vph1);
                        if (j + 1 < T) take(kst0, kph0, kst1, kph1);
                        // With one K and one V stage per key tile both are checked here, while the softmax warps still work on
                        // P_0: the ring runs two tiles ahead, so neither wait depends on anything this iteration does.  With
                        // four stages per key tile the ring runs hardly one tile ahead: each stage is waited for where it is used.
                        if (nsplit == 1) {
                            if (!full(vst0, vph0)) { alive = false; break; }
                            if (j + 1 < T && !full(kst0, kph0)) { alive = false; break; }
                        }
                        KSA_TR(0, 40);
                        for (int t = 0; t < nh; ++t) {
                            if (!bounded_wait(bar(BAR_PFULL + t), pf_phase[t], abort_addr, a.status, kStatusWaitPFull)) { alive = false; break; }
                            pf_phase[t] ^= 1u;
                            KSA_TR(0, 20 + t);
                            if (nsplit == 2 && !full(t ? vst1 : vst0, t ? vph1 : vph0)) { alive = false; break; }
                            tc_fence_after();
                            issue_pv(t, t ? vst1 : vst0, j > 0);
                            KSA_TR(0, 25 + t);
                            if (j == T - 1) tc_commit(bar(BAR_OFULL + t));
                            if (j + 1 < T) {
                                if (nsplit == 2) {
                                    if (!full(t ? kst1 : kst0, t ? kph1 : kph0)) { alive = false; break; }
                                    tc_fence_after();
                                }
                                issue_qk(t, t ? kst1 : kst0);
                                tc_commit(bar(BAR_SFULL + t));
                                KSA_TR(0, 30 + t);
                            }
                        }
                        if (!alive) break;
                    }
                }
            }
            // drain the tensor pipe before TMEM is released
            tc_commit(bar(BAR_DRAIN));
            bounded_wait(bar(BAR_DRAIN), 0, abort_addr + 4, a.status, kStatusWaitOFull);
        }
    }
    } else {
        setmaxnreg_inc<kRegsSoftmax>();
        // =============================== softmax warpgroups =========================
        const int t = warp >> 2;
        const int row = tid & 127;
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_sel + (uint32_t)(t * 128);
        const uint32_t tO = tmem + lane_sel + 256u + (uint32_t)(t * 128);
        const float scale_log2 = a.scale_log2;
        uint32_t sf_phase = 0, of_phase = 0;
        const int s_len = a.k + a.m;
        bool alive = true;
        // Shared-memory stages (and the Q tiles) are handed back to the producer by one thread of the
        // LAST query tile's warpgroup: tcgen05 operations of the issuing thread complete in order, so
        // its s_full for key tile j says that every product issued before it has finished reading --
        // K(j) and V(j-1) for both query tiles.  This keeps those signals out of the MMA thread's
        // instruction stream.  Every thread follows the ring position (two stages per key tile).
        int rel_stage = 0;
        auto release_next = [&]() {
            mbar_arrive_relaxed(kv_empty(rel_stage));
            if (++rel_stage == Cfg::kStages) rel_stage = 0;
        };
        for (int r = 0; alive; ++r) {
            const int idx = item_index(r);
            if (idx >= a.num_work) break;
            const WorkItem w = a.work[idx];
            if (t >= w.n_heads) { rel_stage = (rel_stage + 2 * (w.ns_tiles + (w.band_hi - w.band_lo + 1))) % Cfg::kStages; continue; }
            const bool releaser = (t == w.n_heads - 1) && (tid & 127) == 0;
            const int nsplit = ((w.head0 + w.n_heads - 1) / G != w.head0 / G) ? 2 : 1;   // ring stages per K / V tile
            const SeqInfo sq = a.seqs[w.seq];
            const int T = w.ns_tiles + (w.band_hi - w.band_lo + 1);
            const int i_raw = w.q_tile * kTileM + row;
            const bool valid = i_raw < sq.n_text;
            const int i = valid ? i_raw : sq.n_text - 1;     // padding rows mimic the last row; never stored
            const int chunk = i / a.k;
            const int far = max(0, chunk - a.C);
            const int lo_i = far * a.k;                      // Eq. 3: first visible text token
            const int cnt_i = far * a.m;                     // Eq. 3: summaries [0, cnt_i) visible
            float m_used = -INFINITY, l_run = 0.f;

            for (int j = 0; j < T; ++j) {
                bool ok = bounded_wait(bar(BAR_SFULL + t), sf_phase, abort_addr, a.status, kStatusWaitSFull);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { alive = false; break; }
                sf_phase ^= 1u;
                if (row == 0) KSA_TR(1 + t, 1);
                tc_fence_after();
                uint32_t s[128];
                {
                    uint32_t (&c0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[0]);
                    uint32_t (&c1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[32]);
                    uint32_t (&c2)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[64]);
                    uint32_t (&c3)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[96]);
                    tmem_ld32(tS + 0, c0); tmem_ld32(tS + 32, c1); tmem_ld32(tS + 64, c2); tmem_ld32(tS + 96, c3);
                }
                // the stage hand-backs ride on the latency of the loads
                if (nsplit == 2) {
                    // a stage per head (ring order K_0, K_1, V_0, V_1 per key tile): each query tile's first thread hands
                    // back its own head's stages as soon as its own scores say they were read; rel_stage stays at the
                    // item's first stage until the epilogue
                    if ((tid & 127) == 0) {
                        if (j > 0) mbar_arrive_relaxed(kv_empty((rel_stage + 4 * (j - 1) + 2 + t) % Cfg::kStages));   // V_t(j-1)
                        mbar_arrive_relaxed(kv_empty((rel_stage + 4 * j + t) % Cfg::kStages));                         // K_t(j)
                        if (releaser && j == T - 1) mbar_arrive_relaxed(bar(BAR_QEMPTY));
                    }
                } else if (releaser) {
                    if (j > 0) release_next();                   // V(j-1)
                    release_next();                              // K(j)
                    if (j == T - 1) mbar_arrive_relaxed(bar(BAR_QEMPTY));
                } else if ((tid & 127) == 0) {
                    rel_stage = (rel_stage + (j > 0 ? 2 : 1)) % Cfg::kStages;
                }
                tc_wait_ld();
                if (row == 0) KSA_TR(1 + t, 2);
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
                // row maximum, two new scores per instruction
                float mx0 = fmax3(__uint_as_float(s[0]), __uint_as_float(s[1]), __uint_as_float(s[2]));
                float mx1 = fmax3(__uint_as_float(s[3]), __uint_as_float(s[4]), __uint_as_float(s[5]));
                float mx2 = fmax3(__uint_as_float(s[6]), __uint_as_float(s[7]), __uint_as_float(s[8]));
                float mx3 = fmax3(__uint_as_float(s[9]), __uint_as_float(s[10]), __uint_as_float(s[11]));
#pragma unroll
                for (int c = 12; c < 124; c += 8) {
                    mx0 = fmax3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
                    mx3 = fmax3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
                }
                mx0 = fmax3(mx0, __uint_as_float(s[124]), __uint_as_float(s[125]));
                mx1 = fmax3(mx1, __uint_as_float(s[126]), __uint_as_float(s[127]));
                const float mx_sc = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale_log2;
                if (row == 0) KSA_TR(1 + t, 3);
                // lazy rescale: the reference max only moves when some row of the warp outgrew it
                const bool need = mx_sc > m_used + kRescaleThreshold;
                const bool need_any = __any_sync(0xffffffffu, need);
                float alpha = 1.f;
                if (need_any) {
                    const float m_new = fmaxf(m_used, mx_sc);
                    alpha = (m_new == -INFINITY) ? 1.f : ex2_approx(m_used - m_new);
                    m_used = m_new;
                    l_run *= alpha;
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                const float2 sc2 = make_float2(scale_log2, scale_log2);
                const float2 nm2 = make_float2(neg_m, neg_m);
                float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
                // probabilities of the column pair (2q, 2q+1), packed into s[q]; the scale-and-shift
                // and the row sum work on packed pairs (half the FMA-pipe instructions)
#pragma unroll
                for (int q = 0; q < 64; ++q) {
                    const float2 x = ffma2(make_float2(__uint_as_float(s[2 * q]), __uint_as_float(s[2 * q + 1])), sc2, nm2);
                    float2 pr;
                    pr.x = ex2_approx(x.x); pr.y = ex2_approx(x.y);
                    if (q & 1) lb = fadd2(lb, pr); else la = fadd2(la, pr);
                    s[q] = pack_bf16x2(pr.x, pr.y);
                }
                l_run += (la.x + la.y) + (lb.x + lb.y);
                if (row == 0) KSA_TR(1 + t, 4);
                {
                    uint32_t (&p0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[0]);
                    uint32_t (&p1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&s[32]);
                    tmem_st32(tS + 0, p0); tmem_st32(tS + 32, p1);
                }
                if (need_any && j > 0) {
                    // O_t += P V(j-1) has completed (s_full of tile j was committed after it)
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
                if (lane == 0) mbar_arrive_relaxed(bar(BAR_PFULL + t));
                if (row == 0) KSA_TR(1 + t, 6);
                if (lane == 0 && row != 0) KSA_TR(4 + warp, 6);
            }
            if (!alive) break;
            // ---- epilogue: O / l -> bf16 at the row's augmented position (Eq. 1), LSE ----
            bool ok = bounded_wait(bar(BAR_OFULL + t), of_phase, abort_addr, a.status, kStatusWaitOFull);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            of_phase ^= 1u;
            if (nsplit == 2) {
                if ((tid & 127) == 0) {
                    mbar_arrive_relaxed(kv_empty((rel_stage + 4 * (T - 1) + 2 + t) % Cfg::kStages));                   // V_t(T-1)
                    rel_stage = (rel_stage + 4 * T) % Cfg::kStages;
                }
            } else if (releaser) release_next();                 // V(T-1)
            else if ((tid & 127) == 0) rel_stage = (rel_stage + 1) % Cfg::kStages;
            tc_fence_after();
            const float inv_l = 1.f / l_run;
            const int h = w.head0 + t;
            const int64_t aug = sq.aug_off + (int64_t)(i / a.k) * s_len + (i % a.k);
            uint16_t* orow = a.out + aug * a.o_st + (int64_t)h * a.o_sh;
            const bool store = valid && ksa_out_row_ok(a, aug, h);
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
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
            if (store) a.lse[(int64_t)h * a.total_aug + aug] = (m_used + log2f(l_run)) * 0.6931471805599453f;
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
#ifdef KSA_TRACE
    if (tid == 0 && blockIdx.x < 256) { unsigned long long t_; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_)); g_cta_span[1][blockIdx.x] = t_; }
#endif
    if (warp == kProducerWarp) tmem_dealloc(tmem, 512);
}

#ifdef KSA_TRACE
extern "C" __attribute__((visibility("default"))) int ksa_debug_read_spans(void* spans)
{
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(spans, g_cta_span, sizeof(g_cta_span));
}

extern "C" __attribute__((visibility("default"))) int ksa_debug_read_trace(void* ev, void* cnt, int reset)
{
    cudaDeviceSynchronize();
    if (ev) cudaMemcpyFromSymbol(ev, g_trace, sizeof(g_trace));
    if (cnt) cudaMemcpyFromSymbol(cnt, g_trace_cnt, sizeof(g_trace_cnt));
    if (reset) { static uint32_t z[2 * kTraceRoles] = {0}; cudaMemcpyToSymbol(g_trace_cnt, z, sizeof(z)); }
    return (int)cudaGetLastError();
}
#endif

cudaError_t setup_text_tc()
{
    cudaError_t e = cudaFuncSetAttribute(ksa_text_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         TcCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(ksa_text_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TcCfg<64>::kSmemBytes);
}

cudaError_t launch_text_tc(const KernelArgs& a, const TextMaps& maps, int num_sms, cudaStream_t stream)
{
    if (a.num_work <= 0) return cudaSuccess;
    const int grid = a.num_work < num_sms ? a.num_work : num_sms;
    if (a.D == 128)
        ksa_text_tc_kernel<128><<<grid, kThreadsTc, TcCfg<128>::kSmemBytes, stream>>>(a, maps);
    else
        ksa_text_tc_kernel<64><<<grid, kThreadsTc, TcCfg<64>::kSmemBytes, stream>>>(a, maps);
    return cudaGetLastError();
}

}  // namespace ksa
