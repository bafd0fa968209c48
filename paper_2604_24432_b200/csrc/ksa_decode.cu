// Decode path: the Summary KV cache of Sec. 2.3.1 and one attention step over it.
//
// A step reads one contiguous slice of cache rows per (sequence, KV head) -- the layout of the
// cache encodes the visibility rule of Eq. 3 -- so the step is bound by HBM bandwidth: every K
// and V row of the slice is read once and serves all G query heads of the group.  The slice is
// split over several CTAs; a CTA streams 64-row K/V tiles through a 3-stage cp.async pipeline
// into (swizzled) shared memory, its four warps take 16 keys of each tile: S = Q K^T and
// O += P V with mma.sync m16n8k16 (the G <= 16 query heads are the M rows), online softmax in
// fp32.  A second small kernel merges the partial results of the splits.
#include <cuda_bf16.h>

#include <algorithm>

#include "../../include/ksa_decode.h"
#include "ksa_host.h"

namespace ksa {

constexpr int kDecTile = 64;        // cache rows per shared-memory tile
constexpr int kDecStages = 3;
constexpr int kDecThreads = 128;

struct DecodeArgs {
    uint16_t* kc; uint16_t* vc;     // caches [B][Hkv][R][D]
    int32_t* state;                 // [B][2]: text tokens cached, summaries inserted
    const uint16_t* q; const uint16_t* k_new; const uint16_t* v_new;
    uint16_t* out; float* lse;
    float* part_o; float* part_ml;  // partial results [B][Hkv][nsplit][G][D], [..][G][2]
    int32_t* status;
    int32_t B, Hq, Hkv, G, D, k, C, max_summ, R, nsplit;
    int32_t summary_step;           // 0: text step, 1: summary step
    uint32_t flags;
    float scale_log2;
};

// What a step does for one sequence, from its state (the same function decides in every kernel).
struct StepPlan { bool run; int write_row; int lo, hi; int chunk; };

__device__ __forceinline__ StepPlan plan_step(const DecodeArgs& a, int b, int* reason)
{
    StepPlan p{false, 0, 0, 0, 0};
    const int pos = a.state[2 * b], nsum = a.state[2 * b + 1];
    const int c = pos / a.k, o = pos - c * a.k;
    if (!a.summary_step) {
        if (nsum < c) { *reason = KSA_DECODE_STATUS_PENDING_SUMMARY; return p; }
        if (c >= a.max_summ) { *reason = KSA_DECODE_STATUS_FULL; return p; }
        p.run = true;
        p.chunk = c;
        p.write_row = a.k - o;
        p.lo = a.k - o;
        p.hi = 1 + a.k + min(c, a.C) * a.k + max(0, c - a.C);      // Eq. 3 as a row range
    } else {
        if (pos == 0 || o != 0 || nsum != c - 1) return p;          // not due: skipped silently
        p.run = true;
        p.chunk = c - 1;
        p.write_row = 0;
        p.lo = (a.flags & KSA_FLAG_SUMMARY_TEXT_ONLY) ? 1 : 0;
        p.hi = 1 + a.k;
    }
    return p;
}

// ---- step 1: the new token's K/V into its slot ----------------------------------------------
__global__ void __launch_bounds__(128) ksa_decode_append_kernel(DecodeArgs a)
{
    const int b = blockIdx.x;
    int reason = 0;
    const StepPlan p = plan_step(a, b, &reason);
    if (!p.run) {
        if (reason && threadIdx.x == 0) atomicCAS(a.status, 0, reason);
        return;
    }
    const int vecs = a.D / 8;
    for (int idx = threadIdx.x; idx < a.Hkv * vecs; idx += blockDim.x) {
        const int hk = idx / vecs, vv = idx - hk * vecs;
        const size_t src = ((size_t)b * a.Hkv + hk) * a.D + vv * 8;
        const size_t dst = (((size_t)b * a.Hkv + hk) * a.R + p.write_row) * a.D + vv * 8;
        *reinterpret_cast<uint4*>(a.kc + dst) = *reinterpret_cast<const uint4*>(a.k_new + src);
        *reinterpret_cast<uint4*>(a.vc + dst) = *reinterpret_cast<const uint4*>(a.v_new + src);
    }
}

// ---- helpers --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t dsmem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float fast_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- step 2: attention over a share of the slice ------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kDecThreads) ksa_decode_attn_kernel(DecodeArgs a)
{
    extern __shared__ __align__(128) uint8_t dsm[];
    constexpr int kRowB = D * 2, kTileB = kDecTile * kRowB, kStageB = 2 * kTileB, kVec = D / 8;
    const int split = blockIdx.x;
    const int b = blockIdx.y / a.Hkv, hk = blockIdx.y - b * a.Hkv;
    int reason = 0;
    const StepPlan p = plan_step(a, b, &reason);
    if (!p.run) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g0 = lane >> 2, c2 = (lane & 3) * 2;             // fragment row (query head of the group) and column pair
    const int t_lo = p.lo / kDecTile, t_hi = (p.hi + kDecTile - 1) / kDecTile;
    const int tps = (t_hi - t_lo + a.nsplit - 1) / a.nsplit;
    const int my0 = t_lo + split * tps, my1 = min(t_hi, my0 + tps);
    const uint16_t* kc = a.kc + (size_t)(b * a.Hkv + hk) * a.R * D;
    const uint16_t* vc = a.vc + (size_t)(b * a.Hkv + hk) * a.R * D;
    const uint32_t sbase = dsmem_u32(dsm);

    // Q fragments (A operand, 16 x D): rows are the query heads of the group, rows >= G are zero
    uint32_t qa[D / 16][4];
    {
        const uint16_t* q0 = a.q + ((size_t)b * a.Hq + hk * a.G + g0) * D;
        const uint16_t* q1 = q0 + 8 * D;
        const bool v0 = g0 < a.G, v1 = g0 + 8 < a.G;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            qa[kk][0] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + c2) : 0u;
            qa[kk][1] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + c2) : 0u;
            qa[kk][2] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + 8 + c2) : 0u;
            qa[kk][3] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + 8 + c2) : 0u;
        }
    }
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    // rows outside [lo, hi) are zero-filled (src-size 0): they are masked, and their V must be finite
    auto load_tile = [&](int t, int stage) {
        const uint32_t sk = sbase + stage * kStageB, sv = sk + kTileB;
        for (int idx = threadIdx.x; idx < kDecTile * kVec; idx += kDecThreads) {
            const int r = idx / kVec, c16 = idx - r * kVec;
            const int row = t * kDecTile + r;
            const bool valid = row >= p.lo && row < p.hi;
            const size_t off = valid ? ((size_t)row * D + c16 * 8) : 0;
            const uint32_t d = (uint32_t)(r * kRowB + ((c16 ^ (r & 7)) << 4));
            cp_async16(sk + d, kc + off, valid ? 16 : 0);
            cp_async16(sv + d, vc + off, valid ? 16 : 0);
        }
    };
#pragma unroll
    for (int s = 0; s < kDecStages - 1; ++s) {
        if (my0 + s < my1) load_tile(my0 + s, s);
        cp_async_commit();
    }
    const int mi = lane >> 3, r8 = lane & 7;
    for (int t = my0; t < my1; ++t) {
        if (t + kDecStages - 1 < my1) load_tile(t + kDecStages - 1, (t - my0 + kDecStages - 1) % kDecStages);
        cp_async_commit();
        cp_async_wait<kDecStages - 1>();
        __syncthreads();
        const uint32_t sk = sbase + ((t - my0) % kDecStages) * kStageB, sv = sk + kTileB;
        const int wkey0 = warp * 16;
        // S (16 heads x 16 keys of this warp) = Q K^T
        float s[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t kb[4];
            const int key = wkey0 + (mi >> 1) * 8 + r8, chunk = kk * 2 + (mi & 1);
            ldmatrix_x4(kb, sk + key * kRowB + ((chunk ^ (key & 7)) << 4));
            mma_bf16(s[0], qa[kk], kb[0], kb[1]);
            mma_bf16(s[1], qa[kk], kb[2], kb[3]);
        }
        // mask rows of the tile outside the slice, online softmax in log2 units
        const int row0 = t * kDecTile + wkey0 + c2;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int row = row0 + nt * 8 + (e & 1);
                s[nt][e] = (row >= p.lo && row < p.hi) ? s[nt][e] * a.scale_log2 : -INFINITY;
            }
        float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float al0 = (mn0 == -INFINITY) ? 1.f : fast_ex2(m0 - mn0), al1 = (mn1 == -INFINITY) ? 1.f : fast_ex2(m1 - mn1);
        const float sub0 = (mn0 == -INFINITY) ? 0.f : mn0, sub1 = (mn1 == -INFINITY) ? 0.f : mn1;
        m0 = mn0; m1 = mn1;
        float pr[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            pr[nt][0] = fast_ex2(s[nt][0] - sub0); pr[nt][1] = fast_ex2(s[nt][1] - sub0);
            pr[nt][2] = fast_ex2(s[nt][2] - sub1); pr[nt][3] = fast_ex2(s[nt][3] - sub1);
        }
        l0 = l0 * al0 + (pr[0][0] + pr[0][1]) + (pr[1][0] + pr[1][1]);
        l1 = l1 * al1 + (pr[0][2] + pr[0][3]) + (pr[1][2] + pr[1][3]);
#pragma unroll
        for (int i = 0; i < D / 8; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }
        uint32_t pa[4];
        pa[0] = pack2_bf16(pr[0][0], pr[0][1]); pa[1] = pack2_bf16(pr[0][2], pr[0][3]);
        pa[2] = pack2_bf16(pr[1][0], pr[1][1]); pa[3] = pack2_bf16(pr[1][2], pr[1][3]);
        // O += P V
#pragma unroll
        for (int n2 = 0; n2 < D / 16; ++n2) {
            uint32_t vb[4];
            const int key = wkey0 + (mi & 1) * 8 + r8, chunk = n2 * 2 + (mi >> 1);
            ldmatrix_x4_trans(vb, sv + key * kRowB + ((chunk ^ (key & 7)) << 4));
            mma_bf16(o[2 * n2], pa, vb[0], vb[1]);
            mma_bf16(o[2 * n2 + 1], pa, vb[2], vb[3]);
        }
        __syncthreads();      // the stage is refilled by the load issued in the next iteration
    }
    cp_async_wait<0>();
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    // merge the four warps through shared memory: per warp 16 rows of (m, l) and 16 x D of O
    __syncthreads();
    float* sm_o = reinterpret_cast<float*>(dsm);                       // [4][16][D]
    float* sm_ml = sm_o + 4 * 16 * D;                                  // [4][16][2]
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
        float* r0 = sm_o + ((warp * 16 + g0) * D) + i * 8 + c2;
        float* r1 = r0 + 8 * D;
        r0[0] = o[i][0]; r0[1] = o[i][1]; r1[0] = o[i][2]; r1[1] = o[i][3];
    }
    if ((lane & 3) == 0) {
        sm_ml[(warp * 16 + g0) * 2] = m0; sm_ml[(warp * 16 + g0) * 2 + 1] = l0;
        sm_ml[(warp * 16 + g0 + 8) * 2] = m1; sm_ml[(warp * 16 + g0 + 8) * 2 + 1] = l1;
    }
    __syncthreads();
    const size_t pbase = ((size_t)(b * a.Hkv + hk) * a.nsplit + split) * a.G;
    for (int idx = threadIdx.x; idx < a.G * D; idx += kDecThreads) {
        const int g = idx / D, d = idx - g * D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, sm_ml[(w * 16 + g) * 2]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float mw = sm_ml[(w * 16 + g) * 2];
            const float f = (mw == -INFINITY) ? 0.f : fast_ex2(mw - M);
            L += sm_ml[(w * 16 + g) * 2 + 1] * f;
            acc += sm_o[(w * 16 + g) * D + d] * f;
        }
        a.part_o[(pbase + g) * D + d] = acc;
        if (d == 0) { a.part_ml[(pbase + g) * 2] = M; a.part_ml[(pbase + g) * 2 + 1] = L; }
    }
}

// ---- step 3: merge the splits, write out / lse ---------------------------------------------------
__global__ void __launch_bounds__(128) ksa_decode_merge_kernel(DecodeArgs a)
{
    const int b = blockIdx.x / a.Hq, h = blockIdx.x - b * a.Hq;
    int reason = 0;
    const StepPlan p = plan_step(a, b, &reason);
    if (!p.run) return;
    const int hk = h / a.G, g = h - hk * a.G;
    const size_t pbase = (size_t)(b * a.Hkv + hk) * a.nsplit;
    float M = -INFINITY;
    for (int s = 0; s < a.nsplit; ++s) M = fmaxf(M, a.part_ml[((pbase + s) * a.G + g) * 2]);
    float L = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
        const float ms = a.part_ml[((pbase + s) * a.G + g) * 2];
        L += (ms == -INFINITY) ? 0.f : a.part_ml[((pbase + s) * a.G + g) * 2 + 1] * fast_ex2(ms - M);
    }
    const float inv = 1.f / L;
    for (int d = threadIdx.x; d < a.D; d += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < a.nsplit; ++s) {
            const float ms = a.part_ml[((pbase + s) * a.G + g) * 2];
            if (ms != -INFINITY) acc += a.part_o[((pbase + s) * a.G + g) * a.D + d] * fast_ex2(ms - M);
        }
        a.out[((size_t)b * a.Hq + h) * a.D + d] = __bfloat16_as_ushort(__float2bfloat16_rn(acc * inv));
    }
    if (threadIdx.x == 0) a.lse[(size_t)b * a.Hq + h] = (M + log2f(L)) * 0.6931471805599453f;
}

// ---- step 4: advance the state; the summary step also recycles the chunk -------------------------
// One CTA per sequence, so that the state is written only after everything that reads it is done.
__global__ void __launch_bounds__(128) ksa_decode_commit_kernel(DecodeArgs a)
{
    const int b = blockIdx.x;
    int reason = 0;
    const StepPlan p = plan_step(a, b, &reason);
    if (!p.run) return;
    if (a.summary_step) {
        const int vecs = a.D / 8;
        const int slot_row = 1 + a.k + (a.C > 0 ? (p.chunk % a.C) * a.k : 0);
        const int summ_row = 1 + a.k + a.C * a.k + p.chunk;
        // rows to copy per KV head: the k chunk rows into the ring (if there is a ring), the scratch row into the buffer
        const int nrows = (a.C > 0 ? a.k : 0) + 1;
        for (int idx = threadIdx.x; idx < a.Hkv * nrows * vecs; idx += blockDim.x) {
            const int hk = idx / (nrows * vecs);
            const int rem = idx - hk * nrows * vecs;
            const int rr = rem / vecs, vv = rem - rr * vecs;
            const bool is_summ = (rr == nrows - 1);
            const int src_row = is_summ ? 0 : 1 + rr;
            const int dst_row = is_summ ? summ_row : slot_row + rr;
            const size_t base = (size_t)(b * a.Hkv + hk) * a.R;
            const size_t so = (base + src_row) * a.D + vv * 8, dd = (base + dst_row) * a.D + vv * 8;
            *reinterpret_cast<uint4*>(a.kc + dd) = *reinterpret_cast<const uint4*>(a.kc + so);
            *reinterpret_cast<uint4*>(a.vc + dd) = *reinterpret_cast<const uint4*>(a.vc + so);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (a.summary_step) a.state[2 * b + 1] += 1; else a.state[2 * b] += 1;
    }
}

// ---- cache construction from a prefill ----------------------------------------------------------
struct FillArgs {
    uint16_t* kc; uint16_t* vc; int32_t* state;
    const uint16_t* k; const uint16_t* v;
    const int64_t* aug_off; const int32_t* n_text;     // per sequence (device)
    int64_t k_st, k_sh, v_st, v_sh;
    int32_t B, Hkv, D, kk, C, R, max_summ;
};

// One thread per 16-byte vector of a cache row: finds the augmented row (Eq. 1) the cache row
// holds after n_text tokens were decoded one by one, or nothing.
__global__ void __launch_bounds__(256) ksa_cache_fill_kernel(FillArgs a)
{
    const int b = blockIdx.z, hk = blockIdx.y;
    const int vecs = a.D / 8;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)a.R * vecs) return;
    const int r = (int)(idx / vecs), vv = (int)(idx - (int64_t)r * vecs);
    const int n = a.n_text[b], k = a.kk, s = k + 1;
    const int J = min(n / k, a.max_summ);              // full chunks = summaries inserted
    if (idx == 0 && hk == 0) { a.state[2 * b] = n; a.state[2 * b + 1] = J; }
    int64_t text = -1, aug = -1;
    if (r >= 1 && r <= k) {                            // Current Chunk: token o at row k - o
        const int o = k - r;
        if (o < n - J * k && n / k == J) text = (int64_t)J * k + o;
    } else if (r > k && r < 1 + k + a.C * k) {         // ring: chunk c in slot c mod C, same row order as Current Chunk
        const int slot = (r - 1 - k) / k, o = k - 1 - ((r - 1 - k) % k);
        if (J > 0) {
            const int c = J - 1 - ((((J - 1 - slot) % a.C) + a.C) % a.C);    // newest chunk in this slot
            if (c >= 0 && c >= J - a.C) text = (int64_t)c * k + o;
        }
    } else if (r >= 1 + k + a.C * k) {                 // Summary Token Buffer
        const int j = r - (1 + k + a.C * k);
        if (j < J) aug = (int64_t)j * s + k;
    }
    if (text >= 0) aug = (text / k) * s + (text % k);
    if (aug < 0) return;
    const size_t dst = ((size_t)(b * a.Hkv + hk) * a.R + r) * a.D + vv * 8;
    const int64_t row = a.aug_off[b] + aug;
    *reinterpret_cast<uint4*>(a.kc + dst) = *reinterpret_cast<const uint4*>(a.k + row * a.k_st + (int64_t)hk * a.k_sh + vv * 8);
    *reinterpret_cast<uint4*>(a.vc + dst) = *reinterpret_cast<const uint4*>(a.v + row * a.v_st + (int64_t)hk * a.v_sh + vv * 8);
}

__global__ void ksa_cache_reset_kernel(int32_t* state, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) state[i] = 0;
}

}  // namespace ksa

// =================================================================================================
// C ABI
// =================================================================================================
using namespace ksa;

#define KSA_API extern "C" __attribute__((visibility("default")))

static int validate_cache(const ksa_cache_params* p)
{
    if (!p || p->struct_size != (int32_t)sizeof(ksa_cache_params)) return KSA_ERR_INVALID_ARG;
    if (p->batch < 1 || p->chunk_len < 1 || p->window_chunks < 0 || p->max_summaries < 1) return KSA_ERR_INVALID_ARG;
    if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0) return KSA_ERR_INVALID_ARG;
    if (!(p->softmax_scale > 0.f) || p->softmax_scale > 1e30f) return KSA_ERR_INVALID_ARG;
    if (p->flags & ~KSA_FLAG_SUMMARY_TEXT_ONLY) return KSA_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return KSA_ERR_UNSUPPORTED;
    if (p->num_q_heads / p->num_kv_heads > 16) return KSA_ERR_UNSUPPORTED;
    const int64_t rows = 1 + (int64_t)p->chunk_len * (1 + (int64_t)p->window_chunks) + p->max_summaries;
    if (rows > (1ll << 30) || (int64_t)p->batch * p->num_kv_heads > 65535) return KSA_ERR_UNSUPPORTED;
    return KSA_OK;
}

// Splits of a slice: the grid (splits x batch x KV heads) should fill whole waves of the 2 x 148
// resident CTAs (two per SM) -- the smallest split count of at least two waves that wastes less
// than 5 % of the last wave, or the most efficient one up to 32.
static int decode_splits(const ksa_cache_params* p)
{
    const int64_t units = (int64_t)p->batch * p->num_kv_heads, slots = 2 * 148;
    int best = 1;
    double best_eff = 0.0;
    for (int n = 1; n <= 32; ++n) {
        const int64_t total = units * n;
        if (total < 2 * slots && n < 32) continue;
        const double eff = (double)total / (double)(((total + slots - 1) / slots) * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = n; }
        if (eff >= 0.95) break;
    }
    return best;
}

KSA_API int64_t ksa_cache_rows(const ksa_cache_params* p)
{
    if (validate_cache(p) != KSA_OK) return -1;
    return 1 + (int64_t)p->chunk_len * (1 + (int64_t)p->window_chunks) + p->max_summaries;
}

KSA_API int ksa_cache_bytes(const ksa_cache_params* p, size_t* cache_bytes, size_t* state_bytes, size_t* workspace_bytes)
{
    int rc = validate_cache(p);
    if (rc != KSA_OK) return rc;
    const size_t rows = (size_t)ksa_cache_rows(p);
    if (cache_bytes) *cache_bytes = (size_t)p->batch * p->num_kv_heads * rows * p->head_dim * 2;
    if (state_bytes) *state_bytes = (size_t)p->batch * 2 * sizeof(int32_t);
    if (workspace_bytes)
        *workspace_bytes = (size_t)p->batch * p->num_q_heads * decode_splits(p) * (p->head_dim + 2) * sizeof(float);
    return KSA_OK;
}

KSA_API int ksa_cache_slice(const ksa_cache_params* p, int64_t text_tokens_before, int is_summary, int64_t* row_lo, int64_t* row_hi)
{
    int rc = validate_cache(p);
    if (rc != KSA_OK) return rc;
    if (!row_lo || !row_hi || text_tokens_before < 0) return KSA_ERR_INVALID_ARG;
    const int64_t k = p->chunk_len, C = p->window_chunks;
    if (is_summary) {
        if (text_tokens_before == 0 || text_tokens_before % k != 0) return KSA_ERR_INVALID_ARG;
        *row_lo = (p->flags & KSA_FLAG_SUMMARY_TEXT_ONLY) ? 1 : 0;
        *row_hi = 1 + k;
    } else {
        const int64_t c = text_tokens_before / k, o = text_tokens_before % k;
        *row_lo = k - o;
        *row_hi = 1 + k + std::min(c, C) * k + std::max<int64_t>(0, c - C);
    }
    return KSA_OK;
}

KSA_API int ksa_cache_reset(ksa_ctx* ctx, int32_t* state, const ksa_cache_params* p, void* cuda_stream)
{
    int rc = validate_cache(p);
    if (rc != KSA_OK) return rc;
    if (!ctx || !state) return KSA_ERR_INVALID_ARG;
    const int n = p->batch * 2;
    ksa_cache_reset_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)cuda_stream>>>(state, n);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    ksa_ctx_add_launches(ctx, 1);
    return KSA_OK;
}

KSA_API int ksa_cache_fill_from_prefill(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* k, const void* v,
                                        const ksa_params* prefill, const ksa_cache_params* p, void* cuda_stream)
{
    int rc = validate_cache(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate(prefill)) != KSA_OK) return rc;
    if ((rc = validate_strides(prefill)) != KSA_OK) return rc;
    if (!ctx || !kcache || !vcache || !state || !k || !v) return KSA_ERR_INVALID_ARG;
    if (prefill->summaries_per_chunk != 1 || prefill->chunk_len != p->chunk_len || prefill->window_chunks != p->window_chunks ||
        prefill->num_kv_heads != p->num_kv_heads || prefill->head_dim != p->head_dim || prefill->num_seqs != p->batch)
        return KSA_ERR_INVALID_ARG;
    const int B = p->batch;
    std::vector<int64_t> aug(B);
    std::vector<int32_t> nt(B);
    int64_t off = 0;
    for (int b = 0; b < B; ++b) {
        nt[b] = prefill->cu_text_lens[b + 1] - prefill->cu_text_lens[b];
        if (nt[b] / p->chunk_len > p->max_summaries) return KSA_ERR_INVALID_ARG;
        aug[b] = off;
        off += ksa_aug_len(nt[b], p->chunk_len, 1);
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the two small per-sequence tables live in stream-ordered scratch for the duration of the kernel
    char* tab = nullptr;
    cudaError_t e = cudaMallocAsync((void**)&tab, (size_t)B * 12, stream);
    if (e != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    e = cudaMemcpyAsync(tab, aug.data(), (size_t)B * 8, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(tab + (size_t)B * 8, nt.data(), (size_t)B * 4, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) { cudaFreeAsync(tab, stream); return ksa_ctx_cuda_fail(ctx, (int)e); }
    FillArgs a{};
    a.kc = (uint16_t*)kcache; a.vc = (uint16_t*)vcache; a.state = state;
    a.k = (const uint16_t*)k; a.v = (const uint16_t*)v;
    a.aug_off = (const int64_t*)tab; a.n_text = (const int32_t*)(tab + (size_t)B * 8);
    a.k_st = prefill->k_stride_tok; a.k_sh = prefill->k_stride_head; a.v_st = prefill->v_stride_tok; a.v_sh = prefill->v_stride_head;
    a.B = B; a.Hkv = p->num_kv_heads; a.D = p->head_dim; a.kk = p->chunk_len; a.C = p->window_chunks;
    a.R = (int32_t)ksa_cache_rows(p); a.max_summ = p->max_summaries;
    const int64_t vec_total = (int64_t)a.R * (a.D / 8);
    dim3 grid((unsigned)((vec_total + 255) / 256), (unsigned)a.Hkv, (unsigned)B);
    ksa_cache_fill_kernel<<<grid, 256, 0, stream>>>(a);
    e = cudaGetLastError();
    cudaFreeAsync(tab, stream);
    if (e != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    // the host tables were pageable: make sure the copies have left them before they go out of scope
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    ksa_ctx_add_launches(ctx, 1);
    return KSA_OK;
}

static int decode_step(ksa_ctx* ctx, int summary_step, void* kcache, void* vcache, int32_t* state, const void* q,
                       const void* k_new, const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                       const ksa_cache_params* p, void* cuda_stream)
{
    int rc = validate_cache(p);
    if (rc != KSA_OK) return rc;
    if (!ctx || !kcache || !vcache || !state || !q || !k_new || !v_new || !out || !lse) return KSA_ERR_INVALID_ARG;
    const uintptr_t ptrs[7] = {(uintptr_t)kcache, (uintptr_t)vcache, (uintptr_t)q, (uintptr_t)k_new, (uintptr_t)v_new, (uintptr_t)out, (uintptr_t)workspace};
    for (int i = 0; i < 7; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    size_t need = 0;
    ksa_cache_bytes(p, nullptr, nullptr, &need);
    if (!workspace || workspace_bytes < need) return KSA_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    DecodeArgs a{};
    a.kc = (uint16_t*)kcache; a.vc = (uint16_t*)vcache; a.state = state;
    a.q = (const uint16_t*)q; a.k_new = (const uint16_t*)k_new; a.v_new = (const uint16_t*)v_new;
    a.out = (uint16_t*)out; a.lse = lse;
    a.B = p->batch; a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.G = a.Hq / a.Hkv; a.D = p->head_dim;
    a.k = p->chunk_len; a.C = p->window_chunks; a.max_summ = p->max_summaries; a.R = (int32_t)ksa_cache_rows(p);
    a.nsplit = decode_splits(p);
    a.part_o = (float*)workspace;
    a.part_ml = a.part_o + (size_t)a.B * a.Hq * a.nsplit * a.D;
    a.status = ksa_ctx_status_word(ctx);
    a.summary_step = summary_step;
    a.flags = p->flags;
    a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
    bool& attr_done = *ksa_ctx_decode_ready(ctx);         // per context: the opt-in is a per-device setting
    const int smem = kDecStages * 2 * kDecTile * a.D * 2;
    cudaError_t e;
    if (!attr_done) {
        if ((e = cudaFuncSetAttribute(ksa_decode_attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecStages * 2 * kDecTile * 128 * 2)) != cudaSuccess)
            return ksa_ctx_cuda_fail(ctx, (int)e);
        if ((e = cudaFuncSetAttribute(ksa_decode_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecStages * 2 * kDecTile * 64 * 2)) != cudaSuccess)
            return ksa_ctx_cuda_fail(ctx, (int)e);
        attr_done = true;
    }
    ksa_decode_append_kernel<<<a.B, 128, 0, stream>>>(a);
    dim3 grid((unsigned)a.nsplit, (unsigned)(a.B * a.Hkv), 1);
    if (a.D == 128) ksa_decode_attn_kernel<128><<<grid, kDecThreads, smem, stream>>>(a);
    else            ksa_decode_attn_kernel<64><<<grid, kDecThreads, smem, stream>>>(a);
    ksa_decode_merge_kernel<<<a.B * a.Hq, 128, 0, stream>>>(a);
    ksa_decode_commit_kernel<<<a.B, 128, 0, stream>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    ksa_ctx_add_launches(ctx, 4);
    return KSA_OK;
}

KSA_API int ksa_decode_text(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* q, const void* k_new,
                            const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                            const ksa_cache_params* p, void* cuda_stream)
{
    return decode_step(ctx, 0, kcache, vcache, state, q, k_new, v_new, out, lse, workspace, workspace_bytes, p, cuda_stream);
}

KSA_API int ksa_decode_summary(ksa_ctx* ctx, void* kcache, void* vcache, int32_t* state, const void* q, const void* k_new,
                               const void* v_new, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               const ksa_cache_params* p, void* cuda_stream)
{
    return decode_step(ctx, 1, kcache, vcache, state, q, k_new, v_new, out, lse, workspace, workspace_bytes, p, cuda_stream);
}
