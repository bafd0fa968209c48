// Q/K/V preparation upstream of the attention: position ids (Sec. 2.2.1), interpolation of the two projections at
// summary positions (Sec. 4.1) and the rotary embedding, one pass, HBM-bound.
//
// A thread owns one augmented row and one 8-element slice d0 .. d0 + 7 of the first half of a head together
// with its partners d0 + D/2 ..: it works out the row's position id and the eight angles once (the product
// position x frequency and its reduction to [-pi, pi] in double precision: a position of 10^5 times a frequency
// near 1 has no fraction left in fp32; the frequencies come from the host as doubles) and then walks the
// heads of q, k and v with 16-byte loads and stores.  32 rows x D/16 slices per block, one sequence per grid.y.
#include <cuda_runtime.h>

#include "ksa_launch.h"

namespace ksa {

// heads per batch (the loads of a batch are issued before its stores) and resident blocks per SM the register
// budget is held to; measured at 128k: (1, 4) 0.543 ms, (2, 3) 0.542, (2, 4) 0.625, (3, 3) 0.605
constexpr int kPrepBatch = 1, kPrepMinBlocks = 4;

__device__ __forceinline__ float2 bf2_to_f2(uint32_t w) { return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)); }
__device__ __forceinline__ uint32_t f2_to_bf2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(256, kPrepMinBlocks) ksa_prep_kernel(PrepArgs a)
{
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int slices = a.D / 16;                                  // 8-element slices of half a head
    const int rows_per_block = 256 / slices;
    const int slice = threadIdx.x % slices;
    const int64_t row_in_seq = (int64_t)blockIdx.x * rows_per_block + threadIdx.x / slices;
    const int64_t aug_len = (int64_t)sq.n_text + sq.n_summ;
    if (row_in_seq >= aug_len) return;
    // ---- Eq. 1: which token is this, and its position id (Sec. 2.2.1) ------------------------------
    const int s_len = a.k + a.m;
    const int64_t full = (int64_t)sq.n_chunks * s_len;            // rows of the full chunks
    int pos;
    int64_t summ_index = -1;                                      // row of the summary projections, if a summary token
    int64_t stream_row;                                           // row of the packed text or summary stream (stream mode)
    if (row_in_seq < full) {
        const int j = (int)(row_in_seq / s_len), off = (int)(row_in_seq - (int64_t)j * s_len);
        if (off < a.k) { pos = j * a.k + off; stream_row = (int64_t)sq.text_off + pos; }
        else {
            pos = (j + 1) * a.k - 1;
            summ_index = (int64_t)sq.summ_base + (int64_t)j * a.m + (off - a.k);
            stream_row = (int64_t)sq.summ_off + (int64_t)j * a.m + (off - a.k);
        }
    } else {
        pos = sq.n_chunks * a.k + (int)(row_in_seq - full);       // text tokens after the last full chunk
        stream_row = (int64_t)sq.text_off + pos;
    }
    const bool is_summ = summ_index >= 0;
    const int64_t row = sq.aug_off + row_in_seq;
    // ---- the eight angles of this slice ---------------------------------------------------------
    const int d0 = slice * 8;
    float cs[8], sn[8];
    if (a.rope) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            // angle and its reduction to [-pi, pi] in double (a handful of fp64 operations), sine and cosine in fp32
            const double ang = (double)pos * a.inv_freq[d0 + e];
            const double turns = rint(ang * 0.15915494309189535);        // 1 / (2 pi)
            const float r = (float)fma(-turns, 6.283185307179586, ang);
            sincosf(r, &sn[e], &cs[e]);
        }
    }
    const bool blend = summ_index >= 0 && a.lambda != 0.f;
    const float lam = a.lambda, mal = 1.f - a.lambda;
    // ---- the heads of q, k, v, kPrepBatch at a time (the loads of a batch before its stores: more bytes in flight) ----
    const int heads = a.Hq + 2 * a.Hkv;
    constexpr int kBatch = kPrepBatch;
    for (int hb = 0; hb < heads; hb += kBatch) {
        uint4 lo[kBatch], hi[kBatch], slo[kBatch], shi[kBatch];
        uint16_t* outp[kBatch];
        bool rotate[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int hh = hb + u;
            outp[u] = nullptr; rotate[u] = false;
            if (hh >= heads) continue;
            const int which = hh < a.Hq ? 0 : (hh < a.Hq + a.Hkv ? 1 : 2);
            const int h = which == 0 ? hh : (which == 1 ? hh - a.Hq : hh - a.Hq - a.Hkv);
            const uint16_t* mainp; const uint16_t* summp; int H;
            if (which == 0)      { mainp = a.qm + row * a.q_st + (int64_t)h * a.q_sh; outp[u] = a.qo + row * a.q_st + (int64_t)h * a.q_sh; summp = a.qs; H = a.Hq; }
            else if (which == 1) { mainp = a.km + row * a.k_st + (int64_t)h * a.k_sh; outp[u] = a.ko + row * a.k_st + (int64_t)h * a.k_sh; summp = a.ks; H = a.Hkv; }
            else                 { mainp = a.vm + row * a.v_st + (int64_t)h * a.v_sh; outp[u] = a.vo + row * a.v_st + (int64_t)h * a.v_sh; summp = a.vs; H = a.Hkv; }
            if (a.to_streams) {                                   // head-major streams: [head][row][D]
                if (!is_summ) outp[u] = (which == 0 ? a.qt : (which == 1 ? a.kt : a.vt)) + ((int64_t)h * a.text_rows + stream_row) * a.D;
                else          outp[u] = (which == 0 ? a.qs_out : (which == 1 ? a.ks_out : a.vs_out)) + ((int64_t)h * a.summ_rows + stream_row) * a.D;
            }
            rotate[u] = a.rope && which != 2;
            lo[u] = *reinterpret_cast<const uint4*>(mainp + d0);
            hi[u] = *reinterpret_cast<const uint4*>(mainp + a.D / 2 + d0);
            if (blend) {
                const uint16_t* sp = summp + (summ_index * H + h) * a.D;
                slo[u] = *reinterpret_cast<const uint4*>(sp + d0);
                shi[u] = *reinterpret_cast<const uint4*>(sp + a.D / 2 + d0);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (outp[u] == nullptr) continue;
            const uint32_t lw[4] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w}, hw[4] = {hi[u].x, hi[u].y, hi[u].z, hi[u].w};
            float xl[8], xh[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 l2 = bf2_to_f2(lw[e]), h2 = bf2_to_f2(hw[e]);
                xl[2 * e] = l2.x; xl[2 * e + 1] = l2.y; xh[2 * e] = h2.x; xh[2 * e + 1] = h2.y;
            }
            if (blend) {                                          // x = lambda x_s + (1 - lambda) x_main
                const uint32_t slw[4] = {slo[u].x, slo[u].y, slo[u].z, slo[u].w}, shw[4] = {shi[u].x, shi[u].y, shi[u].z, shi[u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 l2 = bf2_to_f2(slw[e]), h2 = bf2_to_f2(shw[e]);
                    xl[2 * e] = fmaf(lam, l2.x, mal * xl[2 * e]);     xl[2 * e + 1] = fmaf(lam, l2.y, mal * xl[2 * e + 1]);
                    xh[2 * e] = fmaf(lam, h2.x, mal * xh[2 * e]);     xh[2 * e + 1] = fmaf(lam, h2.y, mal * xh[2 * e + 1]);
                }
            }
            if (rotate[u]) {                                      // the pair (d, d + D/2) turns by its angle
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float l = xl[e], hgh = xh[e];
                    xl[e] = l * cs[e] - hgh * sn[e];
                    xh[e] = hgh * cs[e] + l * sn[e];
                }
            }
            uint4 olo, ohi;
            olo.x = f2_to_bf2(xl[0], xl[1]); olo.y = f2_to_bf2(xl[2], xl[3]); olo.z = f2_to_bf2(xl[4], xl[5]); olo.w = f2_to_bf2(xl[6], xl[7]);
            ohi.x = f2_to_bf2(xh[0], xh[1]); ohi.y = f2_to_bf2(xh[2], xh[3]); ohi.z = f2_to_bf2(xh[4], xh[5]); ohi.w = f2_to_bf2(xh[6], xh[7]);
            *reinterpret_cast<uint4*>(outp[u] + d0) = olo;
            *reinterpret_cast<uint4*>(outp[u] + a.D / 2 + d0) = ohi;
        }
    }
}

// Padding rows of the streams: rows [n_text, text_pad) of every sequence's part of qt, kt, vt and rows
// [n_summ, summ_pad) of ks, vs, qs.  One block per (sequence, stream); at most 127 rows each.
__global__ void __launch_bounds__(256) ksa_zero_stream_pads_kernel(PrepArgs a)
{
    const SeqInfo sq = a.seqs[blockIdx.y];
    const int which = blockIdx.x;                                  // 0 qt, 1 kt, 2 vt, 3 ks_out, 4 vs_out, 5 qs_out
    const bool text = which < 3;
    uint16_t* base = which == 0 ? a.qt : which == 1 ? a.kt : which == 2 ? a.vt : which == 3 ? a.ks_out : which == 4 ? a.vs_out : a.qs_out;
    const int H = (which == 0 || which == 5) ? a.Hq : a.Hkv;
    const int64_t rows = text ? a.text_rows : a.summ_rows;
    const int64_t r0 = text ? (int64_t)sq.text_off + sq.n_text : (int64_t)sq.summ_off + sq.n_summ;
    const int64_t r1 = text ? (int64_t)sq.text_off + sq.text_pad : (int64_t)sq.summ_off + sq.summ_pad;
    const int vecs = a.D / 8;
    const int64_t total = (r1 - r0) * H * vecs;
    for (int64_t idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int vec = (int)(idx % vecs);
        const int64_t t = idx / vecs;
        const int h = (int)(t % H);
        const int64_t row = r0 + t / H;
        *reinterpret_cast<uint4*>(base + ((int64_t)h * rows + row) * a.D + vec * 8) = make_uint4(0u, 0u, 0u, 0u);
    }
}

cudaError_t launch_zero_stream_pads(const PrepArgs& a, int num_seqs, cudaStream_t stream)
{
    dim3 grid(6u, (unsigned)num_seqs, 1u);
    ksa_zero_stream_pads_kernel<<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_prep(const PrepArgs& a, int64_t max_aug_len, int num_seqs, cudaStream_t stream)
{
    if (max_aug_len <= 0) return cudaSuccess;
    const int rows_per_block = 256 / (a.D / 16);
    dim3 grid((unsigned)((max_aug_len + rows_per_block - 1) / rows_per_block), (unsigned)num_seqs, 1);
    ksa_prep_kernel<<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace ksa
