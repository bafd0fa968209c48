// C ABI of the KSA forward library: argument validation, sequence layout (Eq. 1), the
// block-sparse tile schedule (Eq. 3 at tile granularity) and the kernel launches.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/ksa.h"
#include "../../include/ksa_prep.h"
#include "ksa_host.h"
#include "ksa_bwd.h"
#include "ksa_launch.h"

using namespace ksa;

static_assert(sizeof(ksa_params) == 120, "ksa_params ABI");
static_assert(sizeof(ksa_tile_rec) == 32, "ksa_tile_rec ABI");

// ---------------------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);


struct ksa_ctx {
    int device = -1;
    int num_sms = 0;
    int last_cuda_error = 0;
    int64_t launches = 0;
    EncodeTiledFn encode = nullptr;
    HostSchedule sched;               // cached schedule (one entry)
    SeqInfo* d_seqs = nullptr;  size_t d_seqs_cap = 0;
    WorkItem* d_work = nullptr; size_t d_work_cap = 0;
    int32_t* d_status = nullptr;
    bool timing = false;
    bool timing_valid = false;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    bool tc_ready = false;
    bool pair_ready = false;          // CTA-pair text kernel set up on this device
    int max_pairs = 0;                // clusters of two CTAs the device runs at once
    bool bwd_ready = false, bwd_tc_ready = false, decode_ready = false;
    // host entry point: copy streams and per-chunk events of its upload / compute / download pipeline
    cudaStream_t s_in = nullptr, s_out = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done;
    cudaEvent_t ev_start = nullptr;
};

static int cuda_fail(ksa_ctx* ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda_error = (int)e;
    return KSA_ERR_CUDA;
}

int32_t* ksa_ctx_status_word(ksa_ctx* ctx) { return ctx->d_status; }
int ksa_ctx_num_sms(const ksa_ctx* ctx) { return ctx->num_sms; }
void ksa_ctx_add_launches(ksa_ctx* ctx, int n) { ctx->launches += n; }
int ksa_ctx_cuda_fail(ksa_ctx* ctx, int cuda_error) { return cuda_fail(ctx, (cudaError_t)cuda_error); }
bool* ksa_ctx_decode_ready(ksa_ctx* ctx) { return &ctx->decode_ready; }

// ---------------------------------------------------------------------------------------
// validation and layout
// ---------------------------------------------------------------------------------------
int validate(const ksa_params* p)
{
    if (!p || p->struct_size != (int32_t)sizeof(ksa_params)) return KSA_ERR_INVALID_ARG;
    if (p->num_seqs < 1 || !p->cu_text_lens) return KSA_ERR_INVALID_ARG;
    if (p->chunk_len < 1 || p->summaries_per_chunk < 0 || p->window_chunks < 0) return KSA_ERR_INVALID_ARG;
    if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0)
        return KSA_ERR_INVALID_ARG;
    if (p->reserved != 0) return KSA_ERR_INVALID_ARG;
    if (p->flags & ~(KSA_FLAG_SUMMARY_TEXT_ONLY | KSA_FLAG_REFERENCE_KERNEL | KSA_FLAG_SINGLE_CTA_KERNEL | KSA_FLAG_CTA_PAIR_KERNEL |
                     KSA_FLAG_BWD_MMA_SYNC_KERNELS)) return KSA_ERR_INVALID_ARG;
    if (!(p->softmax_scale > 0.f) || !std::isfinite(p->softmax_scale)) return KSA_ERR_INVALID_ARG;
    if (p->cu_text_lens[0] != 0) return KSA_ERR_INVALID_ARG;
    for (int b = 0; b < p->num_seqs; ++b)
        if (p->cu_text_lens[b + 1] <= p->cu_text_lens[b]) return KSA_ERR_INVALID_ARG;  // empty or non-monotone
    if (p->head_dim != 64 && p->head_dim != 128) return KSA_ERR_UNSUPPORTED;
    if (p->num_q_heads > 1024 || p->chunk_len > (1 << 20) || p->summaries_per_chunk > (1 << 20))
        return KSA_ERR_UNSUPPORTED;
    if (p->num_seqs > 65535) return KSA_ERR_UNSUPPORTED;          // sequences are a grid dimension of the helper kernels
    // padded stream rows must fit comfortably in int32
    int64_t n_total = p->cu_text_lens[p->num_seqs];
    if (n_total + (int64_t)p->num_seqs * kTileM > (1ll << 30)) return KSA_ERR_UNSUPPORTED;
    if (n_total / p->chunk_len * (int64_t)p->summaries_per_chunk + (int64_t)p->num_seqs * kTileN > (1ll << 30))
        return KSA_ERR_UNSUPPORTED;
    return KSA_OK;
}

int validate_strides(const ksa_params* p)
{
    const int64_t st[8] = {p->q_stride_tok, p->q_stride_head, p->k_stride_tok, p->k_stride_head,
                           p->v_stride_tok, p->v_stride_head, p->o_stride_tok, p->o_stride_head};
    for (int i = 0; i < 8; ++i)
        if (st[i] < p->head_dim || (st[i] % 8) != 0) return KSA_ERR_INVALID_ARG;
    return KSA_OK;
}

static inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// The text kernel can read its tiles straight from the caller's interleaved tensors -- no packed
// streams, no workspace -- when a 128-row tile is a whole number of chunks in both views and every
// sequence is a whole number of chunks (the paper's assumption, Sec. 2.2.1), so that sequence b
// starts at chunk aug_off_b / (k + m) of a regular [chunk, k + m] grid.  Padding rows of a partial
// tile then hold rows of the following sequence (or zeros past the end); they are masked.
bool direct_ok(const ksa_params* p)
{
    if (p->flags & KSA_FLAG_REFERENCE_KERNEL) return false;
    const int k = p->chunk_len, m = p->summaries_per_chunk;
    if (kTileM % k != 0 || (m > 0 && kTileN % m != 0)) return false;
    for (int b = 0; b < p->num_seqs; ++b)
        if ((p->cu_text_lens[b + 1] - p->cu_text_lens[b]) % k != 0) return false;
    return true;
}

void build_layout(const ksa_params* p, HostSchedule& hs)
{
    const int k = p->chunk_len, m = p->summaries_per_chunk;
    hs.seqs.resize(p->num_seqs);
    int64_t aug = 0, trow = 0, srow = 0, summ_before = 0;
    hs.max_text_pad = hs.max_summ_pad = hs.max_n_summ = 0;
    for (int b = 0; b < p->num_seqs; ++b) {
        SeqInfo& s = hs.seqs[b];
        std::memset(&s, 0, sizeof s);
        s.n_text = p->cu_text_lens[b + 1] - p->cu_text_lens[b];
        s.n_chunks = s.n_text / k;                        // only full chunks carry summaries
        s.n_summ = s.n_chunks * m;
        s.aug_off = aug;
        s.chunk0 = (int32_t)(aug / (k + m));
        s.summ_base = (int32_t)summ_before;
        summ_before += s.n_summ;
        s.text_off = (int32_t)trow;
        s.summ_off = (int32_t)srow;
        s.text_pad = (int32_t)round_up(s.n_text, kTileM);
        s.summ_pad = (int32_t)round_up(s.n_summ, kTileN);
        aug += (int64_t)s.n_text + s.n_summ;              // Eq. 1: L = n + floor(n/k) m
        trow += s.text_pad;
        srow += s.summ_pad;
        hs.max_text_pad = std::max(hs.max_text_pad, s.text_pad);
        hs.max_summ_pad = std::max(hs.max_summ_pad, s.summ_pad);
        hs.max_n_summ = std::max(hs.max_n_summ, s.n_summ);
    }
    hs.total_aug = aug;
    hs.text_rows = trow;
    hs.summ_rows = std::max<int64_t>(srow, kTileN);       // keep the tensor maps non-empty
}

// ---------------------------------------------------------------------------------------
// Eq. 3 at tile granularity.  For text row i of a sequence (chunk c = i / k):
//   first visible text token   lo(i)  = max(0, c - C) * k
//   visible summary rows       [0, cnt(i)),  cnt(i) = max(0, c - C) * m
// Both are non-decreasing in i, which makes the visited tiles of a query tile two
// contiguous ranges and the unmasked tiles contiguous sub-ranges.
// ---------------------------------------------------------------------------------------
struct Eq3 {
    int k, m, C;
    int64_t lo(int64_t i) const { return std::max<int64_t>(0, i / k - C) * k; }
    int64_t cnt(int64_t i) const { return std::max<int64_t>(0, i / k - C) * m; }
};
struct TileClass { bool any, full; };

// query rows [i0, i1], text key rows [a0, a1] (all in range)
static TileClass classify_text(const Eq3& e, int64_t i0, int64_t i1, int64_t a0, int64_t a1)
{
    TileClass t;
    const int64_t ifirst = std::max(i0, a0);              // first row that can reach the tile causally
    t.any = (ifirst <= i1) && (e.lo(ifirst) <= a1);
    t.full = (e.lo(i1) <= a0) && (i0 >= a1);
    return t;
}
// query rows [i0, i1], summary stream rows [u0, u1]
static TileClass classify_summ(const Eq3& e, int64_t i0, int64_t i1, int64_t u0, int64_t u1)
{
    TileClass t;
    t.any = e.cnt(i1) > u0;
    t.full = e.cnt(i0) > u1;
    return t;
}

struct BaseItem {   // schedule of one (sequence, query tile); heads share it
    int32_t seq, q_tile, ns_tiles, ns_nomask, band_lo, band_hi, nm_lo, nm_hi;
};

static BaseItem schedule_q_tile(const Eq3& e, const SeqInfo& s, int seq, int qt)
{
    BaseItem it{};
    it.seq = seq;
    it.q_tile = qt;
    const int64_t i0 = (int64_t)qt * kTileM;
    const int64_t i1 = std::min<int64_t>(s.n_text, i0 + kTileM) - 1;
    // summary stream: tiles [0, ceil(cnt(i1) / kTileN))
    const int64_t cmax = std::min<int64_t>(e.cnt(i1), s.n_summ);
    it.ns_tiles = (int32_t)((cmax + kTileN - 1) / kTileN);
    it.ns_nomask = 0;
    for (int ut = 0; ut < it.ns_tiles; ++ut) {
        const int64_t u0 = (int64_t)ut * kTileN, u1 = std::min<int64_t>(s.n_summ, u0 + kTileN) - 1;
        const TileClass tc = classify_summ(e, i0, i1, u0, u1);
        if (tc.full && (u1 - u0 + 1) == kTileN && it.ns_nomask == ut) it.ns_nomask = ut + 1;
    }
    // text stream: tiles [lo(i0) / kTileN, qt]
    it.band_lo = (int32_t)(e.lo(i0) / kTileN);
    it.band_hi = qt;
    it.nm_lo = it.nm_hi = it.band_lo;
    bool open = false, closed = false;
    for (int bt = it.band_lo; bt <= it.band_hi; ++bt) {
        const int64_t a0 = (int64_t)bt * kTileN, a1 = std::min<int64_t>(s.n_text, a0 + kTileN) - 1;
        const TileClass tc = classify_text(e, i0, i1, a0, a1);
        const bool nomask = tc.full && (a1 - a0 + 1) == kTileN;
        if (nomask && !open && !closed) { open = true; it.nm_lo = bt; it.nm_hi = bt + 1; }
        else if (nomask && open) it.nm_hi = bt + 1;
        else if (!nomask && open) { open = false; closed = true; }
    }
    return it;
}

void build_schedule(const ksa_params* p, HostSchedule& hs, int target_chunks)
{
    const Eq3 e{p->chunk_len, p->summaries_per_chunk, p->window_chunks};
    const int k = p->chunk_len, m = p->summaries_per_chunk, s = k + m;
    // two query heads per work item: a pair inside a GQA group shares its K / V tiles; a pair that straddles two KV
    // heads (multi-head attention, odd group sizes) streams K / V per head; a single head only if the count is odd
    const int heads_per_item = (p->num_q_heads % 2 == 0) ? 2 : 1;
    struct Tagged { BaseItem it; int32_t chunk; };
    std::vector<Tagged> base;
    hs.chunks.clear();
    int64_t total_tiles = 0;
    for (int b = 0; b < p->num_seqs; ++b) total_tiles += hs.seqs[b].text_pad / kTileM;
    const int64_t per_chunk = target_chunks > 0 ? std::max<int64_t>(1, (total_tiles + target_chunks - 1) / target_chunks) : 0;
    for (int b = 0; b < p->num_seqs; ++b) {
        const SeqInfo& sq = hs.seqs[b];
        const int n_qt = sq.text_pad / kTileM;
        const int64_t n = sq.n_text, L = n + sq.n_summ;
        auto aug_of = [&](int64_t i) -> int64_t { return i >= n ? L : (i / k) * s + (i % k); };   // Eq. 1
        for (int qt = 0; qt < n_qt; ++qt) {
            if (per_chunk > 0 && qt % per_chunk == 0) {
                const int t0 = qt, t1 = (int)std::min<int64_t>(n_qt, qt + per_chunk);
                const bool last = (t1 == n_qt);
                const int64_t i0 = (int64_t)t0 * kTileM, i1 = last ? n : (int64_t)t1 * kTileM;
                RowChunk c{};
                c.seq = b;
                c.text0 = (int32_t)i0; c.text1 = last ? sq.text_pad : (int32_t)i1;
                // summaries of the full chunks whose rows end inside [i0, i1)
                const int64_t j0 = i0 / k, j1 = last ? sq.n_chunks : i1 / k;
                c.summ0 = (int32_t)(j0 * m); c.summq1 = (int32_t)(j1 * m);
                c.summ1 = last ? sq.summ_pad : c.summq1;
                c.aug0 = sq.aug_off + aug_of(i0); c.aug1 = sq.aug_off + aug_of(i1);
                hs.chunks.push_back(c);
            }
            base.push_back({schedule_q_tile(e, sq, b, qt), (int32_t)hs.chunks.size() - 1});
        }
    }
    // longest first (chunk by chunk, if chunked); ties keep (sequence, tile) order so that
    // neighbours share K/V tiles in L2
    std::stable_sort(base.begin(), base.end(), [](const Tagged& x, const Tagged& y) {
        if (x.chunk != y.chunk) return x.chunk < y.chunk;
        return (x.it.ns_tiles + x.it.band_hi - x.it.band_lo) > (y.it.ns_tiles + y.it.band_hi - y.it.band_lo);
    });
    hs.work.clear();
    hs.work.reserve(base.size() * (p->num_q_heads / heads_per_item));
    for (const Tagged& tg : base) {
        const BaseItem& bi = tg.it;
        if (tg.chunk >= 0) {
            RowChunk& c = hs.chunks[tg.chunk];
            if (c.work_cnt == 0) c.work_off = (int64_t)hs.work.size();
            c.work_cnt += p->num_q_heads / heads_per_item;
        }
        for (int h = 0; h < p->num_q_heads; h += heads_per_item) {
            WorkItem w{};
            w.seq = bi.seq; w.q_tile = bi.q_tile; w.head0 = h; w.n_heads = heads_per_item;
            w.ns_tiles = bi.ns_tiles; w.ns_nomask = bi.ns_nomask;
            w.band_lo = bi.band_lo; w.band_hi = bi.band_hi;
            w.band_nomask_lo = bi.nm_lo; w.band_nomask_hi = bi.nm_hi;
            hs.work.push_back(w);
        }
    }
}

// Range check of a freshly built schedule, before it is ever uploaded: every field a kernel will index with.
static bool schedule_in_range(const ksa_params* p, const HostSchedule& hs)
{
    const int G = p->num_q_heads / p->num_kv_heads;
    int64_t aug = 0;
    for (const SeqInfo& s : hs.seqs) {
        if (s.aug_off != aug || s.n_text < 1 || s.text_pad % kTileM || s.summ_pad % kTileN) return false;
        if (s.text_off < 0 || s.text_off + (int64_t)s.text_pad > hs.text_rows) return false;
        if (s.summ_off < 0 || s.summ_off + (int64_t)s.summ_pad > hs.summ_rows) return false;
        aug += (int64_t)s.n_text + s.n_summ;
    }
    if (aug != hs.total_aug) return false;
    for (const WorkItem& w : hs.work) {
        if (w.seq < 0 || w.seq >= (int)hs.seqs.size()) return false;
        const SeqInfo& s = hs.seqs[w.seq];
        if (w.q_tile < 0 || (int64_t)w.q_tile * kTileM >= s.text_pad) return false;
        if (w.n_heads < 1 || w.n_heads > 2 || w.head0 < 0 || w.head0 + w.n_heads > p->num_q_heads) return false;
        if ((w.head0 + w.n_heads - 1) / G - w.head0 / G > 1) return false;                  // one KV head per item, or one per head
        if (w.ns_tiles < 0 || (int64_t)w.ns_tiles * kTileN > s.summ_pad || w.ns_nomask < 0 || w.ns_nomask > w.ns_tiles) return false;
        if (w.band_lo < 0 || w.band_hi < w.band_lo || w.band_hi != w.q_tile) return false;
        if (w.band_nomask_lo < w.band_lo || w.band_nomask_hi > w.band_hi + 1 || w.band_nomask_hi < w.band_nomask_lo) return false;
    }
    for (const RowChunk& c : hs.chunks)
        if (c.work_off < 0 || c.work_off + c.work_cnt > (int64_t)hs.work.size() || c.aug0 < 0 || c.aug1 > hs.total_aug || c.aug1 < c.aug0) return false;
    return true;
}

static std::vector<int32_t> schedule_key(const ksa_params* p)
{
    std::vector<int32_t> key;
    key.reserve(p->num_seqs + 8);
    key.push_back(p->num_seqs);
    for (int b = 0; b <= p->num_seqs; ++b) key.push_back(p->cu_text_lens[b]);
    key.push_back(p->chunk_len); key.push_back(p->summaries_per_chunk); key.push_back(p->window_chunks);
    key.push_back(p->num_q_heads); key.push_back(p->num_kv_heads); key.push_back(p->head_dim);
    return key;
}

WorkspaceLayout workspace_layout(const ksa_params* p, const HostSchedule& hs)
{
    WorkspaceLayout w{};
    const size_t D2 = (size_t)p->head_dim * 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 1024); return o; };
    w.qt = take((size_t)p->num_q_heads * hs.text_rows * D2);
    w.kt = take((size_t)p->num_kv_heads * hs.text_rows * D2);
    w.vt = take((size_t)p->num_kv_heads * hs.text_rows * D2);
    w.ks = take((size_t)p->num_kv_heads * hs.summ_rows * D2);
    w.vs = take((size_t)p->num_kv_heads * hs.summ_rows * D2);
    w.total = off;
    return w;
}

// ---------------------------------------------------------------------------------------
// exported: helpers
// ---------------------------------------------------------------------------------------
extern "C" __attribute__((visibility("default"))) int64_t ksa_aug_len(int64_t n_text, int32_t k, int32_t m)
{
    if (n_text < 0 || k < 1 || m < 0) return -1;
    return n_text + (n_text / k) * (int64_t)m;
}

extern "C" __attribute__((visibility("default"))) int64_t ksa_total_aug_len(const ksa_params* p)
{
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    int64_t t = 0;
    for (int b = 0; b < p->num_seqs; ++b)
        t += ksa_aug_len(p->cu_text_lens[b + 1] - p->cu_text_lens[b], p->chunk_len, p->summaries_per_chunk);
    return t;
}

extern "C" __attribute__((visibility("default"))) int ksa_workspace_bytes(const ksa_ctx*, const ksa_params* p, size_t* bytes)
{
    if (!bytes) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if (direct_ok(p)) { *bytes = 256; return KSA_OK; }     // nothing is packed
    HostSchedule hs;
    build_layout(p, hs);
    *bytes = workspace_layout(p, hs).total;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_visible_pairs(const ksa_params* p, int64_t* pairs)
{
    if (!pairs) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    const Eq3 e{p->chunk_len, p->summaries_per_chunk, p->window_chunks};
    const int64_t k = p->chunk_len, m = p->summaries_per_chunk;
    int64_t total = 0;
    for (int b = 0; b < p->num_seqs; ++b) {
        const int64_t n = p->cu_text_lens[b + 1] - p->cu_text_lens[b];
        for (int64_t c = 0; c * k < n; ++c) {             // rows of chunk c: i = ck .. min(n, ck+k)-1
            const int64_t rows = std::min(n, c * k + k) - c * k;
            const int64_t i0 = c * k;
            // sum over rows of (i - lo + 1) + cnt
            total += rows * (i0 - e.lo(i0) + 1 + e.cnt(i0)) + rows * (rows - 1) / 2;
        }
        const int64_t J = n / k;
        for (int64_t r = 0; r < m; ++r)
            total += J * (k + ((p->flags & KSA_FLAG_SUMMARY_TEXT_ONLY) ? 0 : r + 1));
    }
    *pairs = total;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) const char* ksa_strerror(int status)
{
    switch (status) {
        case KSA_OK: return "ok";
        case KSA_ERR_INVALID_ARG: return "invalid argument";
        case KSA_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case KSA_ERR_WORKSPACE: return "workspace missing or too small";
        case KSA_ERR_CUDA: return "CUDA call failed";
        case KSA_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case KSA_ERR_NOMEM: return "out of host memory";
        case KSA_ERR_INTERNAL: return "the library's schedule failed its own range check";
        default: return "unknown status";
    }
}

// ---------------------------------------------------------------------------------------
// exported: context
// ---------------------------------------------------------------------------------------
extern "C" __attribute__((visibility("default"))) int ksa_create(ksa_ctx** out, int cuda_device)
{
    if (!out) return KSA_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return KSA_ERR_CUDA;
    if (cuda_device < 0 || cuda_device >= count) return KSA_ERR_INVALID_ARG;
    if ((e = cudaSetDevice(cuda_device)) != cudaSuccess) return KSA_ERR_CUDA;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, cuda_device)) != cudaSuccess) return KSA_ERR_CUDA;
    if (prop.major != 10) return KSA_ERR_UNSUPPORTED;     // kernels are built for sm_100a only
    ksa_ctx* ctx = new (std::nothrow) ksa_ctx();
    if (!ctx) return KSA_ERR_NOMEM;
    ctx->device = cuda_device;
    ctx->num_sms = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) { delete ctx; return KSA_ERR_CUDA; }
    ctx->encode = (EncodeTiledFn)fn;
    if ((e = cudaMalloc(&ctx->d_status, sizeof(int32_t))) != cudaSuccess) { delete ctx; return KSA_ERR_CUDA; }
    if ((e = cudaMemset(ctx->d_status, 0, sizeof(int32_t))) != cudaSuccess) { cudaFree(ctx->d_status); delete ctx; return KSA_ERR_CUDA; }
    cudaEventCreate(&ctx->ev0);
    cudaEventCreate(&ctx->ev1);
    *out = ctx;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_destroy(ksa_ctx* ctx)
{
    if (!ctx) return KSA_OK;
    cudaSetDevice(ctx->device);
    if (ctx->d_seqs) cudaFree(ctx->d_seqs);
    if (ctx->d_work) cudaFree(ctx->d_work);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->ev0) cudaEventDestroy(ctx->ev0);
    if (ctx->ev1) cudaEventDestroy(ctx->ev1);
    if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
    for (cudaEvent_t e : ctx->ev_in) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_done) cudaEventDestroy(e);
    if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
    if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
    delete ctx;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_last_device_status(ksa_ctx* ctx, int32_t* status)
{
    if (!ctx || !status) return KSA_ERR_INVALID_ARG;
    cudaError_t e = cudaMemcpy(status, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return *status != 0 ? KSA_ERR_TIMEOUT : KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_clear_device_status(ksa_ctx* ctx)
{
    if (!ctx) return KSA_ERR_INVALID_ARG;
    cudaError_t e = cudaMemset(ctx->d_status, 0, sizeof(int32_t));
    return e == cudaSuccess ? KSA_OK : cuda_fail(ctx, e);
}

extern "C" __attribute__((visibility("default"))) int ksa_last_cuda_error(const ksa_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
extern "C" __attribute__((visibility("default"))) int64_t ksa_launch_count(const ksa_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" __attribute__((visibility("default"))) int ksa_device_info(ksa_ctx* ctx, int32_t* num_sms, int32_t* max_cta_pairs)
{
    if (!ctx) return KSA_ERR_INVALID_ARG;
    if (!ctx->pair_ready) {
        cudaError_t e = setup_text_pair(&ctx->max_pairs);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->pair_ready = true;
    }
    if (num_sms) *num_sms = ctx->num_sms;
    if (max_cta_pairs) *max_cta_pairs = ctx->max_pairs;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_enable_kernel_timing(ksa_ctx* ctx, int on)
{
    if (!ctx) return KSA_ERR_INVALID_ARG;
    ctx->timing = on != 0;
    ctx->timing_valid = false;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_text_kernel_ms(ksa_ctx* ctx, float* ms)
{
    if (!ctx || !ms || !ctx->timing_valid) return KSA_ERR_INVALID_ARG;
    cudaError_t e = cudaEventSynchronize(ctx->ev1);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    e = cudaEventElapsedTime(ms, ctx->ev0, ctx->ev1);
    return e == cudaSuccess ? KSA_OK : cuda_fail(ctx, e);
}

// ---------------------------------------------------------------------------------------
// schedule cache
// ---------------------------------------------------------------------------------------
static int ensure_schedule(ksa_ctx* ctx, const ksa_params* p, bool upload, int target_chunks = 0)
{
    std::vector<int32_t> key = schedule_key(p);
    key.push_back(target_chunks);
    if (ctx->sched.key != key) {
        HostSchedule hs;
        try {
            build_layout(p, hs);
            build_schedule(p, hs, target_chunks);
        } catch (const std::bad_alloc&) { return KSA_ERR_NOMEM; }
        if (!schedule_in_range(p, hs)) return KSA_ERR_INTERNAL;
        hs.key = key;
        ctx->sched = std::move(hs);
        // the device copies belong to the old schedule (cudaFree waits for work in flight)
        if (ctx->d_seqs) { cudaFree(ctx->d_seqs); ctx->d_seqs = nullptr; ctx->d_seqs_cap = 0; }
        if (ctx->d_work) { cudaFree(ctx->d_work); ctx->d_work = nullptr; ctx->d_work_cap = 0; }
    }
    if (upload && !ctx->d_seqs) {
        const HostSchedule& hs = ctx->sched;
        cudaError_t e;
        const size_t sb = hs.seqs.size() * sizeof(SeqInfo), wb = std::max<size_t>(1, hs.work.size()) * sizeof(WorkItem);
        if ((e = cudaMalloc(&ctx->d_seqs, sb)) != cudaSuccess) { ctx->d_seqs = nullptr; return cuda_fail(ctx, e); }
        if ((e = cudaMalloc(&ctx->d_work, wb)) != cudaSuccess) {
            cudaFree(ctx->d_seqs); ctx->d_seqs = nullptr; ctx->d_work = nullptr; return cuda_fail(ctx, e);
        }
        e = cudaMemcpy(ctx->d_seqs, hs.seqs.data(), sb, cudaMemcpyHostToDevice);
        if (e == cudaSuccess && !hs.work.empty())
            e = cudaMemcpy(ctx->d_work, hs.work.data(), hs.work.size() * sizeof(WorkItem), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            cudaFree(ctx->d_seqs); cudaFree(ctx->d_work); ctx->d_seqs = nullptr; ctx->d_work = nullptr;
            return cuda_fail(ctx, e);
        }
        ctx->d_seqs_cap = sb; ctx->d_work_cap = wb;
    }
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_schedule_dump(ksa_ctx* ctx, const ksa_params* p, ksa_tile_rec* recs, int64_t cap,
                                 int64_t* count)
{
    if (!count) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    HostSchedule local;
    build_layout(p, local);
    const Eq3 e{p->chunk_len, p->summaries_per_chunk, p->window_chunks};
    int64_t n = 0;
    bool overflow = false;
    auto emit = [&](const ksa_tile_rec& r) {
        if (recs && n < cap) recs[n] = r; else if (recs) overflow = true;
        ++n;
    };
    (void)ctx;
    for (int b = 0; b < p->num_seqs; ++b) {
        const SeqInfo& s = local.seqs[b];
        for (int qt = 0; qt < s.text_pad / kTileM; ++qt) {
            const BaseItem it = schedule_q_tile(e, s, b, qt);
            const int64_t i0 = (int64_t)qt * kTileM, i1 = std::min<int64_t>(s.n_text, i0 + kTileM) - 1;
            ksa_tile_rec r{};
            r.seq = b; r.q_stream = KSA_STREAM_TEXT; r.q_row0 = (int32_t)i0; r.q_rows = (int32_t)(i1 - i0 + 1);
            for (int ut = 0; ut < it.ns_tiles; ++ut) {
                const int64_t u0 = (int64_t)ut * kTileN, u1 = std::min<int64_t>(s.n_summ, u0 + kTileN) - 1;
                r.kv_stream = KSA_STREAM_SUMMARY; r.kv_row0 = (int32_t)u0; r.kv_rows = (int32_t)(u1 - u0 + 1);
                r.is_full = classify_summ(e, i0, i1, u0, u1).full ? 1 : 0;
                emit(r);
            }
            for (int bt = it.band_lo; bt <= it.band_hi; ++bt) {
                const int64_t a0 = (int64_t)bt * kTileN, a1 = std::min<int64_t>(s.n_text, a0 + kTileN) - 1;
                r.kv_stream = KSA_STREAM_TEXT; r.kv_row0 = (int32_t)a0; r.kv_rows = (int32_t)(a1 - a0 + 1);
                r.is_full = classify_text(e, i0, i1, a0, a1).full ? 1 : 0;
                emit(r);
            }
        }
    }
    *count = n;
    return overflow ? KSA_ERR_INVALID_ARG : KSA_OK;
}

// ---------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------
static int encode_stream_map(ksa_ctx* ctx, CUtensorMap* map, void* base, int D, int64_t rows, int H, int box_rows = kTileN)
{
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)H};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { ctx->last_cuda_error = (int)r; return KSA_ERR_CUDA; }
    return KSA_OK;
}

// Chunked view of a caller tensor [rows, H, D] (element strides st, sh): dims {D, rows_per_chunk, chunks, H},
// a box of box_rows / rows_per_chunk chunks.  `base` points at the first row of the view's first chunk.
static int encode_chunk_map(ksa_ctx* ctx, CUtensorMap* map, const void* base, int D, int rows_per_chunk, int chunk_rows,
                            int64_t chunks, int H, int64_t st, int64_t sh, int box_rows = kTileN)
{
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)rows_per_chunk, (cuuint64_t)chunks, (cuuint64_t)H};
    const cuuint64_t strides[3] = {(cuuint64_t)st * 2, (cuuint64_t)chunk_rows * st * 2, (cuuint64_t)sh * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)rows_per_chunk, (cuuint32_t)(box_rows / rows_per_chunk), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { ctx->last_cuda_error = (int)r; return KSA_ERR_CUDA; }
    return KSA_OK;
}

// Kernel arguments of a whole problem (schedule already cached and uploaded in ctx).
static KernelArgs make_args(ksa_ctx* ctx, const ksa_params* p, const void* q, const void* k, const void* v, void* out,
                            float* lse, void* workspace, const WorkspaceLayout& wl, bool direct = false)
{
    const HostSchedule& hs = ctx->sched;
    char* ws = (char*)workspace;
    KernelArgs a{};
    a.seqs = ctx->d_seqs; a.work = ctx->d_work;
    a.num_seqs = p->num_seqs; a.num_work = (int32_t)hs.work.size();
    a.k = p->chunk_len; a.m = p->summaries_per_chunk; a.C = p->window_chunks;
    a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.flags = p->flags;
    a.scale = p->softmax_scale;
    a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
    a.total_aug = hs.total_aug; a.text_rows = hs.text_rows; a.summ_rows = hs.summ_rows;
    a.max_text_pad = hs.max_text_pad; a.max_summ_pad = hs.max_summ_pad; a.max_n_summ = hs.max_n_summ;
    a.r_seq = -1;
    a.direct = direct ? 1 : 0;
    a.q = (const uint16_t*)q; a.kx = (const uint16_t*)k; a.v = (const uint16_t*)v;
    a.out = (uint16_t*)out; a.lse = lse;
    a.q_st = p->q_stride_tok; a.q_sh = p->q_stride_head; a.k_st = p->k_stride_tok; a.k_sh = p->k_stride_head;
    a.v_st = p->v_stride_tok; a.v_sh = p->v_stride_head; a.o_st = p->o_stride_tok; a.o_sh = p->o_stride_head;
    a.qt = (uint16_t*)(ws + wl.qt); a.kt = (uint16_t*)(ws + wl.kt); a.vt = (uint16_t*)(ws + wl.vt);
    a.ks = (uint16_t*)(ws + wl.ks); a.vs = (uint16_t*)(ws + wl.vs);
    a.status = ctx->d_status;
    return a;
}

// The tensor maps of a forward call: those of the one-CTA kernel, plus the two 64-key-row maps of the CTA-pair
// kernel where that one applies.
struct FwdMaps { TextMaps t; CUtensorMap kt_half, ks_half; bool pair = false; };

// Which tensor-core kernel takes the text rows when the caller does not say (KSA_FLAG_SINGLE_CTA_KERNEL /
// KSA_FLAG_CTA_PAIR_KERNEL): the faster one on the measured workloads.
static constexpr bool kPairKernelByDefault = false;

// The CTA-pair kernel takes work items of two query heads at head_dim 128; reading whole-chunk batches in place
// it also needs half a K tile (64 rows) to be a whole number of chunks in both views.
static bool pair_ok(const KernelArgs& a, uint32_t flags)
{
    if (flags & (KSA_FLAG_REFERENCE_KERNEL | KSA_FLAG_SINGLE_CTA_KERNEL)) return false;
    if (a.D != 128 || ((a.Hq / a.Hkv) & 1)) return false;
    if (a.direct && (64 % a.k != 0 || (a.m > 0 && 64 % a.m != 0))) return false;
    return kPairKernelByDefault || (flags & KSA_FLAG_CTA_PAIR_KERNEL);
}

// One-time kernel setup and the tensor maps of the packed streams (tensor-core paths only).
static int prepare_text(ksa_ctx* ctx, const KernelArgs& a, uint32_t flags, FwdMaps& fm)
{
    if (flags & KSA_FLAG_REFERENCE_KERNEL) return KSA_OK;
    TextMaps& maps = fm.t;
    fm.pair = pair_ok(a, flags);
    if (!ctx->tc_ready) {
        cudaError_t e = setup_text_tc();
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->tc_ready = true;
    }
    if (fm.pair && !ctx->pair_ready) {
        cudaError_t e = setup_text_pair(&ctx->max_pairs);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->pair_ready = true;
    }
    if (fm.pair && ctx->max_pairs < 1) fm.pair = false;
    int rc;
    if (a.direct) {
        const int s_len = a.k + a.m;
        const int64_t chunks = a.total_aug / s_len;
        if ((rc = encode_chunk_map(ctx, &maps.qt, a.q, a.D, a.k, s_len, chunks, a.Hq, a.q_st, a.q_sh)) != KSA_OK) return rc;
        if ((rc = encode_chunk_map(ctx, &maps.kt, a.kx, a.D, a.k, s_len, chunks, a.Hkv, a.k_st, a.k_sh)) != KSA_OK) return rc;
        if ((rc = encode_chunk_map(ctx, &maps.vt, a.v, a.D, a.k, s_len, chunks, a.Hkv, a.v_st, a.v_sh)) != KSA_OK) return rc;
        if (fm.pair && (rc = encode_chunk_map(ctx, &fm.kt_half, a.kx, a.D, a.k, s_len, chunks, a.Hkv, a.k_st, a.k_sh, 64)) != KSA_OK) return rc;
        if (a.m > 0) {      // summary rows start k rows into each chunk
            if ((rc = encode_chunk_map(ctx, &maps.ks, a.kx + (int64_t)a.k * a.k_st, a.D, a.m, s_len, chunks, a.Hkv, a.k_st, a.k_sh)) != KSA_OK) return rc;
            if (fm.pair && (rc = encode_chunk_map(ctx, &fm.ks_half, a.kx + (int64_t)a.k * a.k_st, a.D, a.m, s_len, chunks, a.Hkv, a.k_st, a.k_sh, 64)) != KSA_OK) return rc;
            return encode_chunk_map(ctx, &maps.vs, a.v + (int64_t)a.k * a.v_st, a.D, a.m, s_len, chunks, a.Hkv, a.v_st, a.v_sh);
        }
        maps.ks = maps.kt; maps.vs = maps.vt;    // never used: no summary tiles are scheduled
        fm.ks_half = fm.kt_half;
        return KSA_OK;
    }
    if ((rc = encode_stream_map(ctx, &maps.qt, a.qt, a.D, a.text_rows, a.Hq)) != KSA_OK) return rc;
    if ((rc = encode_stream_map(ctx, &maps.kt, a.kt, a.D, a.text_rows, a.Hkv)) != KSA_OK) return rc;
    if ((rc = encode_stream_map(ctx, &maps.vt, a.vt, a.D, a.text_rows, a.Hkv)) != KSA_OK) return rc;
    if ((rc = encode_stream_map(ctx, &maps.ks, a.ks, a.D, a.summ_rows, a.Hkv)) != KSA_OK) return rc;
    if (fm.pair) {
        if ((rc = encode_stream_map(ctx, &fm.kt_half, a.kt, a.D, a.text_rows, a.Hkv, 64)) != KSA_OK) return rc;
        if ((rc = encode_stream_map(ctx, &fm.ks_half, a.ks, a.D, a.summ_rows, a.Hkv, 64)) != KSA_OK) return rc;
    }
    return encode_stream_map(ctx, &maps.vs, a.vs, a.D, a.summ_rows, a.Hkv);
}

// Text-row kernel over the work items a.work[0 .. a.num_work).
static int launch_text(ksa_ctx* ctx, const KernelArgs& a, uint32_t flags, const FwdMaps& fm, cudaStream_t stream)
{
    cudaError_t e;
    if (flags & KSA_FLAG_REFERENCE_KERNEL) {
        e = launch_text_ref(a, stream);
    } else if (fm.pair) {
        PairMaps pm;
        pm.qt = fm.t.qt; pm.kt = fm.kt_half; pm.vt = fm.t.vt; pm.ks = fm.ks_half; pm.vs = fm.t.vs;
        e = launch_text_pair(a, pm, ctx->max_pairs, stream);
    } else {
        e = launch_text_tc(a, fm.t, ctx->num_sms, stream);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_attn_fwd(ksa_ctx* ctx, const void* q, const void* k, const void* v, void* out, float* lse,
                            void* workspace, size_t workspace_bytes, const ksa_params* p, void* cuda_stream)
{
    if (!ctx || !q || !k || !v || !out || !lse) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    const uintptr_t ptrs[5] = {(uintptr_t)q, (uintptr_t)k, (uintptr_t)v, (uintptr_t)out, (uintptr_t)lse};
    for (int i = 0; i < 5; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    if ((rc = ensure_schedule(ctx, p, true)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    const bool direct = direct_ok(p);
    const WorkspaceLayout wl = workspace_layout(p, hs);
    if (!direct && (!workspace || workspace_bytes < wl.total || ((uintptr_t)workspace & 255))) return KSA_ERR_WORKSPACE;

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    KernelArgs a = make_args(ctx, p, q, k, v, out, lse, workspace, wl, direct);
    cudaError_t e;
    if (!direct) {
        if ((e = launch_pack(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }
    if (a.m > 0 && a.max_n_summ > 0) {
        if ((e = launch_summary(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }
    if (ctx->timing) cudaEventRecord(ctx->ev0, stream);
    FwdMaps maps;
    if ((rc = prepare_text(ctx, a, p->flags, maps)) != KSA_OK) return rc;
    if ((rc = launch_text(ctx, a, p->flags, maps, stream)) != KSA_OK) return rc;
    if (ctx->timing) { cudaEventRecord(ctx->ev1, stream); ctx->timing_valid = true; }
    return KSA_OK;
}

// ---- sequence-parallel parts ---------------------------------------------------------------------
// The query rows are cut into num_parts contiguous parts of about equal work (Eq. 3 makes later rows more
// expensive): the row chunks of a schedule with 16 chunks per part, grouped by their tile counts.
static constexpr int kPartChunkFactor = 16;
static void part_chunk_range(const HostSchedule& hs, int part, int num_parts, size_t& c0, size_t& c1)
{
    const size_t n = hs.chunks.size();
    std::vector<int64_t> before(n + 1, 0);                               // tile visits of the chunks before chunk c
    for (size_t c = 0; c < n; ++c) {
        int64_t cost = 0;
        for (int64_t w = hs.chunks[c].work_off; w < hs.chunks[c].work_off + hs.chunks[c].work_cnt; ++w) {
            const WorkItem& it = hs.work[(size_t)w];
            cost += (int64_t)it.n_heads * (it.ns_tiles + it.band_hi - it.band_lo + 1);
        }
        before[c + 1] = before[c] + cost;
    }
    auto boundary = [&](int i) -> size_t {                               // first chunk with at least i / num_parts of the work before it
        if (i <= 0) return 0;
        if (i >= num_parts) return n;
        const int64_t want = (before[n] * i + num_parts - 1) / num_parts;
        return (size_t)(std::lower_bound(before.begin(), before.end(), want) - before.begin());
    };
    c0 = std::min(boundary(part), n);
    c1 = std::min(std::max(boundary(part + 1), c0), n);
}

extern "C" __attribute__((visibility("default"))) int ksa_part_rows(ksa_ctx* ctx, const ksa_params* p, int32_t part, int32_t num_parts,
                             int64_t* aug_begin, int64_t* aug_end)
{
    if (!ctx || !aug_begin || !aug_end || num_parts < 1 || part < 0 || part >= num_parts) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = ensure_schedule(ctx, p, false, num_parts * kPartChunkFactor)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    size_t c0, c1;
    part_chunk_range(hs, part, num_parts, c0, c1);
    if (c0 == c1) {                                                      // empty part: an empty range at its place in the order
        *aug_begin = *aug_end = (c0 < hs.chunks.size()) ? hs.chunks[c0].aug0 : hs.total_aug;
        return KSA_OK;
    }
    *aug_begin = hs.chunks[c0].aug0;
    *aug_end = hs.chunks[c1 - 1].aug1;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_attn_fwd_part(ksa_ctx* ctx, const void* q, const void* k, const void* v, void* out, float* lse,
                                 void* workspace, size_t workspace_bytes, const ksa_params* p, int32_t part,
                                 int32_t num_parts, void* cuda_stream)
{
    if (!ctx || !q || !k || !v || !out || !lse || num_parts < 1 || part < 0 || part >= num_parts) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    const uintptr_t ptrs[5] = {(uintptr_t)q, (uintptr_t)k, (uintptr_t)v, (uintptr_t)out, (uintptr_t)lse};
    for (int i = 0; i < 5; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    if ((rc = ensure_schedule(ctx, p, true, num_parts * kPartChunkFactor)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    const bool direct = direct_ok(p);
    const WorkspaceLayout wl = workspace_layout(p, hs);
    if (!direct && (!workspace || workspace_bytes < wl.total || ((uintptr_t)workspace & 255))) return KSA_ERR_WORKSPACE;
    size_t c0, c1;
    part_chunk_range(hs, part, num_parts, c0, c1);
    if (c0 == c1) return KSA_OK;

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    KernelArgs a = make_args(ctx, p, q, k, v, out, lse, workspace, wl, direct);
    cudaError_t e;
    if (!direct) {
        // the packed streams of the whole batch (rows after the part's last row are never read unmasked, but
        // packing them all keeps every tile finite)
        if ((e = launch_pack(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }
    const WorkItem* work_base = a.work;
    int64_t work_cnt = 0;
    for (size_t ci = c0; ci < c1; ++ci) {
        const RowChunk& c = hs.chunks[ci];
        work_cnt += c.work_cnt;
        if (a.m > 0 && c.summq1 > c.summ0) {                             // the summary rows whose chunks end inside this row chunk
            a.r_seq = c.seq;
            a.r_text0 = c.text0; a.r_text1 = c.text1;
            a.r_summ0 = c.summ0; a.r_summ1 = c.summ1; a.r_summq1 = c.summq1;
            if ((e = launch_summary(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
            ctx->launches += 1;
        }
    }
    a.r_seq = -1;
    a.work = work_base + hs.chunks[c0].work_off;                         // the chunks' items follow one another in the list
    a.num_work = (int32_t)work_cnt;
    FwdMaps maps;
    if ((rc = prepare_text(ctx, a, p->flags, maps)) != KSA_OK) return rc;
    return launch_text(ctx, a, p->flags, maps, stream);
}

// Number of row chunks the host entry point aims for (upload / compute / download stages).
static constexpr int kHostPipelineChunks = 16;    // 8: 37.3 ms end to end at 128K, 16: 35.4, 24: 35.2

// ---------------------------------------------------------------------------------------
// backward
// ---------------------------------------------------------------------------------------
struct BwdLayout { WorkspaceLayout fwd; size_t dot, lse_t, delta_t, dkt, dvt, dks, dvs, total; };
static BwdLayout bwd_layout(const ksa_params* p, const HostSchedule& hs)
{
    BwdLayout b{};
    // no packed streams and no packed dO where the tensor-core kernels read the caller's tensors in place
    const bool direct = direct_ok(p) && !(p->flags & KSA_FLAG_BWD_MMA_SYNC_KERNELS);
    if (!direct) b.fwd = workspace_layout(p, hs);
    size_t off = b.fwd.total;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 1024); return o; };
    const size_t D = (size_t)p->head_dim;
    b.dot = take(direct ? 0 : (size_t)p->num_q_heads * hs.text_rows * D * 2);
    b.lse_t = take((size_t)p->num_q_heads * hs.text_rows * 4);
    b.delta_t = take((size_t)p->num_q_heads * hs.text_rows * 4);
    b.dkt = take((size_t)p->num_kv_heads * hs.text_rows * D * 4);
    b.dvt = take((size_t)p->num_kv_heads * hs.text_rows * D * 4);
    b.dks = take((size_t)p->num_kv_heads * hs.summ_rows * D * 4);
    b.dvs = take((size_t)p->num_kv_heads * hs.summ_rows * D * 4);
    b.total = off;
    return b;
}

extern "C" __attribute__((visibility("default"))) int ksa_bwd_workspace_bytes(const ksa_ctx*, const ksa_params* p, size_t* bytes)
{
    if (!bytes) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    HostSchedule hs;
    build_layout(p, hs);
    *bytes = bwd_layout(p, hs).total;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_attn_bwd(ksa_ctx* ctx, const void* q, const void* k, const void* v, const void* out,
                            const float* lse, const void* dout, void* dq, void* dk, void* dv, void* workspace,
                            size_t workspace_bytes, const ksa_params* p, void* cuda_stream)
{
    if (!ctx || !q || !k || !v || !out || !lse || !dout || !dq || !dk || !dv) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    if (p->flags & KSA_FLAG_REFERENCE_KERNEL) return KSA_ERR_INVALID_ARG;
    const uintptr_t ptrs[9] = {(uintptr_t)q, (uintptr_t)k, (uintptr_t)v, (uintptr_t)out, (uintptr_t)lse, (uintptr_t)dout,
                               (uintptr_t)dq, (uintptr_t)dk, (uintptr_t)dv};
    for (int i = 0; i < 9; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    if ((rc = ensure_schedule(ctx, p, true)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    const BwdLayout bl = bwd_layout(p, hs);
    if (!workspace || workspace_bytes < bl.total || ((uintptr_t)workspace & 255)) return KSA_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* ws = (char*)workspace;
    cudaError_t e;
    if (!ctx->bwd_ready) {            // the shared-memory opt-in is per device: kept per context
        if ((e = setup_bwd()) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->bwd_ready = true;
    }
    // packed streams of the forward pass (text Q, K, V and summary K, V) -- not needed when the tensor-core kernels
    // can read whole tiles straight from the caller's tensors (the no-pack case of the forward pass)
    const bool direct = direct_ok(p) && !(p->flags & KSA_FLAG_BWD_MMA_SYNC_KERNELS);
    KernelArgs fa = make_args(ctx, p, q, k, v, dq /* unused */, const_cast<float*>(lse), workspace, bl.fwd);
    if (!direct && (e = launch_pack(fa, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    BwdArgs a{};
    a.seqs = ctx->d_seqs; a.num_seqs = p->num_seqs;
    a.k = p->chunk_len; a.m = p->summaries_per_chunk; a.C = p->window_chunks;
    a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.flags = p->flags; a.scale = p->softmax_scale; a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
    a.total_aug = hs.total_aug; a.text_rows = hs.text_rows; a.summ_rows = hs.summ_rows;
    a.max_text_pad = hs.max_text_pad; a.max_summ_pad = hs.max_summ_pad; a.max_n_summ = hs.max_n_summ;
    a.q = (const uint16_t*)q; a.kx = (const uint16_t*)k; a.v = (const uint16_t*)v; a.out = (const uint16_t*)out;
    a.dout = (const uint16_t*)dout; a.lse = lse;
    a.dq = (uint16_t*)dq; a.dk = (uint16_t*)dk; a.dv = (uint16_t*)dv;
    a.q_st = a.dq_st = p->q_stride_tok; a.q_sh = a.dq_sh = p->q_stride_head;
    a.k_st = a.dk_st = p->k_stride_tok; a.k_sh = a.dk_sh = p->k_stride_head;
    a.v_st = a.dv_st = p->v_stride_tok; a.v_sh = a.dv_sh = p->v_stride_head;
    a.o_st = a.do_st = p->o_stride_tok; a.o_sh = a.do_sh = p->o_stride_head;
    a.qt = fa.qt; a.kt = fa.kt; a.vt = fa.vt; a.ks = fa.ks; a.vs = fa.vs;
    a.dot = (uint16_t*)(ws + bl.dot); a.lse_t = (float*)(ws + bl.lse_t); a.delta_t = (float*)(ws + bl.delta_t);
    a.dkt = (float*)(ws + bl.dkt); a.dvt = (float*)(ws + bl.dvt); a.dks = (float*)(ws + bl.dks); a.dvs = (float*)(ws + bl.dvs);
    a.status = ctx->d_status;
    a.direct = direct ? 1 : 0;
    // The four accumulators are contiguous in the workspace: one clear.  Where one CTA of the tensor-core dK / dV kernel
    // covers every query tile that sees a text key tile, that launch stores the text keys' rows instead of adding to them:
    // then only the summary keys' accumulators are cleared and the summary rows' kernel, which adds to both, runs after it.
    const bool text_stored = !(p->flags & KSA_FLAG_BWD_MMA_SYNC_KERNELS) && bwd_text_keys_stored(a);
    const size_t clear0 = text_stored ? bl.dks : bl.dkt;
    if (bl.total > clear0 && (e = cudaMemsetAsync(ws + clear0, 0, bl.total - clear0, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = launch_bwd_prep(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if (!text_stored && (e = launch_bwd_summary(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if (!(p->flags & KSA_FLAG_BWD_MMA_SYNC_KERNELS)) {
        // text rows on the tcgen05 tensor cores, fed by TMA from the packed streams or the caller's tensors
        if (!ctx->bwd_tc_ready) {
            if ((e = setup_bwd_tc()) != cudaSuccess) return cuda_fail(ctx, e);
            ctx->bwd_tc_ready = true;
        }
        BwdMaps bm;
        if (direct) {
            // chunked views [D, rows per chunk, chunk, head] of the caller's tensors; summary rows start k rows into a chunk
            const int s_len = a.k + a.m;
            const int64_t chunks = a.total_aug / s_len;
            if ((rc = encode_chunk_map(ctx, &bm.qt, a.q, a.D, a.k, s_len, chunks, a.Hq, a.q_st, a.q_sh)) != KSA_OK) return rc;
            if ((rc = encode_chunk_map(ctx, &bm.dot, a.dout, a.D, a.k, s_len, chunks, a.Hq, a.do_st, a.do_sh)) != KSA_OK) return rc;
            if ((rc = encode_chunk_map(ctx, &bm.kt, a.kx, a.D, a.k, s_len, chunks, a.Hkv, a.k_st, a.k_sh)) != KSA_OK) return rc;
            if ((rc = encode_chunk_map(ctx, &bm.vt, a.v, a.D, a.k, s_len, chunks, a.Hkv, a.v_st, a.v_sh)) != KSA_OK) return rc;
            if (a.m > 0) {
                if ((rc = encode_chunk_map(ctx, &bm.ks, a.kx + (int64_t)a.k * a.k_st, a.D, a.m, s_len, chunks, a.Hkv, a.k_st, a.k_sh)) != KSA_OK) return rc;
                if ((rc = encode_chunk_map(ctx, &bm.vs, a.v + (int64_t)a.k * a.v_st, a.D, a.m, s_len, chunks, a.Hkv, a.v_st, a.v_sh)) != KSA_OK) return rc;
            } else {
                bm.ks = bm.kt; bm.vs = bm.vt;    // never used: no summary tiles
            }
        } else {
            struct { CUtensorMap* map; const void* base; int64_t rows; int H; } streams[6] = {
                {&bm.qt, a.qt, a.text_rows, a.Hq},   {&bm.dot, a.dot, a.text_rows, a.Hq},
                {&bm.kt, a.kt, a.text_rows, a.Hkv},  {&bm.vt, a.vt, a.text_rows, a.Hkv},
                {&bm.ks, a.ks, a.summ_rows, a.Hkv},  {&bm.vs, a.vs, a.summ_rows, a.Hkv}};
            for (auto& t : streams)
                if ((rc = encode_stream_map(ctx, t.map, const_cast<void*>(t.base), a.D, t.rows, t.H)) != KSA_OK) return rc;
        }
        if ((e = launch_bwd_dq_tc(a, bm, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = launch_bwd_dkv_tc(a, bm, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    } else {
        if ((e = launch_bwd_dq(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = launch_bwd_dkv(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    }
    if (text_stored && (e = launch_bwd_summary(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = launch_bwd_finish(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += (direct ? 4 : 5) + ((a.m > 0 && a.max_n_summ > 0) ? 2 : 0);
    return KSA_OK;
}

// ---- Q/K/V preparation upstream of the attention (include/ksa_prep.h) --------------------------------
extern "C" __attribute__((visibility("default"))) int ksa_anneal_lambda(int64_t step, int64_t s_start, int64_t s_end, float* lambda)
{
    if (!lambda || s_end <= s_start) return KSA_ERR_INVALID_ARG;
    if (step <= s_start) *lambda = 1.f;
    else if (step >= s_end) *lambda = 0.f;
    else *lambda = (float)(1.0 - (double)(step - s_start) / (double)(s_end - s_start));
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int64_t ksa_total_summary_rows(const ksa_params* p)
{
    if (validate(p) != KSA_OK) return KSA_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int b = 0; b < p->num_seqs; ++b)
        total += (int64_t)((p->cu_text_lens[b + 1] - p->cu_text_lens[b]) / p->chunk_len) * p->summaries_per_chunk;
    return total;
}

extern "C" __attribute__((visibility("default"))) int ksa_position_ids(const ksa_params* p, int32_t* position_ids)
{
    if (!position_ids) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    const int k = p->chunk_len, m = p->summaries_per_chunk;
    int64_t row = 0;
    for (int b = 0; b < p->num_seqs; ++b) {
        const int n = p->cu_text_lens[b + 1] - p->cu_text_lens[b];
        for (int i = 0; i < n; ++i) {
            position_ids[row++] = i;                                     // a text token keeps its index
            if ((i + 1) % k == 0)                                        // chunk complete: its summary tokens
                for (int r = 0; r < m; ++r) position_ids[row++] = i;     // ... take its last text token's id (Sec. 2.2.1)
        }
    }
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_qkv_prepare(ksa_ctx* ctx, const void* q_main, const void* k_main, const void* v_main,
                               const void* q_summ, const void* k_summ, const void* v_summ,
                               void* q_out, void* k_out, void* v_out, float lambda, float rope_theta, uint32_t prep_flags,
                               const ksa_params* p, void* cuda_stream)
{
    if (!ctx || !q_main || !k_main || !v_main || !q_out || !k_out || !v_out) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    if (!(lambda >= 0.f && lambda <= 1.f)) return KSA_ERR_INVALID_ARG;
    const bool rope = !(prep_flags & KSA_PREP_NO_ROPE);
    if (rope && !(rope_theta > 0.f)) return KSA_ERR_INVALID_ARG;
    const bool need_summ = lambda != 0.f && ksa_total_summary_rows(p) > 0;
    if (need_summ && (!q_summ || !k_summ || !v_summ)) return KSA_ERR_INVALID_ARG;
    const uintptr_t ptrs[9] = {(uintptr_t)q_main, (uintptr_t)k_main, (uintptr_t)v_main, (uintptr_t)q_summ, (uintptr_t)k_summ,
                               (uintptr_t)v_summ, (uintptr_t)q_out, (uintptr_t)k_out, (uintptr_t)v_out};
    for (int i = 0; i < 9; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    if ((rc = ensure_schedule(ctx, p, true)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    PrepArgs a{};
    a.seqs = ctx->d_seqs;
    a.k = p->chunk_len; a.m = p->summaries_per_chunk; a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.rope = rope ? 1 : 0;
    a.lambda = need_summ ? lambda : 0.f;
    for (int d = 0; d < p->head_dim / 2 && d < 64; ++d)
        a.inv_freq[d] = rope ? std::pow((double)rope_theta, -2.0 * d / (double)p->head_dim) : 0.0;
    a.qm = (const uint16_t*)q_main; a.km = (const uint16_t*)k_main; a.vm = (const uint16_t*)v_main;
    a.qs = (const uint16_t*)q_summ; a.ks = (const uint16_t*)k_summ; a.vs = (const uint16_t*)v_summ;
    a.qo = (uint16_t*)q_out; a.ko = (uint16_t*)k_out; a.vo = (uint16_t*)v_out;
    a.q_st = p->q_stride_tok; a.q_sh = p->q_stride_head; a.k_st = p->k_stride_tok; a.k_sh = p->k_stride_head;
    a.v_st = p->v_stride_tok; a.v_sh = p->v_stride_head;
    int64_t max_aug_len = 0;
    for (const SeqInfo& s : hs.seqs) max_aug_len = std::max<int64_t>(max_aug_len, (int64_t)s.n_text + s.n_summ);
    cudaError_t e = launch_prep(a, max_aug_len, p->num_seqs, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return KSA_OK;
}

// ---- preparation fused into the pack pass (include/ksa_prep.h) ------------------------------------------
// Workspace: the five packed streams of the forward pass, then the prepared query rows of the summary tokens.
static size_t prepared_ws_bytes(const ksa_params* p, const HostSchedule& hs, size_t* qs_off)
{
    const WorkspaceLayout wl = workspace_layout(p, hs);
    if (qs_off) *qs_off = wl.total;
    return wl.total + (size_t)round_up((int64_t)((size_t)p->num_q_heads * hs.summ_rows * p->head_dim * 2), 1024);
}

extern "C" __attribute__((visibility("default"))) int ksa_prepared_workspace_bytes(const ksa_ctx*, const ksa_params* p, size_t* bytes)
{
    if (!bytes) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    HostSchedule hs;
    build_layout(p, hs);
    *bytes = prepared_ws_bytes(p, hs, nullptr);
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_attn_fwd_prepared(ksa_ctx* ctx, const void* q_main, const void* k_main, const void* v_main,
                                     const void* q_summ, const void* k_summ, const void* v_summ,
                                     float lambda, float rope_theta, uint32_t prep_flags,
                                     void* out, float* lse, void* workspace, size_t workspace_bytes,
                                     const ksa_params* p, void* cuda_stream)
{
    if (!ctx || !q_main || !k_main || !v_main || !out || !lse) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    if (p->flags & KSA_FLAG_REFERENCE_KERNEL) return KSA_ERR_INVALID_ARG;
    if (!(lambda >= 0.f && lambda <= 1.f)) return KSA_ERR_INVALID_ARG;
    const bool rope = !(prep_flags & KSA_PREP_NO_ROPE);
    if (rope && !(rope_theta > 0.f)) return KSA_ERR_INVALID_ARG;
    const bool need_summ = lambda != 0.f && ksa_total_summary_rows(p) > 0;
    if (need_summ && (!q_summ || !k_summ || !v_summ)) return KSA_ERR_INVALID_ARG;
    const uintptr_t ptrs[8] = {(uintptr_t)q_main, (uintptr_t)k_main, (uintptr_t)v_main, (uintptr_t)q_summ, (uintptr_t)k_summ,
                               (uintptr_t)v_summ, (uintptr_t)out, (uintptr_t)lse};
    for (int i = 0; i < 8; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;
    if ((rc = ensure_schedule(ctx, p, true)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    size_t qs_off = 0;
    const size_t need = prepared_ws_bytes(p, hs, &qs_off);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return KSA_ERR_WORKSPACE;
    const WorkspaceLayout wl = workspace_layout(p, hs);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the attention kernels read the packed streams only (a.direct = 0); q, k, v of the arguments are the projections
    KernelArgs a = make_args(ctx, p, q_main, k_main, v_main, out, lse, workspace, wl, false);
    uint16_t* qs = (uint16_t*)((char*)workspace + qs_off);

    PrepArgs pa{};
    pa.seqs = ctx->d_seqs;
    pa.k = p->chunk_len; pa.m = p->summaries_per_chunk; pa.Hq = p->num_q_heads; pa.Hkv = p->num_kv_heads; pa.D = p->head_dim;
    pa.rope = rope ? 1 : 0;
    pa.lambda = need_summ ? lambda : 0.f;
    for (int d = 0; d < p->head_dim / 2 && d < 64; ++d)
        pa.inv_freq[d] = rope ? std::pow((double)rope_theta, -2.0 * d / (double)p->head_dim) : 0.0;
    pa.qm = (const uint16_t*)q_main; pa.km = (const uint16_t*)k_main; pa.vm = (const uint16_t*)v_main;
    pa.qs = (const uint16_t*)q_summ; pa.ks = (const uint16_t*)k_summ; pa.vs = (const uint16_t*)v_summ;
    pa.q_st = p->q_stride_tok; pa.q_sh = p->q_stride_head; pa.k_st = p->k_stride_tok; pa.k_sh = p->k_stride_head;
    pa.v_st = p->v_stride_tok; pa.v_sh = p->v_stride_head;
    pa.to_streams = 1;
    pa.qt = a.qt; pa.kt = a.kt; pa.vt = a.vt; pa.ks_out = a.ks; pa.vs_out = a.vs; pa.qs_out = qs;
    pa.text_rows = hs.text_rows; pa.summ_rows = hs.summ_rows;
    int64_t max_aug_len = 0;
    for (const SeqInfo& sq : hs.seqs) max_aug_len = std::max<int64_t>(max_aug_len, (int64_t)sq.n_text + sq.n_summ);
    cudaError_t e;
    if ((e = launch_zero_stream_pads(pa, p->num_seqs, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = launch_prep(pa, max_aug_len, p->num_seqs, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 2;
    if (a.m > 0 && a.max_n_summ > 0) {
        if ((e = launch_summary_streams(a, qs, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }
    if (ctx->timing) cudaEventRecord(ctx->ev0, stream);
    FwdMaps maps;
    if ((rc = prepare_text(ctx, a, p->flags, maps)) != KSA_OK) return rc;
    if ((rc = launch_text(ctx, a, p->flags, maps, stream)) != KSA_OK) return rc;
    if (ctx->timing) { cudaEventRecord(ctx->ev1, stream); ctx->timing_valid = true; }
    return KSA_OK;
}

struct StagingLayout { size_t q, k, v, out, lse, ws, ws_bytes, total; };
static int staging_layout(const ksa_params* p, StagingLayout& s)
{
    HostSchedule hs;
    build_layout(p, hs);
    const size_t D2 = (size_t)p->head_dim * 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 1024); return o; };
    s.q = take((size_t)hs.total_aug * p->num_q_heads * D2);
    s.k = take((size_t)hs.total_aug * p->num_kv_heads * D2);
    s.v = take((size_t)hs.total_aug * p->num_kv_heads * D2);
    s.out = take((size_t)hs.total_aug * p->num_q_heads * D2);
    s.lse = take((size_t)hs.total_aug * p->num_q_heads * 4);
    s.ws_bytes = workspace_layout(p, hs).total;
    s.ws = take(s.ws_bytes);
    s.total = off;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_host_staging_bytes(const ksa_ctx*, const ksa_params* p, size_t* bytes)
{
    if (!bytes) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    StagingLayout s;
    staging_layout(p, s);
    *bytes = s.total;
    return KSA_OK;
}

extern "C" __attribute__((visibility("default"))) int ksa_attn_fwd_host(ksa_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                                 void* out_host, float* lse_host, void* staging, size_t staging_bytes,
                                 const ksa_params* p, void* cuda_stream)
{
    if (!ctx || !q_host || !k_host || !v_host || !out_host || !lse_host) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    StagingLayout s;
    staging_layout(p, s);
    if (!staging || staging_bytes < s.total || ((uintptr_t)staging & 255)) return KSA_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* d = (char*)staging;
    const size_t D2 = (size_t)p->head_dim * 2;
    ksa_params pc = *p;   // contiguous device images
    pc.q_stride_tok = pc.o_stride_tok = (int64_t)p->num_q_heads * p->head_dim;
    pc.k_stride_tok = pc.v_stride_tok = (int64_t)p->num_kv_heads * p->head_dim;
    pc.q_stride_head = pc.k_stride_head = pc.v_stride_head = pc.o_stride_head = p->head_dim;

    // Upload, compute and download overlap: the query tiles are cut into row chunks in sequence
    // order.  A chunk's rows of q, k, v are contiguous on the host; its text rows only need keys at
    // or before their own position (Eq. 3) and its summary rows only their own chunk, all of which
    // earlier stages have already uploaded and packed; its rows of out are contiguous too.
    // Stage c: copy-in stream uploads chunk c -> caller's stream packs it, runs its summary rows and
    // its share of the work list -> copy-out stream downloads its out / lse rows.
    if ((rc = ensure_schedule(ctx, &pc, true, kHostPipelineChunks)) != KSA_OK) return rc;
    const HostSchedule& hs = ctx->sched;
    const WorkspaceLayout wl = workspace_layout(&pc, hs);
    cudaError_t e;
    if (!ctx->s_in) {
        if ((e = cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(ctx, e);
    }
    while (ctx->ev_in.size() < hs.chunks.size()) {
        cudaEvent_t a0, a1;
        if ((e = cudaEventCreateWithFlags(&a0, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = cudaEventCreateWithFlags(&a1, cudaEventDisableTiming)) != cudaSuccess) { cudaEventDestroy(a0); return cuda_fail(ctx, e); }
        ctx->ev_in.push_back(a0); ctx->ev_done.push_back(a1);
    }
    KernelArgs a = make_args(ctx, &pc, d + s.q, d + s.k, d + s.v, d + s.out, (float*)(d + s.lse), d + s.ws, wl);
    FwdMaps maps;
    if ((rc = prepare_text(ctx, a, p->flags, maps)) != KSA_OK) return rc;
    // the copy-in stream starts after whatever the caller queued before this call
    if ((e = cudaEventRecord(ctx->ev_start, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamWaitEvent(ctx->s_in, ctx->ev_start, 0)) != cudaSuccess) return cuda_fail(ctx, e);
    const size_t q_row = (size_t)p->num_q_heads * D2, kv_row = (size_t)p->num_kv_heads * D2;
    const WorkItem* work_base = a.work;
    for (size_t ci = 0; ci < hs.chunks.size(); ++ci) {
        const RowChunk& c = hs.chunks[ci];
        const size_t r0 = (size_t)c.aug0, nr = (size_t)(c.aug1 - c.aug0);
        if (nr > 0) {
            if ((e = cudaMemcpyAsync(d + s.q + r0 * q_row, (const char*)q_host + r0 * q_row, nr * q_row, cudaMemcpyHostToDevice, ctx->s_in)) != cudaSuccess) return cuda_fail(ctx, e);
            if ((e = cudaMemcpyAsync(d + s.k + r0 * kv_row, (const char*)k_host + r0 * kv_row, nr * kv_row, cudaMemcpyHostToDevice, ctx->s_in)) != cudaSuccess) return cuda_fail(ctx, e);
            if ((e = cudaMemcpyAsync(d + s.v + r0 * kv_row, (const char*)v_host + r0 * kv_row, nr * kv_row, cudaMemcpyHostToDevice, ctx->s_in)) != cudaSuccess) return cuda_fail(ctx, e);
        }
        if ((e = cudaEventRecord(ctx->ev_in[ci], ctx->s_in)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = cudaStreamWaitEvent(stream, ctx->ev_in[ci], 0)) != cudaSuccess) return cuda_fail(ctx, e);
        a.r_seq = c.seq;
        a.r_text0 = c.text0; a.r_text1 = c.text1;
        a.r_summ0 = c.summ0; a.r_summ1 = c.summ1; a.r_summq1 = c.summq1;
        if ((e = launch_pack(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
        // The last summary tile this stage's text rows visit may reach past the rows packed so far
        // (those belong to later stages and are masked out).  Their V rows must still be finite,
        // or 0 * V would poison the accumulators: clear them up to the tile boundary.
        {
            const SeqInfo& sq = hs.seqs[c.seq];
            const int64_t z0 = c.summ1, z1 = std::min<int64_t>(sq.summ_pad, round_up(c.summ1, kTileN));
            if (z1 > z0) {
                char* vs_rows = (char*)a.vs + ((size_t)sq.summ_off + (size_t)z0) * D2;
                if ((e = cudaMemset2DAsync(vs_rows, (size_t)hs.summ_rows * D2, 0, (size_t)(z1 - z0) * D2, (size_t)p->num_kv_heads,
                                           stream)) != cudaSuccess) return cuda_fail(ctx, e);
            }
        }
        if (a.m > 0 && c.summq1 > c.summ0) {
            if ((e = launch_summary(a, stream)) != cudaSuccess) return cuda_fail(ctx, e);
            ctx->launches += 1;
        }
        a.work = work_base + c.work_off;
        a.num_work = (int32_t)c.work_cnt;
        if ((rc = launch_text(ctx, a, p->flags, maps, stream)) != KSA_OK) return rc;
        if ((e = cudaEventRecord(ctx->ev_done[ci], stream)) != cudaSuccess) return cuda_fail(ctx, e);
        if ((e = cudaStreamWaitEvent(ctx->s_out, ctx->ev_done[ci], 0)) != cudaSuccess) return cuda_fail(ctx, e);
        if (nr > 0) {
            if ((e = cudaMemcpyAsync((char*)out_host + r0 * q_row, d + s.out + r0 * q_row, nr * q_row, cudaMemcpyDeviceToHost, ctx->s_out)) != cudaSuccess) return cuda_fail(ctx, e);
            // lse is [heads, total rows]: one strip of nr columns per head
            const size_t pitch = (size_t)hs.total_aug * 4;
            if ((e = cudaMemcpy2DAsync((char*)lse_host + r0 * 4, pitch, d + s.lse + r0 * 4, pitch, nr * 4, (size_t)p->num_q_heads,
                                       cudaMemcpyDeviceToHost, ctx->s_out)) != cudaSuccess) return cuda_fail(ctx, e);
        }
    }
    if ((e = cudaStreamSynchronize(ctx->s_out)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(ctx, e);
    return KSA_OK;
}
