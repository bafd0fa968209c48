// ksa_attn_fwd_noalloc: the KSA forward pass for callers that must not allocate device
// memory.  Its scratch (status word, sequence table, work list, packed Q/K/V streams)
// lives in one file-scope __device__ array of fixed size instead of a caller workspace
// and a context's cudaMalloc'd tables.
#include <algorithm>
#include <cstring>
#include <mutex>

#include "../../include/ksa.h"
#include "ksa_host.h"
#include "ksa_launch.h"

using namespace ksa;

namespace {

// Every GPU that loads the library keeps these bytes resident until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)KSA_NOALLOC_MAX_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    unsigned char* scratch = nullptr;   // DEVICE address of g_static_scratch on that device
    int num_sms = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// Once per device, with that device current: resolve the DEVICE address of the scratch
// array (in host code the array's name is only a handle, not an address a kernel may use).
int setup_current_device(int* device_out, DeviceSetup** setup_out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return KSA_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return KSA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[dev];
    if (!s.ready) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return KSA_ERR_CUDA;
        if (major != 10) return KSA_ERR_UNSUPPORTED;
        if (cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return KSA_ERR_CUDA;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return KSA_ERR_CUDA;
        s.scratch = (unsigned char*)ptr;
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
                q != cudaDriverEntryPointSuccess || !fn)
                return KSA_ERR_CUDA;
            g_encode = (EncodeTiledFn)fn;
        }
        if (setup_text_tc() != cudaSuccess) return KSA_ERR_CUDA;
        s.ready = true;
    }
    *device_out = dev;
    *setup_out = &s;
    return KSA_OK;
}

int encode_map(CUtensorMap* map, void* base, int D, int64_t rows, int H)
{
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)H};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kTileN, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KSA_OK : KSA_ERR_CUDA;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

// The status word of the bounded waits is the first word of the scratch array; no context is involved, so it has
// its own reader (a blocking 4-byte copy: allocates nothing).
extern "C" __attribute__((visibility("default")))
int ksa_noalloc_last_device_status(int32_t* status)
{
    if (!status) return KSA_ERR_INVALID_ARG;
    int dev = -1;
    DeviceSetup* setup = nullptr;
    int rc = setup_current_device(&dev, &setup);
    if (rc != KSA_OK) return rc;
    if (cudaMemcpy(status, setup->scratch, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return KSA_ERR_CUDA;
    return *status != 0 ? KSA_ERR_TIMEOUT : KSA_OK;
}

extern "C" __attribute__((visibility("default")))
int ksa_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* out, float* lse,
                         const ksa_params* p, void* cuda_stream)
{
    if (!q || !k || !v || !out || !lse) return KSA_ERR_INVALID_ARG;
    int rc = validate(p);
    if (rc != KSA_OK) return rc;
    if ((rc = validate_strides(p)) != KSA_OK) return rc;
    const uintptr_t ptrs[5] = {(uintptr_t)q, (uintptr_t)k, (uintptr_t)v, (uintptr_t)out, (uintptr_t)lse};
    for (int i = 0; i < 5; ++i) if (ptrs[i] & 15) return KSA_ERR_INVALID_ARG;

    // host-side schedule (host heap only)
    HostSchedule hs;
    try {
        build_layout(p, hs);
        build_schedule(p, hs);
    } catch (const std::bad_alloc&) { return KSA_ERR_NOMEM; }
    const WorkspaceLayout wl = workspace_layout(p, hs);

    // carve the static scratch: [status | sequence table | work list | packed streams]
    const size_t off_status = 0;
    const size_t off_seqs = 256;
    const size_t off_work = align_up(off_seqs + hs.seqs.size() * sizeof(SeqInfo), 256);
    const size_t off_ws = align_up(off_work + std::max<size_t>(1, hs.work.size()) * sizeof(WorkItem), 1024);
    const size_t need = off_ws + wl.total;
    if (need > kStaticScratchBytes) return KSA_ERR_WORKSPACE;   // problem too large for the static scratch

    int dev = -1;
    DeviceSetup* setup = nullptr;
    if ((rc = setup_current_device(&dev, &setup)) != KSA_OK) return rc;
    unsigned char* base = setup->scratch;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    // The array keeps the previous call's contents.  The status word must start at zero;
    // the tables are rewritten here and the pack kernel rewrites every stream row it pads.
    if (cudaMemsetAsync(base + off_status, 0, 256, stream) != cudaSuccess) return KSA_ERR_CUDA;
    if (cudaMemcpyAsync(base + off_seqs, hs.seqs.data(), hs.seqs.size() * sizeof(SeqInfo),
                        cudaMemcpyHostToDevice, stream) != cudaSuccess) return KSA_ERR_CUDA;
    if (!hs.work.empty() &&
        cudaMemcpyAsync(base + off_work, hs.work.data(), hs.work.size() * sizeof(WorkItem),
                        cudaMemcpyHostToDevice, stream) != cudaSuccess) return KSA_ERR_CUDA;
    // the host tables die with this frame: make sure the copies have read them
    if (cudaStreamSynchronize(stream) != cudaSuccess) return KSA_ERR_CUDA;

    char* ws = (char*)(base + off_ws);
    KernelArgs a{};
    a.seqs = (const SeqInfo*)(base + off_seqs);
    a.work = (const WorkItem*)(base + off_work);
    a.num_seqs = p->num_seqs; a.num_work = (int32_t)hs.work.size();
    a.k = p->chunk_len; a.m = p->summaries_per_chunk; a.C = p->window_chunks;
    a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads; a.D = p->head_dim;
    a.flags = p->flags;
    a.scale = p->softmax_scale;
    a.scale_log2 = p->softmax_scale * 1.4426950408889634f;
    a.total_aug = hs.total_aug; a.text_rows = hs.text_rows; a.summ_rows = hs.summ_rows;
    a.max_text_pad = hs.max_text_pad; a.max_summ_pad = hs.max_summ_pad; a.max_n_summ = hs.max_n_summ;
    a.r_seq = -1;
    a.q = (const uint16_t*)q; a.kx = (const uint16_t*)k; a.v = (const uint16_t*)v;
    a.out = (uint16_t*)out; a.lse = lse;
    a.q_st = p->q_stride_tok; a.q_sh = p->q_stride_head; a.k_st = p->k_stride_tok; a.k_sh = p->k_stride_head;
    a.v_st = p->v_stride_tok; a.v_sh = p->v_stride_head; a.o_st = p->o_stride_tok; a.o_sh = p->o_stride_head;
    a.qt = (uint16_t*)(ws + wl.qt); a.kt = (uint16_t*)(ws + wl.kt); a.vt = (uint16_t*)(ws + wl.vt);
    a.ks = (uint16_t*)(ws + wl.ks); a.vs = (uint16_t*)(ws + wl.vs);
    a.status = (int32_t*)(base + off_status);

    if (launch_pack(a, stream) != cudaSuccess) return KSA_ERR_CUDA;
    if (a.m > 0 && a.max_n_summ > 0 && launch_summary(a, stream) != cudaSuccess) return KSA_ERR_CUDA;
    if (p->flags & KSA_FLAG_REFERENCE_KERNEL) {
        if (launch_text_ref(a, stream) != cudaSuccess) return KSA_ERR_CUDA;
    } else {
        TextMaps maps;
        if ((rc = encode_map(&maps.qt, a.qt, a.D, a.text_rows, a.Hq)) != KSA_OK) return rc;
        if ((rc = encode_map(&maps.kt, a.kt, a.D, a.text_rows, a.Hkv)) != KSA_OK) return rc;
        if ((rc = encode_map(&maps.vt, a.vt, a.D, a.text_rows, a.Hkv)) != KSA_OK) return rc;
        if ((rc = encode_map(&maps.ks, a.ks, a.D, a.summ_rows, a.Hkv)) != KSA_OK) return rc;
        if ((rc = encode_map(&maps.vs, a.vs, a.D, a.summ_rows, a.Hkv)) != KSA_OK) return rc;
        if (launch_text_tc(a, maps, setup->num_sms, stream) != cudaSuccess) return KSA_ERR_CUDA;
    }
    return KSA_OK;
}
