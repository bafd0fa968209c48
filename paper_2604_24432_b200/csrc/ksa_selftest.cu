// Self-test of the bounded-wait path: a one-warp kernel waits, with the same helper the attention kernels use, on an
// mbarrier that nothing ever arrives at, with a short cycle limit.  The wait must give up, record its code in the
// context's status word, raise the abort flag (a second wait then returns at once) and the kernel must return.
#include "../../include/ksa.h"
#include "ksa_host.h"
#include "ksa_launch.h"
#include "ksa_ptx.cuh"
#include "ksa_wait.cuh"

namespace ksa {

__global__ void __launch_bounds__(32, 1) ksa_wait_selftest_kernel(int32_t* status, int32_t* report, long long limit_cycles)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ uint32_t abort_flag;
    const uint32_t bar = ptx::smem_u32(&bar_storage);
    const uint32_t abort_addr = ptx::smem_u32(&abort_flag);
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar, 1);
        st_shared_u32(abort_addr, 0u);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool first = bounded_wait(bar, 0, abort_addr, status, kStatusWaitTest, limit_cycles);    // nobody arrives
        const long long t1 = clock64();
        const bool second = bounded_wait(bar, 0, abort_addr, status, kStatusWaitQFull, limit_cycles);  // sees the abort flag
        const long long t2 = clock64();
        report[0] = first ? 1 : 0;
        report[1] = second ? 1 : 0;
        report[2] = (int32_t)ld_shared_u32(abort_addr);
        report[3] = (int32_t)((t1 - t0) >> 10);        // kilo-cycles spent in the wait that gave up
        report[4] = (int32_t)((t2 - t1) >> 10);
    }
}

}  // namespace ksa

extern "C" __attribute__((visibility("default")))
int ksa_selftest_bounded_wait(ksa_ctx* ctx, int64_t limit_cycles, int32_t* report5_device, void* cuda_stream)
{
    if (!ctx || !report5_device || limit_cycles < 1 || limit_cycles > (1ll << 31)) return KSA_ERR_INVALID_ARG;
    ksa::ksa_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(ksa_ctx_status_word(ctx), report5_device, (long long)limit_cycles);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ksa_ctx_cuda_fail(ctx, (int)e);
    ksa_ctx_add_launches(ctx, 1);
    return KSA_OK;
}
