// Test hook for the failure path of the tensor-core kernels: one tiny kernel that runs the same bounded
// wait as they do on a barrier nobody arrives at.  No tensor memory, no TMA, no GEMM: the wait runs out
// after the limit the caller gives (a millisecond or so), the kernel records the code and returns, and the
// context stays usable.

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr uint32_t kSelftestSite = 15;

__global__ void __launch_bounds__(32)
wait_timeout_kernel(unsigned long long limit_ns, uint32_t* dev_status)
{
    __shared__ alignas(8) unsigned long long bar_storage;
    __shared__ uint32_t abort_flag;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    pdl_wait_for_predecessors();
    pdl_release_successors();
    // phase 0 never completes: nobody arrives.  Every lane waits, as the warps of the real kernels do.
    bool ok = mbar_wait_limit(bar, 0u, &abort_flag, dev_status, kSelftestSite, limit_ns);
    ok = __all_sync(0xFFFFFFFFu, ok);
    (void)ok;
}

}  // namespace
}  // namespace elsa

using namespace elsa;

extern "C" elsa_status elsa_selftest_wait_timeout(unsigned long long limit_ns, uint32_t* dev_status, void* stream)
{
    if (!dev_status) return fail(ELSA_ERR_NULL, "dev_status must not be NULL");
    if (limit_ns == 0 || limit_ns > 100000000ull)
        return fail(ELSA_ERR_SHAPE, "limit of %llu ns is outside 1 ns .. 100 ms", limit_ns);
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    launch_pdl(wait_timeout_kernel, dim3(1), dim3(32), 0, (cudaStream_t)stream, 1, limit_ns, dev_status);
    return launched("wait_timeout (self-test)");
}
