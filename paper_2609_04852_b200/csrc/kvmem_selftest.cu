// kvmem_selftest_wait_timeout: runs the bounded mbarrier wait of this library's kernels to its limit, on purpose.
//
// Every kernel here waits for its TMA copies and for its other warps with ptx::mbar_wait, which gives up after a time
// limit, records KVMEM_E_TIMEOUT in the pool's status word and lets the kernel return.  That path is what keeps a
// lost copy or a logic error from hanging the GPU, and nothing in a healthy run ever takes it.  This entry point
// takes it: one warp waits, with a short caller-given limit, for a barrier that nobody arrives at, then reports and
// returns like any other kernel would.  Nothing faults, traps or spins without bound.  The paper has no counterpart.
#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"

namespace kvmem {

__global__ void __launch_bounds__(32)
selftest_wait_kernel(int32_t* __restrict__ status, unsigned long long limit_ns, unsigned long long* __restrict__ waited_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    const uint64_t t0 = ptx::globaltimer_ns();
    const bool ok = ptx::mbar_wait_limited(&bar, 0u, limit_ns);      // phase 0 never completes: no arrival is ever made
    const uint64_t t1 = ptx::globaltimer_ns();
    if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0) {
        atomicExch(status, (int)KVMEM_E_TIMEOUT);
        if (waited_ns) *waited_ns = t1 - t0;
    }
}

}  // namespace kvmem

using namespace kvmem;

extern "C" int kvmem_selftest_wait_timeout(kvmem_pool_t* pool, uint32_t limit_us, uint64_t* waited_ns, void* stream) {
    if (!pool || pool->magic != kMagic) { set_error("pool handle is null or stale"); return KVMEM_E_STATE; }
    if (limit_us < 1 || limit_us > 100000) { set_error("limit_us must be in [1, 100000]"); return KVMEM_E_INVALID; }
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device != pool->cfg.device) {
        (void)cudaGetLastError();
        set_error("the pool lives on device %d but device %d is current", pool->cfg.device, device);
        return KVMEM_E_STATE;
    }
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(pool->status_dev, (unsigned long long)limit_us * 1000ull,
                                                            reinterpret_cast<unsigned long long*>(waited_ns));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("self-test kernel launch: %s", cudaGetErrorString(e)); return KVMEM_E_CUDA; }
    return KVMEM_OK;
}
