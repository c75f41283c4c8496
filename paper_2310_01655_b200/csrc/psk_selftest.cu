// Self-test of the bounded device-side wait (see include/psk.h: psk_selftest_wait_timeout).
#include "psk_internal.cuh"
#include "tc_prims.cuh"

namespace psk {
namespace {

constexpr int kErrSelfTest = 99;

// One CTA of 128 threads waits on an mbarrier that nobody arrives at, through the same bounded
// wait the tensor-core kernels use.  The wait gives up after `limit_ns`, records its code in the
// workspace's status word and raises the CTA's give-up flag; a second wait on the same barrier
// must then come back at once.  out[0] = nanoseconds the first wait took (thread 0),
// out[1] = nanoseconds the second one took, out[2] = threads whose first wait returned false,
// out[3] = threads whose second wait returned false.  Nothing traps, nothing spins without a bound.
__global__ void __launch_bounds__(128) wait_timeout_kernel(int* status, unsigned long long limit_ns,
                                                           unsigned long long* out) {
    __shared__ uint64_t bar;
    __shared__ int failed[2];
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::cta_giveup_init();
        tc::mbar_fence_init();
        failed[0] = failed[1] = 0;
    }
    __syncthreads();
    const uint64_t t0 = tc::globaltimer_ns();
    const bool first = tc::mbar_wait_slow(tc::smem_u32(&bar), 0, status, kErrSelfTest, limit_ns);
    const uint64_t t1 = tc::globaltimer_ns();
    const bool second = tc::mbar_wait_slow(tc::smem_u32(&bar), 0, status, kErrSelfTest, limit_ns);
    const uint64_t t2 = tc::globaltimer_ns();
    if (!first) atomicAdd(&failed[0], 1);
    if (!second) atomicAdd(&failed[1], 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        out[0] = t1 - t0; out[1] = t2 - t1;
        out[2] = (unsigned long long)failed[0]; out[3] = (unsigned long long)failed[1];
    }
}

}  // namespace
}  // namespace psk

extern "C" int psk_selftest_wait_timeout(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* stream) {
    using namespace psk;
    if (!workspace || workspace_bytes < kStatusBytes || (reinterpret_cast<uintptr_t>(workspace) % kAlign))
        return PSK_ERR_WORKSPACE;
    if (limit_ns == 0 || limit_ns > 100000000ull) return PSK_ERR_INVALID_ARG;      // at most 0.1 s
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(workspace, 0, kStatusBytes, s) != cudaSuccess) return PSK_ERR_CUDA;
    // the status word is the first int; the report goes 64 bytes further on, inside the status block
    wait_timeout_kernel<<<1, 128, 0, s>>>(reinterpret_cast<int*>(workspace), limit_ns,
                                          reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + 64));
    return cudaGetLastError() == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}
