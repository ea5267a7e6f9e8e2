// Test-only kernels behind the C boundary: they exercise the failure path and the stream-order contract of the
// head kernels without faulting, trapping or hanging anything.
#include "vt_launch.h"

namespace vt {

// Posts a transaction of 16 bytes on a fresh mbarrier and issues no copy, so the phase can never complete; the
// bounded wait gives up after `limit_ns`, the time-out bit is set and the kernel returns.
__global__ void timeout_probe_kernel(WsHeader* hdr, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_mbar_init();
        mbar_arrive_expect_tx(b, 16u);
        if (!mbar_wait(b, 0u, limit_ns)) atomicOr(&hdr->status, kStatusTimeout);
    }
}

// Lets the next kernel in the stream start (programmatic dependent launch), idles, then copies.
__global__ void late_copy_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, size_t n16,
                                 unsigned long long delay_ns) {
    grid_launch_dependents();
    const unsigned long long t0 = global_timer_ns();
    while (global_timer_ns() - t0 < delay_ns) { }       // bounded by delay_ns (at most 10 ms)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

}  // namespace vt

using namespace vt;

extern "C" vt_status vt_test_timeout_probe(void* workspace, int limit_us, void* stream) {
    reset_launch_count();
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return VT_ERR_WORKSPACE;
    if (limit_us < 1 || limit_us > 1000000) return VT_ERR_SHAPE;
    timeout_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<WsHeader*>(workspace),
                                                            (unsigned long long)limit_us * 1000ull);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

extern "C" vt_status vt_test_late_copy(void* dst, const void* src, size_t n_bytes, int delay_us, void* stream) {
    reset_launch_count();
    if (!dst || !src) return VT_ERR_NULL;
    if (n_bytes == 0 || n_bytes % 16 != 0 || delay_us < 0 || delay_us > 10000) return VT_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(dst) & 15) || (reinterpret_cast<uintptr_t>(src) & 15)) return VT_ERR_ALIGN;
    const size_t n16 = n_bytes / 16;
    const int grid = (int)std::max<size_t>(1, std::min<size_t>((n16 + 255) / 256, 64));
    late_copy_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(reinterpret_cast<uint4*>(dst),
                                                            reinterpret_cast<const uint4*>(src), n16,
                                                            (unsigned long long)delay_us * 1000ull);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}
