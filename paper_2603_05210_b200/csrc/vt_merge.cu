// Stand-alone cross-CTA merge for calls with many draft rows: one warp per draft row, so the rows merge at once
// on M / 8 SMs instead of one after the other in the warps that produced them.
#include "vt_common.cuh"
#include "vt_launch.h"

namespace vt {

constexpr int kMergeThreads = 256;
constexpr int kMergeRowsPerCta = kMergeThreads / 32;

__global__ void __launch_bounds__(kMergeThreads) merge_rowmajor_kernel(const HeadOut o, int P) {
    grid_dependency_wait();            // the head kernel's records must be complete
    const int m = blockIdx.x * kMergeRowsPerCta + (threadIdx.x >> 5);
    __shared__ unsigned long long cbuf[kMergeRowsPerCta][kMergeCap];
    if (m < o.M) merge_row_global(o, P, m, cbuf[threadIdx.x >> 5]);
}

vt_status launch_merge_rowmajor(const HeadOut& o, int P, cudaStream_t st) {
    const int grid = (o.M + kMergeRowsPerCta - 1) / kMergeRowsPerCta;
    cudaError_t e = launch_pdl(merge_rowmajor_kernel, grid, kMergeThreads, 0, st, o, P);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

}  // namespace vt
