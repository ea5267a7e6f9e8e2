// Stand-alone cross-CTA merge for calls with many draft rows: one CTA per group of rows, so the merge
// of M rows runs on M / 8 SMs at once instead of on the last head CTA alone.
#include "vt_common.cuh"
#include "vt_launch.h"

namespace vt {

constexpr int kMergeThreads = 256;
constexpr int kMergeRowsPerCta = kMergeThreads / 32;

__global__ void __launch_bounds__(kMergeThreads) merge_kernel(const HeadOut o, int P, uint32_t stage_bytes) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    grid_dependency_wait();            // the head kernel's records must be complete
    __syncthreads();
    const int m_begin = blockIdx.x * kMergeRowsPerCta;
    const int m_count = min(kMergeRowsPerCta, o.M - m_begin);
    merge_rows(o, P, m_begin, m_count, smem, stage_bytes, smem_u32(&bar));
}

vt_status launch_merge(const HeadOut& o, int P, cudaStream_t st) {
    const int KS = ws_slots(o.k);
    const size_t cand = (size_t)(kMergeThreads / 32) * kMergeCand * 8;
    const size_t one_row = (size_t)P * (KS * 8 + 16);
    size_t want = (size_t)P * ((size_t)kMergeRowsPerCta * KS * 8 + 16);
    const size_t cap = 160 * 1024;
    if (want > cap) want = std::max(one_row, cap / one_row * one_row);
    want += cand;
    if (want > (size_t)kMaxDynSmem - 1024) return VT_ERR_UNSUPPORTED;
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(merge_kernel), (int)(kMaxDynSmem - 1024), &smem_configured); rc != VT_OK)
        return rc;
    const int grid = (o.M + kMergeRowsPerCta - 1) / kMergeRowsPerCta;
    cudaError_t e = launch_pdl(merge_kernel, grid, kMergeThreads, want, st, o, P, (uint32_t)want);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// Row-wise merge of the row-major records (the few-draft-rows kernel with more than 16 draft rows): one warp per
// draft row, so all rows merge at once on M / 8 SMs instead of one after the other in the warps that own them.
__global__ void __launch_bounds__(kMergeThreads) merge_rowmajor_kernel(const HeadOut o, int P) {
    grid_dependency_wait();            // the head kernel's records must be complete
    const int m = blockIdx.x * kMergeRowsPerCta + (threadIdx.x >> 5);
    if (m < o.M) merge_row_global(o, P, m);
}

vt_status launch_merge_rowmajor(const HeadOut& o, int P, cudaStream_t st) {
    const int grid = (o.M + kMergeRowsPerCta - 1) / kMergeRowsPerCta;
    cudaError_t e = launch_pdl(merge_rowmajor_kernel, grid, kMergeThreads, 0, st, o, P);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

}  // namespace vt
