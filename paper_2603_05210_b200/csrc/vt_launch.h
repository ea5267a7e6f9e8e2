// Host-side glue shared by the kernel launchers and the C entry points.
#pragma once

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <utility>

#include "vt_common.cuh"

namespace vt {

constexpr int kMaxDynSmem = 227 * 1024;   // opt-in dynamic shared memory per CTA on sm_100

// One draft-head call after validation (all pointers device).
struct HeadCall {
    const void* h;
    const void* W;
    int d, M, Vt;
    HeadOut out;
    int static_weights;   // 1: the caller declared W_trim constant; its stream may start ahead of the dependency wait
};

vt_status cuda_fail(cudaError_t e);        // records e for vt_last_cuda_error, returns VT_ERR_CUDA
vt_status driver_fail(int cu_result);
void count_launch();
void reset_launch_count();                  // every entry point starts with it, so vt_last_launch_count is per call
vt_status ensure_max_dyn_smem(const void* kernel, int bytes, std::atomic<unsigned long long>* done_mask);
vt_status device_sm_count(int* sms);

// Both head kernels split the vocabulary rows over `*grid` persistent CTAs (one per SM at most); the
// merge needs to know how many CTAs wrote records.
inline int head_grid(int sms, int Vt, int min_rows_per_cta = 1) {
    const int by_rows = (Vt + min_rows_per_cta - 1) / min_rows_per_cta;
    return std::max(1, std::min(std::min(sms, kMaxParts), by_rows));
}

// Launches with programmatic stream serialization (see grid_dependency_wait in vt_common.cuh).
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// The same as clusters of two CTAs (the grid must be even).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster2(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

bool gemv_supports(int d);
vt_status launch_head_gemv(const HeadCall& c, cudaStream_t st, int* grid);
vt_status launch_head_mma(const HeadCall& c, cudaStream_t st, int* grid);
// any M, in passes of 128 draft rows (256 when every CTA has one tile of the vocabulary); a single pass of at most
// 16 rows with the warp-per-row epilogue merges row by row in the same launch (one arrival ticket per draft row),
// everything else launches the row-wise merge kernel after itself; VT_ERR_UNSUPPORTED when the shape does not fit
vt_status launch_head_mma_small(const HeadCall& c, cudaStream_t st, int* grid);
vt_status launch_merge_rowmajor(const HeadOut& o, int P, cudaStream_t st);   // one warp per draft row over the row-major records

vt_status launch_compact(const void* W_full, int V_full, int d, const int32_t* keep_ids, int V_trim,
                         void* W_trim, cudaStream_t st);
vt_status launch_vocab_maps(const int32_t* keep_ids, int V_trim, int V_full, int32_t* d2t_offsets,
                            unsigned char* t2d_mask, cudaStream_t st);
vt_status launch_remap(const int32_t* draft_ids, const int32_t* d2t, int64_t n, int V_trim,
                       int32_t* target_ids, cudaStream_t st);

constexpr int kTreeSelectMaxPairs = 8192;   // M * k pairs one tree-selection call takes
vt_status launch_tree_select(const float* logprobs, const int32_t* target_ids, const float* parent, int M, int k, int T,
                             int32_t* out_rows, int32_t* out_slots, int32_t* out_tokens, float* out_scores, cudaStream_t st);

// Coverage workspace: one 256-byte line of counters, then the membership bitmap.
struct CoverageCounters {
    unsigned long long covered;
    unsigned int out_of_range;
    unsigned int duplicates;
    unsigned int pad[60];
};
static_assert(sizeof(CoverageCounters) == 256, "one line");
inline size_t coverage_bitmap_words(int V_full) { return ((size_t)V_full + 31) / 32; }
vt_status launch_keep_bitmap(const int32_t* keep_ids, int V_trim, int V_full, void* workspace, cudaStream_t st);
vt_status launch_coverage_count(const int32_t* token_ids, int64_t N, int V_full, void* workspace, cudaStream_t st);
// one launch: every CTA builds the bitmap in its shared memory (only where coverage_fused_fits)
bool coverage_fused_fits(int V_full);
vt_status launch_coverage_fused(const int32_t* token_ids, int64_t N, const int32_t* keep_ids, int V_trim, int V_full,
                                void* workspace, cudaStream_t st);

}  // namespace vt
