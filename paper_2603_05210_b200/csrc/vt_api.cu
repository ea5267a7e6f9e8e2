// C entry points: argument checks on the host, path choice, launches.  See include/vt.h for the contract.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "vt_launch.h"

namespace vt {

static thread_local int g_last_cuda_error = 0;
static thread_local int g_launches = 0;

vt_status cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return VT_ERR_CUDA;
}
vt_status driver_fail(int cu_result) {
    g_last_cuda_error = cu_result;
    return VT_ERR_CUDA;
}
void count_launch() { ++g_launches; }
void reset_launch_count() { g_launches = 0; }

vt_status device_sm_count(int* sms) {
    static std::atomic<int> cached[64];       // zero-initialised; racing first calls store the same value
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        cached[dev].store(n, std::memory_order_relaxed);
    }
    *sms = n;
    return VT_OK;
}

// Raises a kernel's dynamic shared-memory limit once per device (an atomic bit per device: concurrent host
// threads may both make the call, which is harmless).
vt_status ensure_max_dyn_smem(const void* kernel, int bytes, std::atomic<unsigned long long>* done_mask) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
    const unsigned long long bit = 1ull << dev;
    if (done_mask->load(std::memory_order_acquire) & bit) return VT_OK;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return cuda_fail(e);
    done_mask->fetch_or(bit, std::memory_order_release);
    return VT_OK;
}

static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static vt_status check_head_args(const void* h, const void* W, const int32_t* d2t, int M, int d, int Vt, int k,
                                 const void* target_ids, const void* logprobs, const void* ws, size_t ws_bytes) {
    if (!h || !W || !d2t || !target_ids || !logprobs) return VT_ERR_NULL;
    if (d < 8 || d % 8 != 0 || M < 1 || Vt < 1 || k < 1 || k > Vt || k > VT_MAX_K) return VT_ERR_SHAPE;
    if (!aligned(h, 16) || !aligned(W, 16) || !aligned(d2t, 4) || !aligned(target_ids, 4) || !aligned(logprobs, 4))
        return VT_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < ws_total_bytes(M, k)) return VT_ERR_WORKSPACE;
    return VT_OK;
}

// Draft rows up to which a head kernel merges the per-CTA records itself (the warp that publishes a row last of
// all CTAs merges it); beyond that the row-wise merge kernel spreads the rows over many SMs.
constexpr int kFusedMergeMaxM = 16;

static HeadOut make_out(const int32_t* d2t, int M, int Vt, int k, int32_t* tid, float* lp, int32_t* did, float* lse,
                        float* logits, void* ws, int d2t_offsets = 0) {
    HeadOut o{};
    o.d2t = d2t;
    o.d2t_offsets = d2t_offsets;
    o.target_ids = tid;
    o.logprobs = lp;
    o.draft_ids = did;
    o.lse = lse;
    o.logits = logits;
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    o.hdr = reinterpret_cast<WsHeader*>(base);
    o.recs = reinterpret_cast<unsigned long long*>(base + kHeaderBytes);
    o.M = M;
    o.k = k;
    o.Vt = Vt;
    o.fused_merge = M <= kFusedMergeMaxM;
    return o;
}

// Automatic path choice, from measurements at d = 4096 over V_trim = 4096 .. 128256:
//  - the CUDA-core GEMV has the least fixed cost and keeps up with the stream for one draft row: M = 1 always,
//    and M = 2 while the weights are under 80 MB, where fixed cost decides;
//  - the vocabulary-rows-on-lanes tensor-core kernel for everything else it can plan (passes of 128 draft rows);
//  - the draft-rows-on-lanes tensor-core kernel for what it declines (very large k times M, very large d).
static bool auto_prefers_gemv(int M, int d, int Vt) {
    if (!gemv_supports(d)) return false;
    const size_t w_bytes = (size_t)Vt * d * 2;
    return M == 1 || (M == 2 && w_bytes <= ((size_t)80 << 20));
}

static vt_status run_head(const HeadCall& c, cudaStream_t st, int path) {
    int grid = 0;
    vt_status r;
    bool merged = c.out.fused_merge != 0;     // the tensor-core kernels see to the merge themselves
    if (path == VT_PATH_GEMV) {
        r = launch_head_gemv(c, st, &grid);
    } else if (path == VT_PATH_MMA) {
        r = launch_head_mma(c, st, &grid);
        merged = true;
    } else if (path == VT_PATH_MMA_SMALL) {
        r = launch_head_mma_small(c, st, &grid);
        merged = true;
    } else if (path != VT_PATH_AUTO) {
        return VT_ERR_SHAPE;
    } else if (auto_prefers_gemv(c.M, c.d, c.Vt)) {
        r = launch_head_gemv(c, st, &grid);
    } else if ((r = launch_head_mma_small(c, st, &grid)) != VT_ERR_UNSUPPORTED) {
        merged = true;     // launched (or failed for a reason another path would not cure)
    } else {
        r = launch_head_mma(c, st, &grid);
        merged = true;
        if (r == VT_ERR_UNSUPPORTED && gemv_supports(c.d)) {
            r = launch_head_gemv(c, st, &grid);
            merged = c.out.fused_merge != 0;
        }
    }
    if (r != VT_OK) return r;
    if (!merged && !c.out.store_only) r = launch_merge_rowmajor(c.out, grid, st);
    return r;
}

}  // namespace vt

using namespace vt;

extern "C" {

const char* vt_strerror(vt_status s) {
    switch (s) {
        case VT_OK: return "ok";
        case VT_ERR_NULL: return "a required pointer is NULL";
        case VT_ERR_SHAPE: return "a size or shape argument is outside the supported range";
        case VT_ERR_ALIGN: return "a pointer is not aligned as required";
        case VT_ERR_RANGE: return "a keep id lies outside [0, V_full)";
        case VT_ERR_DUP: return "keep_ids names an id more than once";
        case VT_ERR_EMPTY: return "coverage of an empty token stream is undefined";
        case VT_ERR_WORKSPACE: return "workspace is NULL, misaligned or too small";
        case VT_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case VT_ERR_CUDA: return "a CUDA call failed";
        case VT_ERR_UNSUPPORTED: return "the forced path cannot run this shape";
    }
    return "unknown status";
}

int vt_last_cuda_error(void) { return g_last_cuda_error; }
int vt_last_launch_count(void) { return g_launches; }

vt_status vt_compact_head(const void* W_full, int V_full, int d, const int32_t* keep_ids, int V_trim, void* W_trim,
                          void* stream) {
    g_launches = 0;
    if (!W_full || !keep_ids || !W_trim) return VT_ERR_NULL;
    if (d < 8 || d % 8 != 0 || V_full < 1 || V_trim < 1 || V_trim > V_full) return VT_ERR_SHAPE;
    if (!aligned(W_full, 16) || !aligned(W_trim, 16) || !aligned(keep_ids, 4)) return VT_ERR_ALIGN;
    return launch_compact(W_full, V_full, d, keep_ids, V_trim, W_trim, (cudaStream_t)stream);
}

size_t vt_coverage_workspace_bytes(int V_full) {
    if (V_full < 1) return 0;
    size_t b = sizeof(CoverageCounters) + coverage_bitmap_words(V_full) * 4;
    return (b + 255) & ~(size_t)255;
}

static vt_status read_counters(void* workspace, cudaStream_t st, CoverageCounters* host) {
    cudaError_t e = cudaMemcpyAsync(host, workspace, sizeof(CoverageCounters), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

vt_status vt_validate_keep_ids(const int32_t* keep_ids, int V_trim, int V_full, void* workspace,
                               size_t workspace_bytes, void* stream) {
    g_launches = 0;
    if (!keep_ids) return VT_ERR_NULL;
    if (V_full < 1 || V_trim < 1) return VT_ERR_SHAPE;
    if (!aligned(keep_ids, 4)) return VT_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < vt_coverage_workspace_bytes(V_full))
        return VT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    vt_status r = launch_keep_bitmap(keep_ids, V_trim, V_full, workspace, st);
    if (r != VT_OK) return r;
    CoverageCounters c;
    r = read_counters(workspace, st, &c);
    if (r != VT_OK) return r;
    if (c.out_of_range) return VT_ERR_RANGE;
    if (c.duplicates) return VT_ERR_DUP;
    if (V_trim > V_full) return VT_ERR_SHAPE;   // unreachable for a valid set; kept for completeness
    return VT_OK;
}

size_t vt_workspace_bytes(int M, int k) {
    if (M < 1 || k < 1 || k > VT_MAX_K) return 0;
    return ws_total_bytes(M, k);
}

vt_status vt_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < kHeaderBytes) return VT_ERR_WORKSPACE;
    cudaError_t e = cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream);
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

vt_status vt_draft_head_path(const void* h, const void* W_trim, const int32_t* d2t, int M, int d, int V_trim, int k,
                             int32_t* target_ids, float* logprobs, int32_t* draft_ids, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream, int options) {
    g_launches = 0;
    vt_status r = check_head_args(h, W_trim, d2t, M, d, V_trim, k, target_ids, logprobs, workspace, workspace_bytes);
    if (r != VT_OK) return r;
    if (options & ~(VT_PATH_MASK | VT_HEAD_STATIC_WEIGHTS | VT_HEAD_D2T_OFFSETS)) return VT_ERR_SHAPE;
    HeadCall c{h, W_trim, d, M, V_trim,
               make_out(d2t, M, V_trim, k, target_ids, logprobs, draft_ids, lse, nullptr, workspace,
                        (options & VT_HEAD_D2T_OFFSETS) ? 1 : 0),
               (options & VT_HEAD_STATIC_WEIGHTS) ? 1 : 0};
    return run_head(c, (cudaStream_t)stream, options & VT_PATH_MASK);
}

vt_status vt_draft_head(const void* h, const void* W_trim, const int32_t* d2t, int M, int d, int V_trim, int k,
                        int32_t* target_ids, float* logprobs, int32_t* draft_ids, float* lse, void* workspace,
                        size_t workspace_bytes, void* stream) {
    return vt_draft_head_path(h, W_trim, d2t, M, d, V_trim, k, target_ids, logprobs, draft_ids, lse, workspace,
                              workspace_bytes, stream, VT_PATH_AUTO);
}

static inline size_t up256(size_t b) { return (b + 255) & ~(size_t)255; }

// Device address of a pinned, mapped host buffer (NULL for pageable memory).  A serving loop passes the same
// two output buffers every step, so each thread remembers the last few answers instead of asking the driver
// twice per call.  (A buffer that is freed and re-allocated at the same address with another kind of memory
// would be answered from the cache: the end-to-end call asks that its output buffers stay what they were.)
static void* mapped_device_pointer(const void* host) {
    struct Entry { const void* host; void* dev; };
    static thread_local Entry cache[4] = {};
    static thread_local int next = 0;
    for (const Entry& e : cache)
        if (e.host == host) return e.dev;
    cudaPointerAttributes at{};
    void* dev = nullptr;
    if (cudaPointerGetAttributes(&at, host) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer)
        dev = at.devicePointer;
    (void)cudaGetLastError();      // a pageable pointer makes the query fail on some drivers; that is not an error here
    cache[next] = Entry{host, dev};
    next = (next + 1) & 3;
    return dev;
}

size_t vt_host_workspace_bytes(int M, int d, int k) {
    if (M < 1 || k < 1 || k > VT_MAX_K || d < 8) return 0;
    return ws_total_bytes(M, k) + up256((size_t)M * d * 2) + 2 * up256((size_t)M * k * 4);
}

vt_status vt_draft_head_host(const void* h_host, const void* W_trim, const int32_t* d2t, int M, int d, int V_trim,
                             int k, int32_t* target_ids_host, float* logprobs_host, void* workspace,
                             size_t workspace_bytes, void* stream) {
    g_launches = 0;
    if (!h_host || !target_ids_host || !logprobs_host) return VT_ERR_NULL;
    if (d < 8 || d % 8 != 0 || M < 1 || k < 1 || k > VT_MAX_K) return VT_ERR_SHAPE;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < vt_host_workspace_bytes(M, d, k))
        return VT_ERR_WORKSPACE;
    unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
    const size_t head_ws = ws_total_bytes(M, k);
    void* h_dev = base + head_ws;
    int32_t* tid_dev = reinterpret_cast<int32_t*>(base + head_ws + up256((size_t)M * d * 2));
    float* lp_dev = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(tid_dev) + up256((size_t)M * k * 4));
    vt_status r = check_head_args(h_dev, W_trim, d2t, M, d, V_trim, k, tid_dev, lp_dev, workspace, head_ws);
    if (r != VT_OK) return r;
    cudaStream_t st = (cudaStream_t)stream;
    // Pinned host outputs are written by the merge directly (they are device-accessible under unified
    // addressing): no device-to-host copies.  Pageable outputs go through the staging buffers.
    int32_t* tid_out = tid_dev;
    float* lp_out = lp_dev;
    void* tid_mapped = mapped_device_pointer(target_ids_host);
    void* lp_mapped = mapped_device_pointer(logprobs_host);
    const bool direct = tid_mapped != nullptr && lp_mapped != nullptr;
    if (direct) {
        tid_out = reinterpret_cast<int32_t*>(tid_mapped);
        lp_out = reinterpret_cast<float*>(lp_mapped);
    }
    cudaError_t e = cudaMemcpyAsync(h_dev, h_host, (size_t)M * d * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
    HeadCall c{h_dev, W_trim, d, M, V_trim, make_out(d2t, M, V_trim, k, tid_out, lp_out, nullptr, nullptr, nullptr, workspace), 0};
    r = run_head(c, st, VT_PATH_AUTO);
    if (r != VT_OK) return r;
    if (!direct) {
        e = cudaMemcpyAsync(target_ids_host, tid_dev, (size_t)M * k * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaMemcpyAsync(logprobs_host, lp_dev, (size_t)M * k * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

vt_status vt_last_status(void* workspace, void* stream) {
    if (!workspace) return VT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    WsHeader* hdr = reinterpret_cast<WsHeader*>(workspace);
    unsigned int status = 0;
    cudaError_t e = cudaMemcpyAsync(&status, &hdr->status, 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (status) {
        e = cudaMemsetAsync(&hdr->status, 0, 4, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return (status & kStatusTimeout) ? VT_ERR_TIMEOUT : VT_OK;
}

vt_status vt_coverage_enqueue(const int32_t* token_ids, int64_t N, const int32_t* keep_ids, int V_trim, int V_full,
                              void* workspace, size_t workspace_bytes, void* stream) {
    g_launches = 0;
    if (!keep_ids || (!token_ids && N > 0)) return VT_ERR_NULL;
    if (V_full < 1 || V_trim < 1 || N < 0) return VT_ERR_SHAPE;
    if (N == 0) return VT_ERR_EMPTY;
    if (!aligned(token_ids, 4) || !aligned(keep_ids, 4)) return VT_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < vt_coverage_workspace_bytes(V_full))
        return VT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (coverage_fused_fits(V_full)) return launch_coverage_fused(token_ids, N, keep_ids, V_trim, V_full, workspace, st);
    vt_status r = launch_keep_bitmap(keep_ids, V_trim, V_full, workspace, st);
    if (r != VT_OK) return r;
    return launch_coverage_count(token_ids, N, V_full, workspace, st);
}

vt_status vt_coverage_result(void* workspace, int64_t N, uint64_t* covered_out, double* fraction_out, void* stream) {
    if (!workspace || !aligned(workspace, 256)) return VT_ERR_WORKSPACE;
    if (N < 1) return VT_ERR_EMPTY;
    CoverageCounters c;
    vt_status r = read_counters(workspace, (cudaStream_t)stream, &c);
    if (r != VT_OK) return r;
    if (covered_out) *covered_out = c.covered;
    if (fraction_out) *fraction_out = (double)c.covered / (double)N;
    return VT_OK;
}

vt_status vt_coverage(const int32_t* token_ids, int64_t N, const int32_t* keep_ids, int V_trim, int V_full,
                      uint64_t* covered_out, double* fraction_out, void* workspace, size_t workspace_bytes,
                      void* stream) {
    vt_status r = vt_coverage_enqueue(token_ids, N, keep_ids, V_trim, V_full, workspace, workspace_bytes, stream);
    if (r != VT_OK) return r;
    return vt_coverage_result(workspace, N, covered_out, fraction_out, stream);
}

vt_status vt_debug_logits(const void* h, const void* W_trim, int M, int d, int V_trim, float* logits, void* workspace,
                          size_t workspace_bytes, void* stream, int path) {
    g_launches = 0;
    if (!logits) return VT_ERR_NULL;
    if (!aligned(logits, 4)) return VT_ERR_ALIGN;
    // the epilogue still runs its top-1 bookkeeping; its outputs land in the tail of the workspace
    if (M < 1) return VT_ERR_SHAPE;
    const size_t head_ws = ws_total_bytes(M, 1);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < ws_total_bytes(M, 2)) return VT_ERR_WORKSPACE;
    unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
    int32_t* tid = reinterpret_cast<int32_t*>(base + head_ws);
    float* lp = reinterpret_cast<float*>(base + head_ws + up256((size_t)M * 4));
    // no d2t here: the merge then reports draft indices; `tid` only stands in for the NULL check
    vt_status r = check_head_args(h, W_trim, tid, M, d, V_trim, 1, tid, lp, workspace, head_ws);
    if (r != VT_OK) return r;
    HeadOut o = make_out(nullptr, M, V_trim, 1, tid, lp, nullptr, nullptr, logits, workspace);
    HeadCall c{h, W_trim, d, M, V_trim, o, 0};
    return run_head(c, (cudaStream_t)stream, path & VT_PATH_MASK);
}

vt_status vt_fuse_features(const void* h3, const void* W_fuse, int M, int d_in, int d_out, void* fused, void* workspace,
                           size_t workspace_bytes, void* stream) {
    g_launches = 0;
    if (!h3 || !W_fuse || !fused) return VT_ERR_NULL;
    if (d_in < 8 || d_in % 8 != 0 || d_out < 1 || M < 1) return VT_ERR_SHAPE;
    if (!aligned(h3, 16) || !aligned(W_fuse, 16) || !aligned(fused, 2)) return VT_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < ws_total_bytes(M, 1)) return VT_ERR_WORKSPACE;
    // the same contraction kernels as the head, rows of W_fuse in the place of vocabulary rows, with an epilogue
    // that stores the rounded sums and nothing else
    HeadOut o = make_out(nullptr, M, d_out, 1, nullptr, nullptr, nullptr, nullptr, nullptr, workspace);
    o.rounded = reinterpret_cast<uint16_t*>(fused);
    o.store_only = 1;
    HeadCall c{h3, W_fuse, d_in, M, d_out, o, 0};
    return run_head(c, (cudaStream_t)stream, VT_PATH_AUTO);
}

vt_status vt_tree_select(const float* logprobs, const int32_t* target_ids, const float* parent_scores, int M, int k, int T,
                         int32_t* out_rows, int32_t* out_slots, int32_t* out_tokens, float* out_scores, void* stream) {
    g_launches = 0;
    if (!logprobs || !target_ids || !parent_scores || !out_rows || !out_tokens || !out_scores || !out_slots) return VT_ERR_NULL;
    if (M < 1 || k < 1 || T < 1 || (long long)M * k > kTreeSelectMaxPairs || T > M * k) return VT_ERR_SHAPE;
    if (!aligned(logprobs, 4) || !aligned(target_ids, 4) || !aligned(parent_scores, 4) || !aligned(out_rows, 4) ||
        !aligned(out_slots, 4) || !aligned(out_tokens, 4) || !aligned(out_scores, 4))
        return VT_ERR_ALIGN;
    return launch_tree_select(logprobs, target_ids, parent_scores, M, k, T, out_rows, out_slots, out_tokens, out_scores,
                              (cudaStream_t)stream);
}

vt_status vt_remap(const int32_t* draft_ids, const int32_t* d2t, int64_t n, int V_trim, int32_t* target_ids,
                   void* stream) {
    g_launches = 0;
    if (!draft_ids || !d2t || !target_ids) return VT_ERR_NULL;
    if (n < 0 || V_trim < 1) return VT_ERR_SHAPE;
    if (!aligned(draft_ids, 4) || !aligned(d2t, 4) || !aligned(target_ids, 4)) return VT_ERR_ALIGN;
    return launch_remap(draft_ids, d2t, n, V_trim, target_ids, (cudaStream_t)stream);
}

vt_status vt_vocab_maps(const int32_t* keep_ids, int V_trim, int V_full, int32_t* d2t_offsets, uint8_t* t2d_mask,
                        void* stream) {
    g_launches = 0;
    if (!keep_ids || (!d2t_offsets && !t2d_mask)) return VT_ERR_NULL;
    if (V_full < 1 || V_trim < 1 || V_trim > V_full) return VT_ERR_SHAPE;
    if (!aligned(keep_ids, 4) || (d2t_offsets && !aligned(d2t_offsets, 4))) return VT_ERR_ALIGN;
    return launch_vocab_maps(keep_ids, V_trim, V_full, d2t_offsets, t2d_mask, (cudaStream_t)stream);
}

}  // extern "C"
