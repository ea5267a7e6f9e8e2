// The memory-bound helpers around the head: row-gather compaction (the draft vocabulary keeps
// only the rows of V_d), the draft-to-target remap, and the Eq. 2 coverage count.
#include "vt_launch.h"

namespace vt {

// ------------------------------------------------------------------------------------------
// W_trim[i, :] = W_full[keep_ids[i], :] in 16-byte chunks; four independent chunks per thread
// per trip keep enough loads in flight to cover HBM latency.
// ------------------------------------------------------------------------------------------
constexpr int kCompactUnroll = 4;

__global__ void __launch_bounds__(256) compact_kernel(const uint4* __restrict__ W_full, int V_full,
                                                      int chunks_per_row, const int32_t* __restrict__ keep_ids,
                                                      long long total_chunks, uint4* __restrict__ W_trim) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long e0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; e0 < total_chunks;
         e0 += stride * kCompactUnroll) {
        uint4 v[kCompactUnroll];
        bool ok[kCompactUnroll];
#pragma unroll
        for (int u = 0; u < kCompactUnroll; ++u) {
            const long long e = e0 + u * stride;
            ok[u] = false;
            if (e < total_chunks) {
                const int row = (int)(e / chunks_per_row);
                const int col = (int)(e - (long long)row * chunks_per_row);
                const int src = __ldg(&keep_ids[row]);
                if (src >= 0 && src < V_full) {
                    v[u] = __ldcs(&W_full[(size_t)src * chunks_per_row + col]);
                    ok[u] = true;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kCompactUnroll; ++u)
            if (ok[u]) __stcs(&W_trim[e0 + u * stride], v[u]);
    }
}

vt_status launch_compact(const void* W_full, int V_full, int d, const int32_t* keep_ids, int V_trim,
                         void* W_trim, cudaStream_t st) {
    int sms = 0;
    vt_status rs = device_sm_count(&sms);
    if (rs != VT_OK) return rs;
    const int cpr = d / 8;
    const long long total = (long long)V_trim * cpr;
    const long long want = (total + 256LL * kCompactUnroll - 1) / (256LL * kCompactUnroll);
    const int grid = (int)std::max(1LL, std::min(want, (long long)sms * 8));
    compact_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const uint4*>(W_full), V_full, cpr, keep_ids, total,
                                         reinterpret_cast<uint4*>(W_trim));
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// target_ids[t] = d2t[draft_ids[t]]
// ------------------------------------------------------------------------------------------
__global__ void remap_kernel(const int32_t* __restrict__ draft_ids, const int32_t* __restrict__ d2t, long long n,
                             int V_trim, int32_t* __restrict__ target_ids) {
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (long long)gridDim.x * blockDim.x) {
        const int i = draft_ids[t];
        target_ids[t] = (i >= 0 && i < V_trim) ? __ldg(&d2t[i]) : -1;
    }
}

vt_status launch_remap(const int32_t* draft_ids, const int32_t* d2t, int64_t n, int V_trim, int32_t* target_ids,
                       cudaStream_t st) {
    if (n == 0) return VT_OK;
    const int grid = (int)std::min<long long>((n + 255) / 256, 1184);
    remap_kernel<<<grid, 256, 0, st>>>(draft_ids, d2t, n, V_trim, target_ids);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// Cross-row selection of a tree-style draft step: score[m, j] = parent[m] + logprobs[m, j] (one fp32 addition), the
// T best of all M * k pairs in descending order, equal scores by ascending flat index.  One CTA: the keys go to
// shared memory and every pair counts the pairs that beat it - its rank - which is its output position (keys are
// distinct: they carry the flat index).  n = M * k is a few hundred in practice (at most kTreeMaxPairs).
// ------------------------------------------------------------------------------------------
constexpr int kTreeThreads = 512;
constexpr int kTreeMaxPairs = kTreeSelectMaxPairs;

__global__ void __launch_bounds__(kTreeThreads) tree_select_kernel(const float* __restrict__ logprobs,
                                                                 const int32_t* __restrict__ target_ids,
                                                                 const float* __restrict__ parent, int M, int k, int T,
                                                                 int32_t* __restrict__ out_rows, int32_t* __restrict__ out_slots,
                                                                 int32_t* __restrict__ out_tokens, float* __restrict__ out_scores) {
    extern __shared__ unsigned long long keys[];
    const int n = M * k;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
        const int m = e / k;
        keys[e] = make_key(__fadd_rn(parent[m], logprobs[e]), e);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
        const unsigned long long mine = keys[e];
        int rank = 0;
        for (int f = 0; f < n; ++f) rank += keys[f] > mine ? 1 : 0;      // every lane reads the same word: a broadcast
        if (rank < T) {
            const int m = e / k;
            out_rows[rank] = m;
            out_slots[rank] = e - m * k;
            out_tokens[rank] = target_ids[e];
            out_scores[rank] = key_logit(mine);
        }
    }
}

vt_status launch_tree_select(const float* logprobs, const int32_t* target_ids, const float* parent, int M, int k, int T,
                             int32_t* out_rows, int32_t* out_slots, int32_t* out_tokens, float* out_scores, cudaStream_t st) {
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(tree_select_kernel), kTreeMaxPairs * 8, &smem_configured);
        rc != VT_OK)
        return rc;
    tree_select_kernel<<<1, kTreeThreads, (size_t)M * k * 8, st>>>(logprobs, target_ids, parent, M, k, T, out_rows, out_slots,
                                                                  out_tokens, out_scores);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// The two index buffers an EAGLE-3 style draft carries: draft-to-target as offsets
// (target id = draft index + offset) and target-to-draft as a membership flag per target id.
// ------------------------------------------------------------------------------------------
__global__ void vocab_maps_kernel(const int32_t* __restrict__ keep_ids, int V_trim, int V_full,
                                  int32_t* __restrict__ d2t_offsets, unsigned char* __restrict__ t2d_mask) {
    const int stride = gridDim.x * blockDim.x;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < V_trim; i += stride) {
        const int v = keep_ids[i];
        if (d2t_offsets) d2t_offsets[i] = v - i;
        if (t2d_mask && v >= 0 && v < V_full) t2d_mask[v] = 1;
    }
}

vt_status launch_vocab_maps(const int32_t* keep_ids, int V_trim, int V_full, int32_t* d2t_offsets,
                            unsigned char* t2d_mask, cudaStream_t st) {
    if (t2d_mask) {
        cudaError_t e = cudaMemsetAsync(t2d_mask, 0, (size_t)V_full, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    const int grid = std::max(1, std::min((V_trim + 255) / 256, 592));
    vocab_maps_kernel<<<grid, 256, 0, st>>>(keep_ids, V_trim, V_full, d2t_offsets, t2d_mask);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// Membership bitmap of the kept set (bit v of the bitmap = "v is in V_d"); the same pass counts
// out-of-range ids and ids seen twice.
// ------------------------------------------------------------------------------------------
__global__ void keep_bitmap_kernel(const int32_t* __restrict__ keep_ids, int V_trim, int V_full,
                                   CoverageCounters* counters, unsigned int* bitmap) {
    unsigned int oor = 0, dup = 0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < V_trim; i += gridDim.x * blockDim.x) {
        const int v = keep_ids[i];
        if (v < 0 || v >= V_full) {
            ++oor;
        } else {
            const unsigned int bit = 1u << (v & 31);
            if (atomicOr(&bitmap[v >> 5], bit) & bit) ++dup;
        }
    }
    if (oor) atomicAdd(&counters->out_of_range, oor);
    if (dup) atomicAdd(&counters->duplicates, dup);
}

vt_status launch_keep_bitmap(const int32_t* keep_ids, int V_trim, int V_full, void* workspace, cudaStream_t st) {
    const size_t bytes = sizeof(CoverageCounters) + coverage_bitmap_words(V_full) * 4;
    cudaError_t e = cudaMemsetAsync(workspace, 0, bytes, st);
    if (e != cudaSuccess) return cuda_fail(e);
    auto* counters = reinterpret_cast<CoverageCounters*>(workspace);
    auto* bitmap = reinterpret_cast<unsigned int*>(counters + 1);
    const int grid = std::max(1, std::min((V_trim + 255) / 256, 592));
    keep_bitmap_kernel<<<grid, 256, 0, st>>>(keep_ids, V_trim, V_full, counters, bitmap);
    count_launch();
    e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// covered = #{t : token_ids[t] in V_d}: each CTA copies the bitmap to shared memory when it
// fits, streams its share of the ids with 16-byte loads and adds one 64-bit count per CTA.
// ------------------------------------------------------------------------------------------
constexpr int kCoverageThreads = 512;
constexpr size_t kCoverageSmemBitmapMax = 160 * 1024;

__device__ __forceinline__ unsigned int member(const unsigned int* bm, int v, int V_full) {
    return ((unsigned int)v < (unsigned int)V_full) ? ((bm[v >> 5] >> (v & 31)) & 1u) : 0u;
}

__global__ void __launch_bounds__(kCoverageThreads) coverage_count_kernel(
    const int32_t* __restrict__ token_ids, long long N, int V_full, const unsigned int* __restrict__ bitmap_g,
    int bitmap_words, int bitmap_in_smem, CoverageCounters* counters) {
    extern __shared__ unsigned int bm_s[];
    __shared__ unsigned int warp_counts[kCoverageThreads / 32];
    const unsigned int* bm = bitmap_g;
    if (bitmap_in_smem) {
        for (int w = threadIdx.x; w < bitmap_words; w += blockDim.x) bm_s[w] = bitmap_g[w];
        __syncthreads();
        bm = bm_s;
    }
    // elements before the first 16-byte boundary and after the last full vector are taken singly
    const uintptr_t addr = reinterpret_cast<uintptr_t>(token_ids);
    long long head = (long long)(((16 - (addr & 15)) & 15) / 4);
    if (head > N) head = N;
    const long long nvec = (N - head) / 4;
    const long long tail_begin = head + nvec * 4;
    const int4* vec = reinterpret_cast<const int4*>(token_ids + head);

    unsigned int c = 0;
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long gstride = (long long)gridDim.x * blockDim.x;
    // four independent 16-byte loads per thread and trip keep enough bytes in flight to cover HBM latency
    long long i = gtid;
    for (; i + 3 * gstride < nvec; i += 4 * gstride) {
        int4 t[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) t[u] = __ldcs(&vec[i + u * gstride]);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            c += member(bm, t[u].x, V_full) + member(bm, t[u].y, V_full) + member(bm, t[u].z, V_full) + member(bm, t[u].w, V_full);
    }
    for (; i < nvec; i += gstride) {
        const int4 t = __ldcs(&vec[i]);
        c += member(bm, t.x, V_full) + member(bm, t.y, V_full) + member(bm, t.z, V_full) + member(bm, t.w, V_full);
    }
    for (long long i = gtid; i < head; i += gstride) c += member(bm, token_ids[i], V_full);
    for (long long i = tail_begin + gtid; i < N; i += gstride) c += member(bm, token_ids[i], V_full);

#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0) warp_counts[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long total = 0;
        for (int w = 0; w < kCoverageThreads / 32; ++w) total += warp_counts[w];
        if (total) atomicAdd(&counters->covered, total);
    }
}

vt_status launch_coverage_count(const int32_t* token_ids, int64_t N, int V_full, void* workspace, cudaStream_t st) {
    int sms = 0;
    vt_status rs = device_sm_count(&sms);
    if (rs != VT_OK) return rs;
    auto* counters = reinterpret_cast<CoverageCounters*>(workspace);
    auto* bitmap = reinterpret_cast<unsigned int*>(counters + 1);
    const size_t words = coverage_bitmap_words(V_full);
    const int in_smem = words * 4 <= kCoverageSmemBitmapMax;
    const size_t smem = in_smem ? words * 4 : 0;
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(coverage_count_kernel), (int)((int)kCoverageSmemBitmapMax), &smem_configured); rc != VT_OK)
        return rc;
    const long long per_cta = (long long)kCoverageThreads * 4 * 8;   // ids one CTA takes in two trips of four loads
    const int grid = (int)std::max(1LL, std::min((N + per_cta - 1) / per_cta, (long long)sms * 4));
    coverage_count_kernel<<<grid, kCoverageThreads, smem, st>>>(token_ids, N, V_full, bitmap, (int)words, in_smem,
                                                               counters);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// The same count in ONE launch, for vocabularies whose bitmap fits in shared memory: every CTA builds the whole
// membership bitmap for itself from keep_ids (V_trim ids from L2, a few microseconds) and then counts its share of
// the stream.  No bitmap in global memory, no second kernel: the stream's read is all that touches HBM.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kCoverageThreads) coverage_fused_kernel(
    const int32_t* __restrict__ token_ids, long long N, const int32_t* __restrict__ keep_ids, int V_trim, int V_full,
    int bitmap_words, CoverageCounters* counters) {
    extern __shared__ unsigned int bm_s[];
    __shared__ unsigned int warp_counts[kCoverageThreads / 32];
    for (int w = threadIdx.x; w < bitmap_words; w += blockDim.x) bm_s[w] = 0u;
    __syncthreads();
    // sixteen ids in flight per thread (four 16-byte loads where keep_ids allows): the whole list costs a few L2
    // round trips, not one per id
    auto mark = [&](int v) {
        if ((unsigned int)v < (unsigned int)V_full) atomicOr(&bm_s[v >> 5], 1u << (v & 31));
    };
    const int kvec = (reinterpret_cast<uintptr_t>(keep_ids) & 15) == 0 ? V_trim / 4 : 0;
    const int4* keep4 = reinterpret_cast<const int4*>(keep_ids);
    for (int i0 = threadIdx.x; i0 < kvec; i0 += 4 * blockDim.x) {
        int4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * blockDim.x;
            v[u] = i < kvec ? __ldg(&keep4[i]) : make_int4(-1, -1, -1, -1);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) { mark(v[u].x); mark(v[u].y); mark(v[u].z); mark(v[u].w); }
    }
    for (int i = 4 * kvec + threadIdx.x; i < V_trim; i += blockDim.x) mark(__ldg(&keep_ids[i]));
    __syncthreads();
    const uintptr_t addr = reinterpret_cast<uintptr_t>(token_ids);
    long long head = (long long)(((16 - (addr & 15)) & 15) / 4);
    if (head > N) head = N;
    const long long nvec = (N - head) / 4;
    const long long tail_begin = head + nvec * 4;
    const int4* vec = reinterpret_cast<const int4*>(token_ids + head);
    unsigned int c = 0;
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long gstride = (long long)gridDim.x * blockDim.x;
    long long i = gtid;
    for (; i + 3 * gstride < nvec; i += 4 * gstride) {      // four independent 16-byte loads in flight per thread
        int4 t[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) t[u] = __ldcs(&vec[i + u * gstride]);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            c += member(bm_s, t[u].x, V_full) + member(bm_s, t[u].y, V_full) + member(bm_s, t[u].z, V_full) + member(bm_s, t[u].w, V_full);
    }
    for (; i < nvec; i += gstride) {
        const int4 t = __ldcs(&vec[i]);
        c += member(bm_s, t.x, V_full) + member(bm_s, t.y, V_full) + member(bm_s, t.z, V_full) + member(bm_s, t.w, V_full);
    }
    for (long long j = gtid; j < head; j += gstride) c += member(bm_s, token_ids[j], V_full);
    for (long long j = tail_begin + gtid; j < N; j += gstride) c += member(bm_s, token_ids[j], V_full);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0) warp_counts[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long total = 0;
        for (int w = 0; w < kCoverageThreads / 32; ++w) total += warp_counts[w];
        if (total) atomicAdd(&counters->covered, total);
    }
}

bool coverage_fused_fits(int V_full) { return coverage_bitmap_words(V_full) * 4 <= kCoverageSmemBitmapMax; }

vt_status launch_coverage_fused(const int32_t* token_ids, int64_t N, const int32_t* keep_ids, int V_trim, int V_full,
                                void* workspace, cudaStream_t st) {
    int sms = 0;
    vt_status rs = device_sm_count(&sms);
    if (rs != VT_OK) return rs;
    const size_t words = coverage_bitmap_words(V_full);
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(coverage_fused_kernel), (int)kCoverageSmemBitmapMax, &smem_configured); rc != VT_OK)
        return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, sizeof(CoverageCounters), st);
    if (e != cudaSuccess) return cuda_fail(e);
    // few enough CTAs that re-reading keep_ids once per CTA stays well below the stream's own bytes
    const long long per_cta = (long long)kCoverageThreads * 4 * 8;
    const long long by_keep = std::max<long long>(1, (4 * (long long)N) / std::max(1, V_trim));           // CTAs whose keep_ids reads add up to the stream's
    const long long want = std::min<long long>(((long long)N + per_cta - 1) / per_cta, (long long)sms * 2);
    const int grid = (int)std::max<long long>(1, std::min<long long>(want, std::max<long long>(8, by_keep)));
    coverage_fused_kernel<<<grid, kCoverageThreads, words * 4, st>>>(token_ids, N, keep_ids, V_trim, V_full, (int)words,
                                                                   reinterpret_cast<CoverageCounters*>(workspace));
    count_launch();
    e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// ------------------------------------------------------------------------------------------
// Coverage without caller-provided scratch: the bitmap and the counters live in a fixed array that is
// part of the library image on every device that loads it.
// ------------------------------------------------------------------------------------------
constexpr int kStaticCoverageMaxV = 262144;    // largest V_full vt_coverage_static accepts (bitmap: 32 KiB)
static __device__ __align__(256) unsigned char g_static_coverage[sizeof(CoverageCounters) + kStaticCoverageMaxV / 8];

// Device address of g_static_coverage on the current device.  In host code the array's name is only a
// handle for the runtime, not a pointer a kernel could use, so the address is asked for once per device
// (with that device current) and remembered.
static vt_status static_coverage_address(void** out) {
    static std::atomic<void*> cached[64];     // racing first calls on a device look up and store the same address
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
    void* ptr = cached[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(&ptr, g_static_coverage);
        if (e != cudaSuccess) return cuda_fail(e);
        cached[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return VT_OK;
}

}  // namespace vt

extern "C" vt_status vt_coverage_static(const int32_t* token_ids, int64_t N, const int32_t* keep_ids, int V_trim,
                                        int V_full, uint64_t* covered_out, double* fraction_out, void* stream) {
    using namespace vt;
    reset_launch_count();
    if (!keep_ids || (!token_ids && N > 0)) return VT_ERR_NULL;
    if (V_full < 1 || V_trim < 1 || N < 0) return VT_ERR_SHAPE;
    if (V_full > kStaticCoverageMaxV) return VT_ERR_SHAPE;       // the built-in scratch holds no larger bitmap
    if (N == 0) return VT_ERR_EMPTY;
    if ((reinterpret_cast<uintptr_t>(token_ids) & 3) || (reinterpret_cast<uintptr_t>(keep_ids) & 3)) return VT_ERR_ALIGN;
    void* scratch = nullptr;
    vt_status r = static_coverage_address(&scratch);
    if (r != VT_OK) return r;
    cudaStream_t st = (cudaStream_t)stream;
    r = launch_keep_bitmap(keep_ids, V_trim, V_full, scratch, st);   // starts by zeroing counters and bitmap
    if (r != VT_OK) return r;
    r = launch_coverage_count(token_ids, N, V_full, scratch, st);
    if (r != VT_OK) return r;
    CoverageCounters c;
    cudaError_t e = cudaMemcpyAsync(&c, scratch, sizeof c, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (covered_out) *covered_out = c.covered;
    if (fraction_out) *fraction_out = (double)c.covered / (double)N;
    return VT_OK;
}
