// Vocabulary-size selection on the GPU: the paper's Method section as an exhaustive scan.
//
//   f(v)   token frequencies of the stream                               (Section 2.2)
//   order  ids by (f descending, id ascending)                           (Section 2.1: top-k most frequent)
//   C(k)   = sum of the k largest f / sum of all f                       (Eq. 2)
//   R(k)   = 1 - (F_fixed + 2 d k) / (F_fixed + 2 d V)                   (Eq. 3)
//   U(k)   = alpha C(k) + (1 - alpha) R(k),  U~(k) = U(k) if C(k) >= c_min else -1      (Eq. 4, 5)
//   k*     = argmax over k in [k_min, k_max] of U~(k), smallest k among equal maxima    (Eq. 1)
//
// The paper samples 100 values of k with a TPE optimiser; evaluating every k costs one pass over a
// 128K-entry prefix sum, so the scan returns the exact optimum of the same objective.  Three steps:
// a histogram with warp-aggregated atomics (HBM-bound read of the stream), a stable least-significant-
// digit radix sort of (count, id), and a prefix sum + objective + arg-max, the last two over 128 CTAs
// that each own one contiguous chunk of the vocabulary.  Doubles are combined with explicit round-to-nearest
// operations so that no fused multiply-add changes a result against the fp64 definition.
#include "vt_launch.h"

namespace vt {

struct SelectResult {
    int k_star;
    int pad;
    double C, R, U;
    unsigned long long total;
    double unique;              // of the distinct ids that occur, the fraction inside the top k*
    unsigned long long pad2[26];
};
static_assert(sizeof(SelectResult) == 256, "one line");

// ------------------------------------------------------------------------------------------ histogram
__global__ void __launch_bounds__(512) select_hist_kernel(const int32_t* __restrict__ token_ids, long long N, int V,
                                                           unsigned int* __restrict__ counts) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += stride) {
        const int t = token_ids[i];
        const bool ok = (unsigned int)t < (unsigned int)V;
        // lanes that hold the same id add once: a Zipf stream repeats its head tokens within a warp
        const unsigned int active = __ballot_sync(__activemask(), ok);
        if (ok) {
            const unsigned int peers = __match_any_sync(active, t);
            if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&counts[t], (unsigned int)__popc(peers));
        }
    }
}

// ------------------------------------------------------------------------------------------ sort
// Stable LSD radix sort of V (key, id) pairs, 8 bits per pass, over kSortBlocks CTAs that each own one contiguous
// chunk of the array: per pass every CTA counts its chunk's digits, one CTA turns the counts into output positions
// (digit-major, CTA-minor: all of digit 0 first, within a digit the chunks in order), and every CTA scatters its
// chunk in order.  key = key_max - count, so ascending keys are descending counts; ids start ascending and every
// pass is stable, so equal counts stay in ascending id order.
constexpr int kSortThreads = 1024;
constexpr int kSortBlocks = 128;

__host__ __device__ inline int sort_chunk(int V) {            // elements per CTA: whole sub-chunks of kSortThreads
    const int per = (V + kSortBlocks - 1) / kSortBlocks;
    return ((per + kSortThreads - 1) / kSortThreads) * kSortThreads;
}

__global__ void __launch_bounds__(kSortThreads) select_keys_kernel(const unsigned int* __restrict__ counts, int V,
                                                                    unsigned int key_max, unsigned int* keyA, int* valA) {
    for (int i = blockIdx.x * kSortThreads + threadIdx.x; i < V; i += gridDim.x * kSortThreads) {
        keyA[i] = key_max - counts[i];
        valA[i] = i;
    }
}

__global__ void __launch_bounds__(kSortThreads) sort_count_kernel(const unsigned int* __restrict__ kin, int V, int shift,
                                                                   unsigned int* __restrict__ hist) {
    __shared__ unsigned int cnt[256];
    const int tid = threadIdx.x;
    if (tid < 256) cnt[tid] = 0;
    __syncthreads();
    const int chunk = sort_chunk(V), begin = blockIdx.x * chunk, end = min(V, begin + chunk);
    for (int i = begin + tid; i < end; i += kSortThreads) atomicAdd(&cnt[(kin[i] >> shift) & 255u], 1u);
    __syncthreads();
    if (tid < 256) hist[tid * kSortBlocks + blockIdx.x] = cnt[tid];
}

// Exclusive prefix sum of the 256 x kSortBlocks counts in place (one CTA).  Warp w owns the 1024 consecutive
// entries from 1024 w: it loads them as 32 coalesced rows of 32, scans row after row with a running carry, and adds
// the totals of the warps before it.
__global__ void __launch_bounds__(kSortThreads) sort_offsets_kernel(unsigned int* __restrict__ hist) {
    static_assert(256 * kSortBlocks == 32 * kSortThreads, "one 1024-entry segment per warp");
    __shared__ unsigned int warp_tot[32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned int* seg = hist + warp * 1024;
    unsigned int v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = seg[j * 32 + lane];
    unsigned int carry = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        unsigned int inc = v[j];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += n;
        }
        v[j] = carry + inc - v[j];                       // exclusive, within the segment
        carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) warp_tot[warp] = carry;
    __syncthreads();
    unsigned int before = 0;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
#pragma unroll
    for (int j = 0; j < 32; ++j) seg[j * 32 + lane] = before + v[j];
}

__global__ void __launch_bounds__(kSortThreads) sort_scatter_kernel(const unsigned int* __restrict__ kin,
                                                                     const int* __restrict__ vin, int V, int shift,
                                                                     const unsigned int* __restrict__ offs,
                                                                     unsigned int* __restrict__ kout, int* __restrict__ vout) {
    __shared__ unsigned int base[256];                 // running output position of each digit for this CTA's chunk
    __shared__ unsigned int warp_cnt[32][256];         // per sub-chunk: occurrences of each digit in each warp
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < 256) base[tid] = offs[tid * kSortBlocks + blockIdx.x];
    __syncthreads();
    const int chunk = sort_chunk(V), begin = blockIdx.x * chunk, end = min(V, begin + chunk);
    for (int c0 = begin; c0 < end; c0 += kSortThreads) {
        const int i = c0 + tid;
        const bool ok = i < end;
        const unsigned int key = ok ? kin[i] : 0u;
        const int val = ok ? vin[i] : 0;
        const unsigned int dg = ok ? (key >> shift) & 255u : 256u;     // 256: a lane past the end
        for (int j = lane; j < 256; j += 32) warp_cnt[warp][j] = 0;
        __syncwarp();
        const unsigned int peers = __match_any_sync(0xFFFFFFFFu, dg);
        const unsigned int before = __popc(peers & ((1u << lane) - 1u));
        if (ok && before == 0) warp_cnt[warp][dg] = __popc(peers);
        __syncthreads();
        if (tid < 256) {                                // digit tid: warps in order, then advance its base
            unsigned int run = base[tid];
            for (int w = 0; w < 32; ++w) {
                const unsigned int n = warp_cnt[w][tid];
                warp_cnt[w][tid] = run;
                run += n;
            }
            base[tid] = run;
        }
        __syncthreads();
        if (ok) {
            const unsigned int pos = warp_cnt[warp][dg] + before;
            kout[pos] = key;
            vout[pos] = val;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------ scan + objective
// Over the same kSortBlocks chunks: (1) every CTA sums its chunk's counts and counts the ids that occur;
// (2) every CTA adds the sums of the chunks before it, scans its chunk, writes the cumulative counts and the ranking,
// and evaluates the objective for the k of its chunk; (3) one small CTA picks the best of the CTAs' bests.
struct ScanScratch {
    unsigned long long sum[kSortBlocks];
    double best_u[kSortBlocks], best_c[kSortBlocks], best_r[kSortBlocks];
    int best_k[kSortBlocks];
    unsigned int distinct[kSortBlocks];
};

__global__ void __launch_bounds__(kSortThreads) scan_sums_kernel(const unsigned int* __restrict__ key_sorted, int V,
                                                                  unsigned int key_max, ScanScratch* sc) {
    __shared__ unsigned long long wsum[32];
    __shared__ unsigned int wocc[32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunk = sort_chunk(V), begin = blockIdx.x * chunk, end = min(V, begin + chunk);
    unsigned long long s = 0ull;
    unsigned int occ = 0u;
    for (int i = begin + tid; i < end; i += kSortThreads) {
        const unsigned int v = key_max - key_sorted[i];
        s += v;
        occ += v > 0u ? 1u : 0u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        occ += __shfl_xor_sync(0xFFFFFFFFu, occ, o);
    }
    if (lane == 0) { wsum[warp] = s; wocc[warp] = occ; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 32; ++w) { s += wsum[w]; occ += wocc[w]; }
        sc->sum[blockIdx.x] = s;
        sc->distinct[blockIdx.x] = occ;
    }
}

__global__ void __launch_bounds__(kSortThreads) scan_apply_kernel(const unsigned int* __restrict__ key_sorted,
                                                                   const int* __restrict__ val_sorted, int V,
                                                                   unsigned int key_max, int d, double F_fixed, double alpha,
                                                                   double c_min, int k_min, int k_max,
                                                                   unsigned long long* __restrict__ cum,
                                                                   int32_t* __restrict__ ranked_ids,
                                                                   unsigned long long* __restrict__ cum_out,
                                                                   ScanScratch* sc) {
    __shared__ unsigned long long warp_tot[32];
    __shared__ unsigned long long carry_s, total_s;
    __shared__ double best_u[32], best_c[32], best_r[32];
    __shared__ int best_k[32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunk = sort_chunk(V), begin = blockIdx.x * chunk, end = min(V, begin + chunk);
    if (tid == 0) {
        unsigned long long before = 0ull, all = 0ull;
        for (int b = 0; b < kSortBlocks; ++b) {
            const unsigned long long s = sc->sum[b];
            if (b < (int)blockIdx.x) before += s;
            all += s;
        }
        carry_s = before;
        total_s = all;
    }
    __syncthreads();
    for (int c0 = begin; c0 < end; c0 += kSortThreads) {   // inclusive prefix sum of the sorted counts
        const int i = c0 + tid;
        unsigned long long v = i < end ? (unsigned long long)(key_max - key_sorted[i]) : 0ull;
        if (i < end) ranked_ids[i] = val_sorted[i];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long n = __shfl_up_sync(0xFFFFFFFFu, v, o);
            if (lane >= o) v += n;
        }
        if (lane == 31) warp_tot[warp] = v;
        __syncthreads();
        unsigned long long off = carry_s;
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        v += off;
        if (i < end) {
            cum[i] = v;
            if (cum_out) cum_out[i] = v;
        }
        __syncthreads();
        if (tid == kSortThreads - 1) carry_s = v;
        __syncthreads();
    }
    const unsigned long long total = total_s;
    const double tot_d = (double)total;
    const double two_d = __dmul_rn(2.0, (double)d);
    const double denom = __dadd_rn(F_fixed, __dmul_rn(two_d, (double)V));
    const double one_minus_alpha = __dsub_rn(1.0, alpha);
    double bu = -2.0, bc = 0.0, br = 0.0;
    int bk = 0x7FFFFFFF;
    if (total > 0) {
        // k = i + 1 for the chunk's positions i; every thread reads back what it wrote itself
        for (int i = begin + tid; i < end; i += kSortThreads) {
            const int k = i + 1;
            if (k < k_min || k > k_max) continue;
            const double C = __ddiv_rn((double)cum[i], tot_d);
            const double R = __dsub_rn(1.0, __ddiv_rn(__dadd_rn(F_fixed, __dmul_rn(two_d, (double)k)), denom));
            const double U = __dadd_rn(__dmul_rn(alpha, C), __dmul_rn(one_minus_alpha, R));
            const double Up = C >= c_min ? U : -1.0;
            if (Up > bu) { bu = Up; bk = k; bc = C; br = R; }
        }
    }
    // arg-max over the block: larger value wins, equal values go to the smaller k
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ou = __shfl_xor_sync(0xFFFFFFFFu, bu, o);
        const int ok = __shfl_xor_sync(0xFFFFFFFFu, bk, o);
        const double oc = __shfl_xor_sync(0xFFFFFFFFu, bc, o);
        const double orr = __shfl_xor_sync(0xFFFFFFFFu, br, o);
        if (ou > bu || (ou == bu && ok < bk)) { bu = ou; bk = ok; bc = oc; br = orr; }
    }
    if (lane == 0) { best_u[warp] = bu; best_k[warp] = bk; best_c[warp] = bc; best_r[warp] = br; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 32; ++w)
            if (best_u[w] > bu || (best_u[w] == bu && best_k[w] < bk)) { bu = best_u[w]; bk = best_k[w]; bc = best_c[w]; br = best_r[w]; }
        sc->best_u[blockIdx.x] = bu;
        sc->best_k[blockIdx.x] = bk;
        sc->best_c[blockIdx.x] = bc;
        sc->best_r[blockIdx.x] = br;
    }
}

__global__ void __launch_bounds__(kSortBlocks) scan_pick_kernel(const ScanScratch* sc, SelectResult* result) {
    __shared__ unsigned long long s_sum[kSortBlocks];
    __shared__ unsigned int s_dis[kSortBlocks];
    __shared__ double s_u[kSortBlocks], s_c[kSortBlocks], s_r[kSortBlocks];
    __shared__ int s_k[kSortBlocks];
    const int b = threadIdx.x;
    s_sum[b] = sc->sum[b]; s_dis[b] = sc->distinct[b];
    s_u[b] = sc->best_u[b]; s_k[b] = sc->best_k[b]; s_c[b] = sc->best_c[b]; s_r[b] = sc->best_r[b];
    __syncthreads();
    if (b != 0) return;
    double bu = -2.0, bc = 0.0, br = 0.0;
    int bk = 0x7FFFFFFF;
    unsigned long long total = 0ull;
    unsigned int distinct = 0u;
    for (int i = 0; i < kSortBlocks; ++i) {
        total += s_sum[i];
        distinct += s_dis[i];
        if (s_u[i] > bu || (s_u[i] == bu && s_k[i] < bk)) { bu = s_u[i]; bk = s_k[i]; bc = s_c[i]; br = s_r[i]; }
    }
    result->k_star = total > 0 ? bk : 0;
    result->C = bc;
    result->R = br;
    result->U = bu;
    result->total = total;
    // counts descend, so the ids that occur are exactly the first `distinct` of the ranking (Table 4's
    // "unique coverage": kept distinct ids over all distinct ids)
    result->unique = distinct > 0 ? __ddiv_rn((double)min((unsigned int)max(bk, 0), distinct), (double)distinct) : 0.0;
}

static inline size_t up256s(size_t b) { return (b + 255) & ~(size_t)255; }
constexpr size_t kSortHistBytes = (size_t)256 * kSortBlocks * 4;
constexpr size_t kSelectScratchBytes = kSortHistBytes + ((sizeof(ScanScratch) + 255) & ~(size_t)255);

}  // namespace vt

using namespace vt;

extern "C" size_t vt_select_workspace_bytes(int V_full) {
    if (V_full < 1) return 0;
    const size_t v = (size_t)V_full;
    // result | counts | keyA keyB valA valB | cum | digit counts of the sort | partial sums of the scan
    return 256 + up256s(v * 4) * 5 + up256s(v * 8) + kSelectScratchBytes;
}

extern "C" vt_status vt_select_vocab(const int32_t* token_ids, int64_t N, int V_full, int d, double F_fixed, double alpha,
                                     double c_min, int k_min, int k_max, int32_t* ranked_ids, uint64_t* cum_counts,
                                     int* k_star, double* C_star, double* R_star, double* U_star, double* unique_star,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    reset_launch_count();
    if (!ranked_ids || !k_star || (!token_ids && N > 0)) return VT_ERR_NULL;
    if (N > 0xFFFFFFFFll) return VT_ERR_SHAPE;                 // the histogram counts in 32 bits
    if (V_full < 1 || d < 1 || N < 0 || k_min < 1 || k_max < k_min || k_max > V_full || !(alpha >= 0.0 && alpha <= 1.0) ||
        !(F_fixed >= 0.0))
        return VT_ERR_SHAPE;
    if (N == 0) return VT_ERR_EMPTY;
    if ((reinterpret_cast<uintptr_t>(token_ids) & 3) || (reinterpret_cast<uintptr_t>(ranked_ids) & 3) ||
        (cum_counts && (reinterpret_cast<uintptr_t>(cum_counts) & 7)))
        return VT_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < vt_select_workspace_bytes(V_full))
        return VT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
    const size_t a4 = up256s((size_t)V_full * 4);
    SelectResult* result = reinterpret_cast<SelectResult*>(base);
    unsigned int* counts = reinterpret_cast<unsigned int*>(base + 256);
    unsigned int* keyA = reinterpret_cast<unsigned int*>(base + 256 + a4);
    unsigned int* keyB = reinterpret_cast<unsigned int*>(base + 256 + 2 * a4);
    int* valA = reinterpret_cast<int*>(base + 256 + 3 * a4);
    int* valB = reinterpret_cast<int*>(base + 256 + 4 * a4);
    unsigned long long* cum = reinterpret_cast<unsigned long long*>(base + 256 + 5 * a4);
    unsigned int* hist = reinterpret_cast<unsigned int*>(base + 256 + 5 * a4 + up256s((size_t)V_full * 8));

    cudaError_t e = cudaMemsetAsync(base, 0, 256 + a4, st);          // result and counts
    if (e != cudaSuccess) return cuda_fail(e);
    int sms = 0;
    vt_status r = device_sm_count(&sms);
    if (r != VT_OK) return r;
    const int grid = (int)std::max<long long>(1, std::min<long long>((N + 511) / 512, (long long)sms * 4));
    select_hist_kernel<<<grid, 512, 0, st>>>(token_ids, N, V_full, counts);
    count_launch();
    // a count is at most N: sort only the bits that can be set
    int bits = 1;
    while (bits < 32 && (1ll << bits) <= N) ++bits;
    const unsigned int key_max = bits >= 32 ? 0xFFFFFFFFu : ((1u << bits) - 1u);
    const int passes = (bits + 7) / 8;
    select_keys_kernel<<<std::min(kSortBlocks, (V_full + kSortThreads - 1) / kSortThreads), kSortThreads, 0, st>>>(counts, V_full, key_max, keyA, valA);
    count_launch();
    unsigned int *kin = keyA, *kout = keyB;
    int *vin = valA, *vout = valB;
    for (int pass = 0; pass < passes; ++pass) {
        sort_count_kernel<<<kSortBlocks, kSortThreads, 0, st>>>(kin, V_full, 8 * pass, hist);
        sort_offsets_kernel<<<1, kSortThreads, 0, st>>>(hist);
        sort_scatter_kernel<<<kSortBlocks, kSortThreads, 0, st>>>(kin, vin, V_full, 8 * pass, hist, kout, vout);
        count_launch();
        count_launch();
        count_launch();
        std::swap(kin, kout);
        std::swap(vin, vout);
    }
    ScanScratch* sc = reinterpret_cast<ScanScratch*>(reinterpret_cast<unsigned char*>(hist) + kSortHistBytes);
    scan_sums_kernel<<<kSortBlocks, kSortThreads, 0, st>>>(kin, V_full, key_max, sc);
    scan_apply_kernel<<<kSortBlocks, kSortThreads, 0, st>>>(kin, vin, V_full, key_max, d, F_fixed, alpha, c_min, k_min, k_max, cum,
                                                            ranked_ids, reinterpret_cast<unsigned long long*>(cum_counts), sc);
    scan_pick_kernel<<<1, kSortBlocks, 0, st>>>(sc, result);
    count_launch();
    count_launch();
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    SelectResult host;
    e = cudaMemcpyAsync(&host, result, sizeof host, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (host.total == 0) return VT_ERR_EMPTY;                       // no token id fell inside [0, V_full)
    *k_star = host.k_star;
    if (C_star) *C_star = host.C;
    if (R_star) *R_star = host.R;
    if (U_star) *U_star = host.U;
    if (unique_star) *unique_star = host.unique;
    return VT_OK;
}
