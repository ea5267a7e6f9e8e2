// Shared device/host helpers of the draft-head library: workspace layout, PTX wrappers for
// mbarriers and bulk copies with bounded waits, sortable (logit, index) keys, the per-thread
// top-k list and the cross-CTA merge that ends a draft-head call.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/vt.h"

namespace vt {

// ------------------------------------------------------------------------------------------
// Workspace of a draft-head call:
//   [0, 256)                       WsHeader
//   keys  [kMaxParts][M][k] u64    per-CTA partial top-k lists (sortable keys, descending)
//   ms    [kMaxParts][M] float2    per-CTA (running max, sum of exp(x - max))
// ------------------------------------------------------------------------------------------
constexpr int kMaxParts = 256;             // upper bound on CTAs that contribute partials
constexpr size_t kHeaderBytes = 256;

struct WsHeader {
    unsigned int ticket;     // CTAs that have published their partials in the running call
    unsigned int status;     // bit 0: a bounded wait ran out
    unsigned int pad[62];
};
static_assert(sizeof(WsHeader) == kHeaderBytes, "header is one 256-byte line");

constexpr unsigned int kStatusTimeout = 1u;

__host__ __device__ inline size_t ws_keys_bytes(int M, int k) { return (size_t)kMaxParts * M * k * 8; }
__host__ __device__ inline size_t ws_ms_bytes(int M) { return (size_t)kMaxParts * M * 8; }
__host__ __device__ inline size_t ws_total_bytes(int M, int k) {
    size_t b = kHeaderBytes + ws_keys_bytes(M, k) + ws_ms_bytes(M);
    return (b + 255) & ~(size_t)255;
}

struct HeadOut {
    const int32_t* d2t;
    int32_t* target_ids;
    float* logprobs;
    int32_t* draft_ids;   // may be null
    float* lse;           // may be null
    float* logits;        // debug: [M, Vt] fp32, null on the fast path
    WsHeader* hdr;
    unsigned long long* keys;
    float2* ms;
    int M, k, Vt;
};

#ifdef __CUDACC__
// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;   // 1 s per wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits for the phase with the given parity to complete, for at most kWaitLimitNs.
// Returns false when the limit ran out (the caller records it and unwinds; nothing spins forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (((++spins) & 0xFFu) == 0 && global_timer_ns() - t0 > kWaitLimitNs) return false;
    }
    return true;
}

// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses and the size must be multiples of 16 bytes.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------
// Sortable keys: a larger key is a better candidate (higher logit, then lower draft index).
// Key 0 means "no candidate" (no finite logit maps to a zero high word).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long make_key(float x, int idx) {
    uint32_t u = __float_as_uint(x + 0.0f);                 // -0 -> +0 so equal logits tie on index
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}
__device__ __forceinline__ float key_logit(unsigned long long key) {
    uint32_t u = (uint32_t)(key >> 32);
    u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
    return __uint_as_float(u);
}
__device__ __forceinline__ int key_index(unsigned long long key) {
    return (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
}

// Insert into a descending list of k keys held at list[j * stride]; returns the new k-th key.
__device__ __forceinline__ unsigned long long list_insert(unsigned long long* list, int stride, int k,
                                                          unsigned long long key) {
    int j = k - 1;
    while (j > 0) {
        unsigned long long prev = list[(j - 1) * stride];
        if (prev >= key) break;
        list[j * stride] = prev;
        --j;
    }
    list[j * stride] = key;
    return list[(k - 1) * stride];
}

// Online log-sum-exp state: s = sum exp(x - mx) over the logits seen so far.
__device__ __forceinline__ void lse_update(float& mx, float& s, float x) {
    if (x > mx) {
        s = s * __expf(mx - x) + 1.0f;
        mx = x;
    } else {
        s += __expf(x - mx);
    }
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long w = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = w > v ? w : v;
    }
    return v;
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ------------------------------------------------------------------------------------------
// Cross-CTA merge of one draft row by one warp.
//   P partial lists (descending, k keys each, 0-padded) and
//   P pairs (mx_p, s_p); both already staged in shared memory: stage[p * k + j], stage_ms[p].
// Writes the row's k winners in descending key order with their log-probs and target ids.
// ------------------------------------------------------------------------------------------
constexpr int kMergeSlots = kMaxParts / 32;

__device__ inline void merge_row(const HeadOut& o, int P, int m, const unsigned long long* stage,
                                 const float2* stage_ms) {
    const int lane = threadIdx.x & 31;
    const int k = o.k;

    // log-sum-exp over the partials: lse = mx + log sum_p s_p * exp(mx_p - mx)
    float mx = -INFINITY;
    for (int p = lane; p < P; p += 32) mx = fmaxf(mx, stage_ms[p].x);
    mx = warp_max_f32(mx);
    float s = 0.0f;
    for (int p = lane; p < P; p += 32) {
        const float2 v = stage_ms[p];
        if (v.y > 0.0f) s += v.y * __expf(v.x - mx);
    }
    s = warp_sum_f32(s);
    const float lse = mx + logf(s);

    // lane owns lists lane, lane+32, ...; every list is sorted, so its best is its head
    int head[kMergeSlots];
    unsigned long long hk[kMergeSlots];
#pragma unroll
    for (int q = 0; q < kMergeSlots; ++q) {
        const int p = lane + 32 * q;
        head[q] = 0;
        hk[q] = (p < P) ? stage[p * k] : 0ull;
    }
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int q = 0; q < kMergeSlots; ++q) best = hk[q] > best ? hk[q] : best;
        best = warp_max_u64(best);
        // keys are unique across lists (disjoint vocabulary rows), so exactly one head matches
#pragma unroll
        for (int q = 0; q < kMergeSlots; ++q) {
            if (best != 0ull && hk[q] == best) {
                const int p = lane + 32 * q;
                ++head[q];
                hk[q] = head[q] < k ? stage[p * k + head[q]] : 0ull;
            }
        }
        if (lane == 0) {
            const size_t out = (size_t)m * k + j;
            if (best != 0ull) {
                const int idx = key_index(best);
                o.target_ids[out] = o.d2t ? __ldg(&o.d2t[idx]) : idx;
                o.logprobs[out] = key_logit(best) - lse;
                if (o.draft_ids) o.draft_ids[out] = idx;
            } else {   // fewer than k candidates exist only if a wait ran out upstream
                o.target_ids[out] = -1;
                o.logprobs[out] = -INFINITY;
                if (o.draft_ids) o.draft_ids[out] = -1;
            }
        }
    }
    if (lane == 0 && o.lse) o.lse[m] = lse;
}

// Publishes this CTA's partials (already written to global memory by the calling threads) and
// returns true in every thread of the last CTA to arrive.  Must be called by all threads.
__device__ inline bool publish_and_check_last(WsHeader* hdr, int* smem_flag) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int t = atomicAdd(&hdr->ticket, 1u);
        *smem_flag = (t == gridDim.x - 1) ? 1 : 0;
        __threadfence();
    }
    __syncthreads();
    return *smem_flag != 0;
}

// Last CTA: merges draft rows [m_begin, m_begin + m_count).  All threads first copy the partials of
// a batch of rows from L2 into shared memory (independent loads, a few per thread), then each warp
// merges one row at a time out of shared memory.  `stage_base` is shared memory the CTA no longer
// uses; the host sizes it to hold at least one row: P * (k + 1) * 8 bytes.
__device__ inline void merge_rows(const HeadOut& o, int P, int m_begin, int m_count,
                                  unsigned char* stage_base, size_t stage_bytes) {
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int k = o.k, M = o.M;
    const size_t per_row = (size_t)P * (k + 1) * 8;
    int batch = (int)(stage_bytes / per_row);
    if (batch < 1) batch = 1;
    if (batch > m_count) batch = m_count;
    unsigned long long* skeys = reinterpret_cast<unsigned long long*>(stage_base);
    float2* sms = reinterpret_cast<float2*>(stage_base + (size_t)batch * P * k * 8);
    const int Pk = P * k;
    for (int b0 = 0; b0 < m_count; b0 += batch) {
        const int nb = min(batch, m_count - b0);
        const int total = nb * Pk;
        constexpr int U = 4;
        for (int e0 = threadIdx.x; e0 < total; e0 += blockDim.x * U) {
            unsigned long long v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int e = e0 + u * blockDim.x;
                if (e < total) {
                    const int r = e / Pk, rem = e - r * Pk;
                    const int p = rem / k, j = rem - p * k;
                    v[u] = __ldcg(&o.keys[((size_t)p * M + (m_begin + b0 + r)) * k + j]);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int e = e0 + u * blockDim.x;
                if (e < total) skeys[e] = v[u];
            }
        }
        for (int e = threadIdx.x; e < nb * P; e += blockDim.x) {
            const int r = e / P, p = e - r * P;
            sms[e] = __ldcg(&o.ms[(size_t)p * M + (m_begin + b0 + r)]);
        }
        __syncthreads();
        for (int r = warp; r < nb; r += nwarps)
            merge_row(o, P, m_begin + b0 + r, skeys + (size_t)r * Pk, sms + (size_t)r * P);
        __syncthreads();
    }
    if (threadIdx.x == 0) o.hdr->ticket = 0u;   // ready for the next call on this stream
}
#endif  // __CUDACC__

}  // namespace vt
