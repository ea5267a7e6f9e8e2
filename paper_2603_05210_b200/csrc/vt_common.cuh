// Shared device/host helpers of the draft-head library: workspace layout, PTX wrappers for
// mbarriers and bulk copies with bounded waits, sortable (logit, index) keys, the per-warp and per-thread
// top-k updates and the cross-CTA merge that ends a draft-head call.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/vt.h"

namespace vt {

// ------------------------------------------------------------------------------------------
// Workspace of a draft-head call:
//   [0, 512)   WsHeader
//   records    per draft row m, kMaxParts * (k + 1) consecutive u64 (row-major: what one CTA wrote for one row is
//              strided, what all CTAs wrote for one row is contiguous, so the warp that merges a row reads every
//              CTA's j-th best key with one coalesced load):
//                ms   [kMaxParts]        every CTA's (running max, sum of exp(x - max)) as two floats
//                keys [k][kMaxParts]     keys[j][p] = CTA p's j-th best candidate as a sortable key, 0 = none
// ------------------------------------------------------------------------------------------
constexpr int kMaxParts = 256;             // upper bound on CTAs that contribute partials
constexpr size_t kHeaderBytes = 512;

constexpr int kRowTickets = 64;            // draft rows that can be merged row by row (one ticket each)

struct WsHeader {
    unsigned int reserved;
    unsigned int status;     // bit 0: a bounded wait ran out
    unsigned int row_ticket[kRowTickets];   // per draft row: CTAs that have published that row (row-wise merge)
    unsigned int pad[126 - kRowTickets];
};
static_assert(sizeof(WsHeader) == kHeaderBytes, "header is two 256-byte lines");

constexpr unsigned int kStatusTimeout = 1u;

__host__ __device__ inline size_t ws_total_bytes(int M, int k) {
    size_t b = kHeaderBytes + (size_t)M * kMaxParts * (size_t)(k + 1) * 8;
    return (b + 255) & ~(size_t)255;
}

#define VT_ROW_MS(o, m) ((o).recs + (size_t)(m) * kMaxParts * ((o).k + 1))
#define VT_ROW_KEYS(o, m, j) (VT_ROW_MS(o, m) + (size_t)((j) + 1) * kMaxParts)

struct HeadOut {
    const int32_t* d2t;   // null: report draft indices as target ids
    int d2t_offsets;      // 1: d2t holds offsets, target id = draft index + d2t[draft index]
    int32_t* target_ids;
    float* logprobs;
    int32_t* draft_ids;   // may be null
    float* lse;           // may be null
    float* logits;        // debug: [M, Vt] fp32, null on the fast path
    uint16_t* rounded;    // the contraction rounded to bf16, [M, Vt], null for the head
    int store_only;       // 1: the contraction is the result (a plain projection): no top-k, no log-sum-exp, no records
    WsHeader* hdr;
    unsigned long long* recs;
    int M, k, Vt;
    int fused_merge;      // 1: the warp that publishes a row last of all CTAs merges it; 0: the merge kernel follows
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
__device__ __forceinline__ void fence_proxy_async() {      // generic <-> async proxy, all state spaces
    asm volatile("fence.proxy.async;" ::: "memory");
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
// Waits for the phase with the given parity to complete, for at most `limit_ns` (one second unless the caller
// asks for less).  Returns false when the limit ran out (the caller records it and unwinds; nothing spins forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns = kWaitLimitNs) {
    for (int i = 0; i < 64; ++i)                       // the common case: no clock read on the way
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (((++spins) & 0xFFu) == 0 && global_timer_ns() - t0 > limit_ns) return false;
    }
    return true;
}
// The same wait against an absolute deadline (a %globaltimer value): an unwinding CTA that lets several copies
// land shares one deadline between them instead of granting each its own second.
__device__ __forceinline__ bool mbar_wait_until(uint32_t bar, uint32_t parity, unsigned long long deadline_ns) {
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (((++spins) & 0x3Fu) == 0 && global_timer_ns() > deadline_ns) return false;
    }
    return true;
}

// Programmatic dependent launch.  A head kernel is launched with the programmatic-serialization attribute:
// its CTAs may become resident while the previous kernel in the stream is still finishing (for back-to-back
// head calls: while the last CTA of the previous call merges), run their set-up that touches no global
// memory, and then wait here until that previous kernel has completed and its writes are visible.  Without
// the attribute both instructions do nothing.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses and the size must be multiples of 16 bytes.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Writes x[m, col] where the caller asked for the contraction itself: fp32 for inspection, and / or rounded once
// to bf16 (round-to-nearest-even) for a projection whose output feeds the next layer.
__device__ __forceinline__ bool wants_logits(const HeadOut& o) { return o.logits != nullptr || o.rounded != nullptr; }
__device__ __forceinline__ void store_logit(const HeadOut& o, int m, int col, float x) {
    const size_t at = (size_t)m * o.Vt + col;
    if (o.logits) o.logits[at] = x;
    if (o.rounded) o.rounded[at] = __bfloat16_as_ushort(__float2bfloat16_rn(x));
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

__device__ __forceinline__ unsigned long long pack_ms(float mx, float s) {
    return ((unsigned long long)__float_as_uint(s) << 32) | (unsigned long long)__float_as_uint(mx);
}
__device__ __forceinline__ float2 unpack_ms(unsigned long long v) {
    return make_float2(__uint_as_float((uint32_t)v), __uint_as_float((uint32_t)(v >> 32)));
}


// ------------------------------------------------------------------------------------------
// Thread-private top-k: one thread owns one draft row and keeps its KR best (logit, index) pairs in registers.
// ------------------------------------------------------------------------------------------
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Sorted insertion into a thread's register list: v descends, equal logits keep their order of arrival (logits
// reach a thread in ascending vocabulary order, so a later equal one ranks below).  p[j] = "x beats entry j" is
// monotone in j; entry j takes its upper neighbour where that one is beaten, x where only it is, else stays.
// Inserting a logit that beats nothing changes nothing.
template <int KR>
__device__ __forceinline__ void rows_insert(float (&v)[KR], int (&ix)[KR], float x, int xi) {
    bool p[KR];
#pragma unroll
    for (int j = 0; j < KR; ++j) p[j] = x > v[j];
#pragma unroll
    for (int j = KR - 1; j > 0; --j) {
        v[j] = p[j - 1] ? v[j - 1] : (p[j] ? x : v[j]);
        ix[j] = p[j - 1] ? ix[j - 1] : (p[j] ? xi : ix[j]);
    }
    v[0] = p[0] ? x : v[0];
    ix[0] = p[0] ? xi : ix[0];
}

// The same insertion for logits alone (no indices): two min/max per entry.
template <int KR>
__device__ __forceinline__ void vals_insert(float (&g)[KR], float x) {
#pragma unroll
    for (int j = KR - 1; j > 0; --j) g[j] = fmaxf(g[j], fminf(g[j - 1], x));
    g[0] = fmaxf(g[0], x);
}


// 16 consecutive logits of a draft row from shared memory (columns c .. c + 15, c a multiple of 4 floats from a
// 16-byte aligned row); columns at or past `ce` come back as -inf.
__device__ __forceinline__ void row_load16(const float* rowp, int c, int ce, float (&x)[16]) {
#pragma unroll
    for (int u4 = 0; u4 < 4; ++u4) {
        const float4 f = *reinterpret_cast<const float4*>(rowp + c + 4 * u4);
        x[4 * u4 + 0] = f.x; x[4 * u4 + 1] = f.y; x[4 * u4 + 2] = f.z; x[4 * u4 + 3] = f.w;
    }
    const int left = ce - c;
    if (left < 16) {
#pragma unroll
        for (int e = 0; e < 16; ++e) x[e] = e < left ? x[e] : -INFINITY;
    }
}

// Running log-sum-exp of one draft row over its columns [cb, ce) (at most 128): (max, sum of exp(x - max)).
__device__ __forceinline__ void row_scan_lse(const float* rowp, int cb, int ce, float& mx, float& ssum) {
    const int nch = (ce - cb + 15) >> 4;
    for (int q = 0; q < nch; ++q) {
        float x[16];
        row_load16(rowp, cb + 16 * q, ce, x);
        float cm = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
        cm = fmaxf(cm, fmaxf(fmaxf(fmaxf(x[8], x[9]), fmaxf(x[10], x[11])), fmaxf(fmaxf(x[12], x[13]), fmaxf(x[14], x[15]))));
        const float nm = fmaxf(mx, cm);
        const float nml = nm * kLog2e;
        float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
            a0 += ex2_approx(fmaf(x[e], kLog2e, -nml));             // exp(-inf) = 0
            a1 += ex2_approx(fmaf(x[e + 1], kLog2e, -nml));
        }
        ssum = ssum * ex2_approx((mx - nm) * kLog2e) + (a0 + a1);   // first chunk: 0 * 0
        mx = nm;
    }
}

constexpr int kRowQueue = 64;      // candidate columns a thread can queue per scan; more than that and the warp inserts every column

// Top-k update of one draft row by ONE thread over the row's columns [cb, ce) in shared memory (at most 128
// columns; column c is vocabulary row idx0 + c).  `full` says whether the thread's list already holds KR entries
// (the same in every lane of the warp: all lanes have scanned equally many logits).
//   list full:      candidates are the logits above the list's last entry (strictly: a later row loses a tie);
//   first scan of a long range: the KR-th largest of the maxima of groups of 4 or 8 logits has at least KR logits
//                   at or above it, so nothing below it can be among the KR best: candidates are the logits not
//                   below that bound;
//   first scan of a short range: every logit goes through the list.
// The candidates' columns are compacted into the thread's queue (`queue`: the thread's first byte, entries 128
// bytes apart; branch-free: every column is stored and a candidate keeps its slot), then inserted one per turn
// of a loop that runs for the busiest lane's count, each turn's column and logit fetched ahead of its
// insertion.  The compare-and-select pipe runs at half rate, which makes the insertion (5 such operations
// per list entry) the cost of this function: it is spent on the candidates only.  All lanes must call it.
template <int KR>
__device__ __forceinline__ void row_scan_topk(const float* rowp, int cb, int ce, int idx0, bool full, float (&v)[KR],
                                              int (&ix)[KR], unsigned char* queue) {
    const int n = ce - cb, nch = (n + 15) >> 4;
    const int gs = full ? 0 : n >= 8 * (KR + 2) ? 8 : n >= 4 * (KR + 2) ? 4 : 0;
    bool all = !full && gs == 0;
    int cnt = 0;
    if (!all) {
        float tau = v[KR - 1];
        if (!full) {       // bound from group maxima: at least KR + 2 whole groups exist
            float g[KR];
#pragma unroll
            for (int j = 0; j < KR; ++j) g[j] = -INFINITY;
            for (int q = 0; q < nch; ++q) {
                float x[16];
                row_load16(rowp, cb + 16 * q, ce, x);
                if (gs == 8) {
#pragma unroll
                    for (int u8 = 0; u8 < 2; ++u8)
                        vals_insert<KR>(g, fmaxf(fmaxf(fmaxf(x[8 * u8], x[8 * u8 + 1]), fmaxf(x[8 * u8 + 2], x[8 * u8 + 3])),
                                                 fmaxf(fmaxf(x[8 * u8 + 4], x[8 * u8 + 5]), fmaxf(x[8 * u8 + 6], x[8 * u8 + 7]))));
                } else {
#pragma unroll
                    for (int u4 = 0; u4 < 4; ++u4)
                        vals_insert<KR>(g, fmaxf(fmaxf(x[4 * u4], x[4 * u4 + 1]), fmaxf(x[4 * u4 + 2], x[4 * u4 + 3])));
                }
            }
            tau = g[KR - 1];
        }
        for (int q = 0; q < nch; ++q) {
            float x[16];
            row_load16(rowp, cb + 16 * q, ce, x);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                queue[min(cnt, kRowQueue - 1) * 128] = (unsigned char)(16 * q + e);
                cnt += (full ? x[e] > tau : x[e] >= tau) ? 1 : 0;
            }
        }
        const int most = (int)__reduce_max_sync(0xFFFFFFFFu, (unsigned)cnt);
        all = most > kRowQueue;
        if (!all) {
            // turn i inserts the lane's i-th candidate; its column was fetched two turns earlier, its logit one
            int c1 = queue[0], c2 = queue[128];
            float x1 = rowp[cb + (cnt > 0 ? c1 : 0)];
            for (int i = 0; i < most; ++i) {
                const float xv = i < cnt ? x1 : -INFINITY;         // -inf beats nothing
                const int xi = idx0 + cb + c1;
                c1 = c2;
                x1 = rowp[cb + (i + 1 < cnt ? c1 : 0)];
                c2 = queue[min(i + 2, kRowQueue - 1) * 128];
                rows_insert<KR>(v, ix, xv, xi);
            }
        }
    }
    if (all) {
        for (int q = 0; q < nch; ++q) {
            float x[16];
            row_load16(rowp, cb + 16 * q, ce, x);
#pragma unroll
            for (int e = 0; e < 16; ++e) rows_insert<KR>(v, ix, x[e], idx0 + cb + 16 * q + e);
        }
    }
}

// Register-list length for a top-k of k: the smallest instantiated length that holds k entries, 0 if none does.
__host__ __device__ inline int topk_list_regs(int k) { return k <= 4 ? 4 : k <= 8 ? 8 : k <= 10 ? 10 : k <= 16 ? 16 : 0; }

// Warp-wide maximum of 64-bit keys with two 32-bit redux operations.
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long v) {
    const uint32_t hi = (uint32_t)(v >> 32), lo = (uint32_t)v;
    const uint32_t mhi = __reduce_max_sync(0xFFFFFFFFu, hi);
    const uint32_t mlo = __reduce_max_sync(0xFFFFFFFFu, hi == mhi ? lo : 0u);
    return ((unsigned long long)mhi << 32) | mlo;
}

// Top-k update of one draft row by a whole warp.  `vals` is the row's logits for `ncols` consecutive
// vocabulary columns (first column = vocabulary row `col0`), in shared memory; `list` is the row's k best
// so far (descending keys, 0 = empty) and `tau` the logit of its k-th best (-inf while the list is not
// full).  Lane L looks at columns L, L+32, ...
//   1. bound: the 32 lanes form 8, 16 or 32 groups (whichever is >= k; k <= 32); the smallest group maximum
//      has at least k logits at or above it, so nothing below it can be among the k best of these columns;
//   2. the logits above tau (strictly: a later row loses a tie) and not below the bound are the candidates;
//      a ballot per column group gives each its slot in `cbuf`, and the current list follows them;
//   3. every entry of cbuf counts the entries larger than itself - its rank - and the entries of rank < k
//      form the new list.  Keys are distinct, so ranks are too.  No step depends on the previous candidate,
//      unlike an insertion loop.
// The same pass folds the columns into the row's running (max, sum-exp) in *ms.
// Returns the new tau.  All lanes must call it; NI * 32 >= ncols; `cbuf` holds NI * 32 + k keys.
template <int NI>
__device__ __forceinline__ float warp_topk_update(const float* vals, int ncols, int col0, unsigned long long* list,
                                                  int k, float tau, unsigned long long* cbuf, float2* ms, int lane) {
    float v[NI];
    float lmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int c = lane + 32 * i;
        v[i] = c < ncols ? vals[c] : -INFINITY;
        lmax = fmaxf(lmax, v[i]);
    }
    {   // running log-sum-exp of the row: (max, sum of exp(x - max)), folded over these columns by the warp
        const float2 old = *ms;
        const float bmax = warp_max_f32(lmax);
        const float nmx = fmaxf(old.x, bmax);
        float add = 0.0f;
#pragma unroll
        for (int i = 0; i < NI; ++i) add += __expf(v[i] - nmx);      // exp(-inf) = 0 for the padding
        add = warp_sum_f32(add);
        __syncwarp();
        if (lane == 0) *ms = make_float2(nmx, old.y * __expf(old.x - nmx) + add);
    }
    if (!__any_sync(0xFFFFFFFFu, lmax > tau)) return tau;
    float bound = -INFINITY;
    if (k <= 32) {      // 8 groups of 4 lanes, 16 of 2 or 32 of 1: at least k group maxima, all distinct logits
        float g = lmax;
        if (k <= 16) g = fmaxf(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
        if (k <= 8) g = fmaxf(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) g = fminf(g, __shfl_xor_sync(0xFFFFFFFFu, g, o));
        bound = g;
    }
    int n = 0;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const bool is_cand = v[i] > tau && v[i] >= bound;
        const unsigned int m = __ballot_sync(0xFFFFFFFFu, is_cand);
        if (is_cand) cbuf[n + __popc(m & ((1u << lane) - 1u))] = make_key(v[i], col0 + lane + 32 * i);
        n += __popc(m);
    }
    const int kl = list[0] != 0ull ? k : 0;                       // an empty list (the row's first tile) has nothing to rank
    for (int j = lane; j < kl; j += 32) cbuf[n + j] = list[j];     // empty slots are 0 and rank last
    __syncwarp();
    const int total = n + kl;
    for (int e = lane; e < total; e += 32) {
        const unsigned long long key = cbuf[e];
        int rank = 0;
        for (int f = 0; f < total; ++f) rank += cbuf[f] > key ? 1 : 0;
        if (key != 0ull && rank < k) list[rank] = key;
    }
    __syncwarp();
    const unsigned long long kth = list[k - 1];
    __syncwarp();
    return kth != 0ull ? key_logit(kth) : -INFINITY;
}

// ------------------------------------------------------------------------------------------
// Merge of P partial results of one draft row by one warp.  Partial p is a record in shared memory
// at rec[p * stride]: k keys in descending order (0-padded), then (mx_p, s_p) in slot k.
//   lse = mx + log sum_p s_p * exp(mx_p - mx),  mx = max_p mx_p
// Every list is sorted, so a list's best remaining candidate is its head; lane L owns lists
// L, L+32, ... and k rounds of a warp-wide maximum pick the winners in order.  Keys are unique
// across lists (they carry distinct vocabulary rows), so exactly one head matches each round.
// ------------------------------------------------------------------------------------------
constexpr int kMergeSlots = kMaxParts / 32;

// SLOTS >= ceil(P / 32).  Returns this lane's share of the winners: winner j sits in lane j % 32,
// element j / 32 of `mine` (k <= 64).
template <int SLOTS>
__device__ __forceinline__ void warp_merge_lists_n(const unsigned long long* rec, int stride, int P, int k,
                                                   unsigned long long (&mine)[2]) {
    const int lane = threadIdx.x & 31;
    int head[SLOTS];
    unsigned long long hk[SLOTS];
    unsigned long long local = 0ull;
#pragma unroll
    for (int q = 0; q < SLOTS; ++q) {
        const int p = lane + 32 * q;
        head[q] = 0;
        hk[q] = (p < P) ? rec[(size_t)p * stride] : 0ull;
        local = hk[q] > local ? hk[q] : local;
    }
    mine[0] = mine[1] = 0ull;
    for (int j = 0; j < k; ++j) {
        const unsigned long long best = warp_max_key(local);
        if (best != 0ull && local == best) {          // the one lane whose head won advances that list
            local = 0ull;
#pragma unroll
            for (int q = 0; q < SLOTS; ++q) {
                if (hk[q] == best) {
                    ++head[q];
                    hk[q] = head[q] < k ? rec[(size_t)(lane + 32 * q) * stride + head[q]] : 0ull;
                }
                local = hk[q] > local ? hk[q] : local;
            }
        }
        if ((j & 31) == lane) mine[j >> 5] = best;
    }
}

__device__ __forceinline__ void warp_merge_lists(const unsigned long long* rec, int stride, int P, int k,
                                                 unsigned long long (&mine)[2]) {
    if (P <= 32) warp_merge_lists_n<1>(rec, stride, P, k, mine);
    else if (P <= 64) warp_merge_lists_n<2>(rec, stride, P, k, mine);
    else if (P <= 160) warp_merge_lists_n<5>(rec, stride, P, k, mine);
    else warp_merge_lists_n<kMergeSlots>(rec, stride, P, k, mine);
}

__device__ __forceinline__ float2 warp_merge_ms(const unsigned long long* rec, int stride, int P, int k) {
    const int lane = threadIdx.x & 31;
    float2 v[kMergeSlots];
    float mx = -INFINITY;
#pragma unroll
    for (int q = 0; q < kMergeSlots; ++q) {
        const int p = lane + 32 * q;
        v[q] = p < P ? unpack_ms(rec[(size_t)p * stride + k]) : make_float2(-INFINITY, 0.0f);
        mx = fmaxf(mx, v[q].x);
    }
    mx = warp_max_f32(mx);
    float s = 0.0f;
#pragma unroll
    for (int q = 0; q < kMergeSlots; ++q)
        if (v[q].y > 0.0f) s += v[q].y * __expf(v[q].x - mx);
    return make_float2(mx, warp_sum_f32(s));
}

constexpr int kMergeCand = 256;      // candidate slots per warp in warp_select_topk

// The k best keys of P descending lists (rec[p * stride + j], 0 = empty) without k sequential rounds.
//   1. bound: every lane takes the best head of its lists; the lanes that have one are packed to the
//      front and fall into G groups (lane % G; G = 8, 16 or 32 >= k); the smallest group maximum has at
//      least k keys at or above it, so a key whose logit word is below that bound's cannot be among the
//      k best;
//   2. the remaining keys (typically one or two dozen) are packed into `cbuf` with ballots, walking the
//      lists from their heads and stopping at the first depth where no list has a candidate left;
//   3. each candidate counts the candidates above it: that is its rank, and emit(rank, key) is called
//      for rank < k by the lane that holds the candidate.
// Falls back to the round-based merge when the bound does not apply (k > 32, or fewer than G lists) or the
// candidates do not fit.  emit may be called by several lanes at once, each with a different rank.
template <class Emit>
__device__ __forceinline__ void warp_select_topk(const unsigned long long* rec, int stride, int P, int k,
                                                 unsigned long long* cbuf, Emit emit) {
    const int lane = threadIdx.x & 31;
    bool fast = k <= 32;
    int n = 0;
    if (fast) {
        uint32_t lhead = 0;
#pragma unroll
        for (int q = 0; q < kMergeSlots; ++q) {
            const int p = lane + 32 * q;
            if (p < P) lhead = max(lhead, (uint32_t)(rec[(size_t)p * stride] >> 32));
        }
        // pack the lanes that own a non-empty list to the front, then lane L belongs to group L % G
        const int G = k <= 8 ? 8 : k <= 16 ? 16 : 32;
        const unsigned int have = __ballot_sync(0xFFFFFFFFu, lhead != 0u);
        const int nvalid = __popc(have);
        const unsigned int src = __fns(have, 0, lane + 1);
        uint32_t v = __shfl_sync(0xFFFFFFFFu, lhead, src & 31);
        if (lane >= nvalid) v = 0u;
        fast = nvalid >= G;                                   // every group has a key: G >= k keys are >= the bound
        if (G <= 16) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 16));
        if (G <= 8) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 8));
        const uint32_t bound = __reduce_min_sync(0xFFFFFFFFu, lane < G ? v : 0xFFFFFFFFu);
        for (int q = 0; q < kMergeSlots && q * 32 < P && fast; ++q) {
            const int p = lane + 32 * q;
            for (int j = 0; j < k; ++j) {
                const unsigned long long key = p < P ? rec[(size_t)p * stride + j] : 0ull;
                const bool is_cand = key != 0ull && (uint32_t)(key >> 32) >= bound;
                const unsigned int m = __ballot_sync(0xFFFFFFFFu, is_cand);
                if (m == 0u) break;                           // lists descend: nothing deeper qualifies
                if (n + __popc(m) > kMergeCand) { fast = false; break; }
                if (is_cand) cbuf[n + __popc(m & ((1u << lane) - 1u))] = key;
                n += __popc(m);
            }
        }
    }
    __syncwarp();
    if (fast) {
        for (int e = lane; e < n; e += 32) {
            const unsigned long long key = cbuf[e];
            int rank = 0;
#pragma unroll 4
            for (int f = 0; f < n; ++f) rank += cbuf[f] > key ? 1 : 0;
            if (rank < k) emit(rank, key);
        }
        for (int j = n + lane; j < k; j += 32) emit(j, 0ull);     // fewer than k keys exist at all
    } else {
        unsigned long long mine[2];
        warp_merge_lists(rec, stride, P, k, mine);
        if (lane < k) emit(lane, mine[0]);
        if (lane + 32 < k) emit(lane + 32, mine[1]);
    }
    __syncwarp();
}

// The same for at most 32 lists, one per lane, and k <= kSelectLanesMaxK: the k-th largest head (k rounds of one
// warp-wide maximum on the logit words) bounds the winners from below; each lane walks its own list down to the
// bound, the lanes' counts give the candidates consecutive slots of `cbuf`, and a candidate's rank among them is its
// place.  With one list per lane nothing is packed or grouped: 0.15 us against 0.6 us for the 30 lists of one GEMV
// CTA (k = 1; device timestamps).
constexpr int kSelectLanesMaxK = 12;
template <class Emit>
__device__ __forceinline__ void warp_select_topk_lanes(const unsigned long long* rec, int stride, int P, int k,
                                                       unsigned long long* cbuf, Emit emit) {
    const int lane = threadIdx.x & 31;
    const unsigned long long* mine = rec + (size_t)min(lane, P - 1) * stride;
    uint32_t t = lane < P ? (uint32_t)(mine[0] >> 32) : 0u;
    uint32_t b = 0u;
    for (int r = 0; r < k; ++r) {
        b = __reduce_max_sync(0xFFFFFFFFu, t);
        t = t == b ? 0u : t;
    }
    const uint32_t tau = max(b, 1u);                  // fewer than k lists with a key: every key is a candidate
    int cnt = 0;
    if (lane < P)
        while (cnt < k && (uint32_t)(mine[cnt] >> 32) >= tau) ++cnt;
    int incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
    }
    const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    if (total <= kMergeCand) {
        for (int i = 0; i < cnt; ++i) cbuf[incl - cnt + i] = mine[i];
        __syncwarp();
        for (int e = lane; e < total; e += 32) {
            const unsigned long long key = cbuf[e];
            int rank = 0;
#pragma unroll 4
            for (int f = 0; f < total; ++f) rank += cbuf[f] > key ? 1 : 0;
            if (rank < k) emit(rank, key);
        }
        for (int j = total + lane; j < k; j += 32) emit(j, 0ull);     // fewer than k keys exist at all
    } else {                                          // more ties than the buffer holds
        unsigned long long best[2];
        warp_merge_lists(rec, stride, P, k, best);
        if (lane < k) emit(lane, best[0]);
        if (lane + 32 < k) emit(lane + 32, best[1]);
    }
    __syncwarp();
}

// Winner j of draft row m: its target id (the d2t gather), log-prob and draft index.
__device__ __forceinline__ void write_winner(const HeadOut& o, int m, int j, unsigned long long best, float lse) {
    const size_t out = (size_t)m * o.k + j;
    if (best != 0ull) {
        const int idx = key_index(best);
        o.target_ids[out] = o.d2t ? (o.d2t_offsets ? idx + __ldg(&o.d2t[idx]) : __ldg(&o.d2t[idx])) : idx;
        o.logprobs[out] = key_logit(best) - lse;
        if (o.draft_ids) o.draft_ids[out] = idx;
    } else {   // fewer than k candidates exist only if a wait ran out upstream
        o.target_ids[out] = -1;
        o.logprobs[out] = -INFINITY;
        if (o.draft_ids) o.draft_ids[out] = -1;
    }
}

// Row-wise final merge by one warp, straight from the row-major records in global memory (VT_ROW_*), for the
// warp that published draft row m last.  One round trip to L2 brings every CTA's (max, sum-exp) and its three
// best keys into registers (lane L owns CTAs L, L+32, ...); the log-sum-exp follows from the former.
//   k <= kMergeSelectMaxK with a scratch buffer: the k-th largest of the lanes' best heads (k rounds of one
//   warp-wide maximum on the logit words, nothing else in the loop) bounds the winners from below, since k keys at
//   least that large exist.  The keys not below it - the k winners and rarely more than a few others - get
//   consecutive slots of `cbuf` (a prefix sum of the lanes' counts), and the number of candidates that beat a
//   candidate is its place in the output: one lane per candidate counts, gathers d2t and writes.  Measured for
//   148 lists: 3.2 K against 5.5 K cycles (k = 8), 3.4 K against 6.4 K (k = 10).  A list with three keys at or above
//   the bound may hold a fourth, and more than kMergeCap candidates do not fit: both fall back to
//   the rounds: every list descends, so its best remaining key is its head: k rounds of a warp-wide maximum over
//   the heads pick the winners in order, and the lane whose head won moves on to that list's next key - from its
//   registers, or, for the rare list that places more than three winners, with one more load.  The lanes holding
//   the winners gather d2t and write the outputs together.
// Reads bypass L1: the records were written by other SMs.
constexpr int kMergeCap = 32;              // candidates the scratch buffer of one merging warp holds (u64 each)
constexpr int kMergeSelectMaxK = 12;       // beyond: lists with more than three winners are common, the rounds are faster
template <int SLOTS>
__device__ __forceinline__ void merge_row_global_n(const HeadOut& o, int P, int m, unsigned long long* cbuf) {
    constexpr int kPre = 3;
    const int lane = threadIdx.x & 31;
    const int k = o.k;
    const unsigned long long* msr = VT_ROW_MS(o, m);
    unsigned long long pre[kPre][SLOTS];
    float2 ms[SLOTS];
#pragma unroll
    for (int q = 0; q < SLOTS; ++q) {
        const int p = lane + 32 * q;
        ms[q] = p < P ? unpack_ms(__ldcg(msr + p)) : make_float2(-INFINITY, 0.0f);
#pragma unroll
        for (int j = 0; j < kPre; ++j) pre[j][q] = (p < P && j < k) ? __ldcg(VT_ROW_KEYS(o, m, j) + p) : 0ull;
    }
    float mx = -INFINITY;
#pragma unroll
    for (int q = 0; q < SLOTS; ++q) mx = fmaxf(mx, ms[q].x);
    mx = warp_max_f32(mx);
    float s = 0.0f;
#pragma unroll
    for (int q = 0; q < SLOTS; ++q)
        if (ms[q].y > 0.0f) s += ms[q].y * __expf(ms[q].x - mx);
    s = warp_sum_f32(s);
    const float lse = mx + __logf(s);
    if (lane == 0 && o.lse) o.lse[m] = lse;

    if (cbuf != nullptr && k <= kMergeSelectMaxK) {
        uint32_t t = 0u;
#pragma unroll
        for (int q = 0; q < SLOTS; ++q) t = max(t, (uint32_t)(pre[0][q] >> 32));
        uint32_t b = 0u;
        for (int r = 0; r < k; ++r) {
            b = __reduce_max_sync(0xFFFFFFFFu, t);
            t = t == b ? 0u : t;
        }
        const uint32_t tau = max(b, 1u);              // fewer than k lanes with a key: every key is a candidate
        int cnt = 0;
        bool deep = false;
#pragma unroll
        for (int q = 0; q < SLOTS; ++q) {
#pragma unroll
            for (int j = 0; j < kPre; ++j) cnt += (uint32_t)(pre[j][q] >> 32) >= tau ? 1 : 0;
            deep = deep || (k > kPre && (uint32_t)(pre[kPre - 1][q] >> 32) >= tau);
        }
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += v;
        }
        const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        if (total <= kMergeCap && !__any_sync(0xFFFFFFFFu, deep)) {
            int at = incl - cnt;
#pragma unroll
            for (int q = 0; q < SLOTS; ++q)
#pragma unroll
                for (int j = 0; j < kPre; ++j)
                    if ((uint32_t)(pre[j][q] >> 32) >= tau) cbuf[at++] = pre[j][q];
            __syncwarp();
            if (lane < total) {
                const unsigned long long mine = cbuf[lane];
                int rank = 0, j = 0;
                for (; j + 4 <= total; j += 4) {
                    const unsigned long long a0 = cbuf[j], a1 = cbuf[j + 1], a2 = cbuf[j + 2], a3 = cbuf[j + 3];
                    rank += (a0 > mine ? 1 : 0) + (a1 > mine ? 1 : 0) + (a2 > mine ? 1 : 0) + (a3 > mine ? 1 : 0);
                }
                for (; j < total; ++j) rank += cbuf[j] > mine ? 1 : 0;
                if (rank < k) write_winner(o, m, rank, mine, lse);
            } else if (lane < k) {
                write_winner(o, m, lane, 0ull, lse);  // fewer than k keys in all lists
            }
            __syncwarp();
            return;
        }
    }

    int depth[SLOTS];
    unsigned long long cur[SLOTS];
    unsigned long long local = 0ull, mine0 = 0ull, mine1 = 0ull;   // winners lane and lane + 32
#pragma unroll
    for (int q = 0; q < SLOTS; ++q) {
        depth[q] = 0;
        cur[q] = pre[0][q];
        local = cur[q] > local ? cur[q] : local;
    }
    for (int j = 0; j < k; ++j) {
        const unsigned long long best = warp_max_key(local);
        if (best != 0ull && local == best) {          // keys are unique: exactly one lane, one list
            local = 0ull;
#pragma unroll
            for (int q = 0; q < SLOTS; ++q) {
                if (cur[q] == best) {
                    const int dq = ++depth[q];
                    cur[q] = dq == 1 ? pre[1][q] : dq == 2 ? pre[2][q]
                           : dq < k ? __ldcg(VT_ROW_KEYS(o, m, dq) + lane + 32 * q) : 0ull;
                }
                local = cur[q] > local ? cur[q] : local;
            }
        }
        if (j == lane) mine0 = best;
        if (j == lane + 32) mine1 = best;
    }
    if (lane < k) write_winner(o, m, lane, mine0, lse);
    if (lane + 32 < k) write_winner(o, m, lane + 32, mine1, lse);
    __syncwarp();
}

// `cbuf`: kMergeCap u64 of shared memory for this warp alone, or null.
__device__ inline void merge_row_global(const HeadOut& o, int P, int m, unsigned long long* cbuf) {
    if (P <= 160) merge_row_global_n<5>(o, P, m, cbuf);
    else merge_row_global_n<kMergeSlots>(o, P, m, cbuf);
}

#endif  // __CUDACC__

}  // namespace vt
