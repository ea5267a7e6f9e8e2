// Draft head, tensor-core path for many draft rows: the head contraction as a tcgen05 GEMM with the draft rows on
// the TMEM lanes and a thread-private epilogue.
//
//   D[m, i] = sum_j h[m, j] * W_trim[i, j]       (the d -> k linear head, 2*d*k FLOPs per draft row)
//
// Operand roles: A = h (one or two tiles of 128 draft rows = the 128 TMEM lanes), B = a tile of NT vocabulary rows
// of W_trim (K-major as stored), D = fp32 accumulators of 128 lanes x NT columns in tensor memory, two buffers of
// up to 256 columns, so the epilogue of tile t overlaps the MMAs of tile t+1.  With two A tiles (129-256 draft rows
// in one pass) every weight tile is loaded once and multiplied twice: the weights are streamed once per 256 rows.
//
// tcgen05.ld hands each epilogue thread ONE draft row and a run of consecutive vocabulary logits, so everything a
// row needs is private to a thread and lives in registers: the running (max, sum-exp) and a sorted list of the KR
// best (logit, index) pairs.  No shuffle, no ballot, no shared-memory transposition, no barrier between the
// epilogue threads.  Per chunk of 16 logits a thread folds the chunk into its log-sum-exp state, marks the
// logits above its current KR-th best in a bit mask and parks the chunk in shared memory (its own column, no
// conflicts); the warp then loops while any lane has a marked logit left, each lane inserting its own next
// candidate (a branch-free compare-and-select pass over the KR registers).  A lane's candidates thin out as its
// threshold rises, so the loop runs for the busiest lane's count, not for every logit.
//
// One persistent CTA per SM owns a contiguous range of vocabulary rows:
//   warps 0 .. 4*MT-1  epilogue: warp w reads TMEM lanes 32*(w%4) .. +31 of A tile w/4; never stores a logit
//   next warp          TMA producer: per 64-column k-block one box of W and one box of h per A tile into a
//                      shared-memory ring (h comes from L2: every CTA reads the same h)
//   last warp          MMA issuer: four K=16 tcgen05.mma per k-block and A tile, tcgen05.commit frees the ring slot
// The kernel writes one record per (CTA, draft row) - the row's best k keys and its (max, sum-exp) - and the
// row-wise merge kernel follows it in the stream.
#include <cuda.h>

#include "vt_common.cuh"
#include "vt_launch.h"
#include "vt_tc.cuh"

namespace vt {

constexpr int kRowsMaxThreads = 11 * 32;       // two A tiles: 8 epilogue warps, two producers, the MMA issuer
constexpr int kRowsMaxWStages = 24;
constexpr int kRowsMaxHStages = 6;
constexpr int kRowsAccStride = 256;            // TMEM columns between the two accumulator buffers
constexpr int kRowsChunk = 16;                 // logits a thread takes from TMEM at a time
constexpr int kRowsLoopMax = 4;                // a chunk with at most this many candidates in every lane is taken one by one

struct RowsParams {
    HeadOut out;
    int m_begin, m_count;     // draft rows of this pass: m_count <= 128 * MT
    int MT;                   // A tiles of 128 draft rows: 1 or 2
    int d, nk;                // nk = 64-column k-blocks
    int NT;                   // vocabulary rows per tile: a multiple of 16, <= 256 (<= 128 with two A tiles)
    int kbw;                  // k-blocks one stage of the weight ring holds (one barrier hand-over per stage)
    int w_stages, h_stages;   // the weight ring (from HBM: deep) and the ring of h blocks (from L2: shallow), one k-block each
    uint32_t a_slot;          // bytes of one A tile's k-block (the box's rows rounded up to 8-row groups)
    uint32_t b_slot;          // bytes of one k-block of a weight tile
    uint32_t a_tx, b_tx;      // bytes each TMA box delivers
    uint32_t idesc;
    uint32_t h_off;           // the h ring: h_stages x MT x a_slot
    uint32_t park_off;        // per epilogue warp: kRowsChunk x 32 floats
    uint32_t list_off;        // generic top-k lists [k][epilogue threads] keys (only when the register list is too short)
    uint32_t bar_off, total_smem;   // from the 1024-aligned base
};

__device__ __forceinline__ void rows_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
// KR > 0: the register list holds KR >= k entries.  KR == 0: k is larger than any register list; the list is k
// keys in shared memory (list[j * stride], thread-private) and insertion is a loop.
template <int KR>
__global__ void __launch_bounds__(kRowsMaxThreads, 1)
head_rows_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH, const RowsParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int MT = p.MT, n_epi = 4 * MT, w_warp = n_epi, h_warp = n_epi + 1, mma_warp = n_epi + 2;
    const int G = gridDim.x, cta = blockIdx.x;
    const int Vt = p.out.Vt, k = p.out.k, NT = p.NT, SW = p.w_stages, SH = p.h_stages, nk = p.nk, mc = p.m_count;
    const int row_begin = (int)((long long)cta * Vt / G);
    const int row_end = (int)((long long)(cta + 1) * Vt / G);
    const int nrows = row_end - row_begin;
    const int ntiles = (nrows + NT - 1) / NT;
    const int n_live = (mc + 31) / 32;             // epilogue warps that own at least one draft row
    const int kbw = p.kbw;
    const int wspt = (nk + kbw - 1) / kbw;         // weight-ring stages per tile

    const uint32_t bar_wfull = base + p.bar_off, bar_wempty = bar_wfull + 8u * SW;
    const uint32_t bar_hfull = bar_wempty + 8u * SW, bar_hempty = bar_hfull + 8u * SH;
    const uint32_t bar_accf = bar_hempty + 8u * SH, bar_acce = bar_accf + 16u, bar_drain = bar_acce + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + p.bar_off + 8u * (2 * SW + 2 * SH + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (lane == 0) {      // descriptor fetches overlap the barrier set-up below
        if (warp == w_warp) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
        if (warp == h_warp) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmH) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < SW; ++s) {
            mbar_init(bar_wfull + 8u * s, 1);
            mbar_init(bar_wempty + 8u * s, 1);
        }
        for (int s = 0; s < SH; ++s) {
            mbar_init(bar_hfull + 8u * s, 1);
            mbar_init(bar_hempty + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_accf + 8u * b, 1);
            mbar_init(bar_acce + 8u * b, n_live);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    // The MMA always reads 128 A rows; rows past the pass's last row hold whatever follows the A block in shared
    // memory (or zeros the TMA filled in).  They only feed TMEM lanes whose results no thread keeps.
    if (warp == mma_warp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched only shared memory, tensor memory and kernel parameters.  Every thread now waits
    // until the previous kernel in the stream has completed.
    grid_dependency_wait();
    if (tid == 0) grid_launch_dependents();

    auto fail = [&]() {
        *abort_flag = 1;
        atomicOr(&p.out.hdr->status, kStatusTimeout);
    };

    if (warp == w_warp) {
        // ------------------------------------------------------------------ TMA producer of the weight ring (HBM)
        if (lane == 0) {
            const int total = ntiles * wspt;
            const uint64_t stream_once = l2_policy_evict_first();
            auto issue = [&](int q, int s) {
                const int t = q / wspt, ks = (q - t * wspt) * kbw;
                const int nb = min(kbw, nk - ks);
                const uint32_t bar = bar_wfull + 8u * s;
                mbar_arrive_expect_tx(bar, (uint32_t)nb * p.b_tx);
                for (int kb = 0; kb < nb; ++kb)
                    tma_load_2d_hint(base + ((uint32_t)s * (uint32_t)kbw + (uint32_t)kb) * p.b_slot, &tmW, (ks + kb) * kBoxK,
                                     row_begin + t * NT, bar, stream_once);
            };
            int s = 0, issued = 0;
            uint32_t wrap = 0;          // times the ring has wrapped: stage s is free once its (wrap-1)-th use retired
            for (int q = 0; q < total; ++q) {
                if (wrap > 0 && !mbar_wait(bar_wempty + 8u * s, (wrap - 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                issue(q, s);
                ++issued;
                if (++s == SW) { s = 0; ++wrap; }
            }
            if (*abort_flag) {   // let copies in flight land before the CTA gives its shared memory back
                const unsigned long long deadline = global_timer_ns() + kWaitLimitNs;
                for (int i = max(0, issued - SW); i < issued; ++i)
                    (void)mbar_wait_until(bar_wfull + 8u * (i % SW), (uint32_t)(i / SW) & 1u, deadline);
            }
        }
    } else if (warp == h_warp) {
        // ------------------------------------------------------------------ TMA producer of the h ring (L2)
        if (lane == 0) {
            const int total = ntiles * nk;
            int s = 0, issued = 0;
            uint32_t wrap = 0;
            for (int q = 0; q < total; ++q) {
                if (wrap > 0 && !mbar_wait(bar_hempty + 8u * s, (wrap - 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                const int kb = q % nk;
                const uint32_t bar = bar_hfull + 8u * s;
                mbar_arrive_expect_tx(bar, (uint32_t)MT * p.a_tx);
                for (int a = 0; a < MT; ++a)
                    tma_load_2d(base + p.h_off + ((uint32_t)s * (uint32_t)MT + (uint32_t)a) * p.a_slot, &tmH, kb * kBoxK,
                                p.m_begin + 128 * a, bar);
                ++issued;
                if (++s == SH) { s = 0; ++wrap; }
            }
            if (*abort_flag) {
                const unsigned long long deadline = global_timer_ns() + kWaitLimitNs;
                for (int i = max(0, issued - SH); i < issued; ++i)
                    (void)mbar_wait_until(bar_hfull + 8u * (i % SH), (uint32_t)(i / SH) & 1u, deadline);
            }
        }
    } else if (warp == mma_warp) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int sw = 0, sh = 0;
            uint32_t wphase = 0, hphase = 0;
            bool ok = true;
            const uint64_t w_desc0 = smem_desc_sw128(base);                    // descriptor of the weight ring's first byte
            const uint64_t h_desc0 = smem_desc_sw128(base + p.h_off);
            const uint32_t a_units = p.a_slot >> 4, b_units = p.b_slot >> 4;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int buf = t & 1;
                if (t >= 2 && !mbar_wait(bar_acce + 8u * buf, (uint32_t)((t >> 1) - 1) & 1u)) { fail(); break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kRowsAccStride);
                for (int ks = 0; ks < nk && ok; ks += kbw) {
                    if (!mbar_wait(bar_wfull + 8u * sw, wphase)) { fail(); ok = false; break; }
                    const int nb = min(kbw, nk - ks);
                    for (int kb = 0; kb < nb; ++kb) {
                        if (!mbar_wait(bar_hfull + 8u * sh, hphase)) { fail(); ok = false; break; }
                        if (*abort_flag) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t b_desc = w_desc0 + (uint64_t)(((uint32_t)sw * (uint32_t)kbw + (uint32_t)kb) * b_units);
                        const uint64_t a_desc = h_desc0 + (uint64_t)((uint32_t)sh * (uint32_t)MT * a_units);
                        // 16 bf16 = 32 bytes = 2 descriptor address units per MMA along K; the A tiles take turns, so
                        // consecutive MMAs write different accumulators
#pragma unroll
                        for (uint32_t kk = 0; kk < 4; ++kk)
                            for (int a = 0; a < MT; ++a)
                                tc_mma_bf16(d_tmem + (uint32_t)(a * 128), a_desc + (uint64_t)((uint32_t)a * a_units) + 2u * kk,
                                            b_desc + 2u * kk, p.idesc, ((ks | kb) != 0 || kk != 0) ? 1u : 0u);
                        tc_commit(bar_hempty + 8u * sh);
                        if (++sh == SH) { sh = 0; hphase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit(bar_wempty + 8u * sw);
                    if (++sw == SW) { sw = 0; wphase ^= 1u; }
                }
                if (ok) tc_commit(bar_accf + 8u * buf);
            }
            if (*abort_flag) {   // every MMA issued so far must retire before TMEM is freed
                tc_commit(bar_drain);
                (void)mbar_wait(bar_drain, 0u);
            }
        }
    } else if (warp < n_live) {
        // ------------------------------------------------------------------ epilogue: one draft row per thread
        const int a = warp >> 2, q = warp & 3;
        const int m_local = a * 128 + q * 32 + lane;
        const bool live = m_local < mc;
        const int row = p.m_begin + m_local;                                   // among the call's draft rows
        float* park = reinterpret_cast<float*>(smem + p.park_off) + (size_t)warp * (kRowsChunk * 32) + lane;
        constexpr int KL = KR > 0 ? KR : 1;
        float v[KL];
        int ix[KL];
#pragma unroll
        for (int j = 0; j < KL; ++j) { v[j] = -INFINITY; ix[j] = -1; }
        // generic list (KR == 0): k keys, thread-private, [j][epilogue thread]
        const int list_stride = n_epi * 32;
        unsigned long long* list = reinterpret_cast<unsigned long long*>(smem + p.list_off) + (warp * 32 + lane);
        if (KR == 0)
            for (int j = 0; j < k; ++j) list[(size_t)j * list_stride] = 0ull;
        float thr = -INFINITY;                   // generic list: logit of its last entry (-inf while it is not full)
        int filled = 0;
        float mx = -INFINITY, ssum = 0.0f;
        bool ok = true;
        for (int t = 0; t < ntiles; ++t) {
            const int buf = t & 1;
            // warp-uniform decisions: tcgen05.ld needs the whole warp
            if (ok && !__any_sync(0xFFFFFFFFu, *abort_flag != 0)) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_accf + 8u * buf, (uint32_t)(t >> 1) & 1u));
                if (!ok) fail();
            } else {
                ok = false;
            }
            if (!ok) break;
            tc_fence_after();
            const int row0 = row_begin + t * NT;
            const int ncols = min(NT, row_end - row0);
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * kRowsAccStride + a * 128);
            for (int c0 = 0; c0 < ncols; c0 += kRowsChunk) {
                uint32_t r[kRowsChunk];
                rows_ld16(taddr + (uint32_t)c0, r);
                tc_wait_ld();
                const int nv = min(kRowsChunk, ncols - c0);
                float x[kRowsChunk];
#pragma unroll
                for (int c = 0; c < kRowsChunk; ++c) x[c] = __uint_as_float(r[c]);
                if (nv < kRowsChunk) {                   // columns past the CTA's rows are not its logits
#pragma unroll
                    for (int c = 0; c < kRowsChunk; ++c)
                        if (c >= nv) x[c] = -INFINITY;
                }
                if (wants_logits(p.out) && live) {
#pragma unroll
                    for (int c = 0; c < kRowsChunk; ++c)
                        if (c < nv) store_logit(p.out, row, row0 + c0 + c, x[c]);
                }
                if (p.out.store_only) continue;
                // running log-sum-exp of the row: (max, sum of exp(x - max))
                float cm = x[0];
#pragma unroll
                for (int c = 1; c < kRowsChunk; ++c) cm = fmaxf(cm, x[c]);
                const float nm = fmaxf(mx, cm);
                const float nml = nm * kLog2e;
                float add = 0.0f;
#pragma unroll
                for (int c = 0; c < kRowsChunk; ++c) add += ex2_approx(fmaf(x[c], kLog2e, -nml));   // exp(-inf) = 0
                ssum = ssum * ex2_approx((mx - nm) * kLog2e) + add;                                   // first chunk: 0 * 0
                mx = nm;
                // top-k.  Candidates are the logits above the thread's current last entry (strictly: a later row
                // loses a tie).  How many a lane has shrinks quickly as its list fills.
                const float t0 = KR > 0 ? v[KL - 1] : thr;
                uint32_t mask = 0;
#pragma unroll
                for (int c = 0; c < kRowsChunk; ++c) mask |= (x[c] > t0) ? (1u << c) : 0u;
                if (KR == 0 && filled < k) mask = nv >= kRowsChunk ? 0xFFFFu : ((1u << nv) - 1u);
                const int most = (int)__reduce_max_sync(0xFFFFFFFFu, (unsigned)__popc(mask));
                if (most == 0) continue;
                if (KR > 0 && most > kRowsLoopMax) {
                    // many candidates somewhere in the warp: insert the whole chunk, no loop, no vote, every
                    // compare-and-select independent of its neighbours
#pragma unroll
                    for (int c = 0; c < kRowsChunk; ++c) rows_insert<KL>(v, ix, x[c], row0 + c0 + c);
                    continue;
                }
                // few candidates: each lane inserts its own next one while any lane has one left
#pragma unroll
                for (int c = 0; c < kRowsChunk; ++c) park[c * 32] = x[c];
                do {
                    float xv = -INFINITY;
                    int xi = 0;
                    if (mask != 0u) {
                        const int c = __ffs(mask) - 1;
                        mask &= mask - 1u;
                        xv = park[c * 32];
                        xi = row0 + c0 + c;
                    }
                    if (KR > 0) {
                        rows_insert<KL>(v, ix, xv, xi);
                    } else if (xv > thr || (filled < k && xv > -INFINITY)) {
                        const unsigned long long kth = list_insert(list, list_stride, k, make_key(xv, xi));
                        if (filled < k) ++filled;
                        if (filled == k) thr = key_logit(kth);
                    }
                } while (__any_sync(0xFFFFFFFFu, mask != 0u));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acce + 8u * buf);   // the MMAs of the tile after next may start
        }
        // the row's record: best k keys and (max, sum-exp); an unfilled entry is key 0
        if (live && !p.out.store_only) {
            if (KR > 0) {
#pragma unroll
                for (int j = 0; j < KL; ++j)
                    if (j < k) VT_ROW_KEYS(p.out, row, j)[cta] = ix[j] >= 0 ? make_key(v[j], ix[j]) : 0ull;
            } else {
                for (int j = 0; j < k; ++j) VT_ROW_KEYS(p.out, row, j)[cta] = list[(size_t)j * list_stride];
            }
            VT_ROW_MS(p.out, row)[cta] = pack_ms(mx, ssum);
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == mma_warp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static vt_status get_encode(EncodeTiledFn* out) {
    static std::atomic<EncodeTiledFn> fn{nullptr};
    EncodeTiledFn f = fn.load(std::memory_order_acquire);
    if (!f) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q);
        if (e != cudaSuccess) return cuda_fail(e);
        if (q != cudaDriverEntryPointSuccess || !ptr) return cuda_fail(cudaErrorSymbolNotFound);
        f = reinterpret_cast<EncodeTiledFn>(ptr);
        fn.store(f, std::memory_order_release);
    }
    *out = f;
    return VT_OK;
}

// bf16 matrix [rows, d] row-major, box = 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
vt_status make_tensor_map_bf16(CUtensorMap* map, const void* ptr, int rows, int d, int box_rows) {
    EncodeTiledFn enc;
    vt_status r = get_encode(&enc);
    if (r != VT_OK) return r;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBoxK, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    CUresult cr = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return cr == CUDA_SUCCESS ? VT_OK : driver_fail((int)cr);
}

// Tile height for the most rows a CTA owns: a multiple of 16 up to `cap`, with the least padding - rows a tile
// loads past the CTA's range are wasted HBM traffic - and, among equals, the height nearest 128 from below (with
// two or more tiles per CTA all epilogues but the last hide behind the stream, and the last one is short).
static int choose_tile_rows(int rows, int cap) {
    if (rows <= 96) return ((rows + 15) / 16) * 16;
    int best = cap, best_cost = 1 << 30;
    for (int nt = 96; nt <= cap; nt += 16) {
        const int pad = (rows + nt - 1) / nt * nt - rows;
        const int cost = pad * 1024 + (nt <= 128 ? 128 - nt : nt);
        if (cost < best_cost) {
            best_cost = cost;
            best = nt;
        }
    }
    return best;
}


// Geometry and shared-memory layout of one pass of mc draft rows; false if it does not fit.
static bool rows_plan(int mc, int MT, int d, int Vt, int k, int grid, RowsParams* p) {
    const int R = (Vt + grid - 1) / grid;
    p->m_count = mc;
    p->MT = MT;
    p->d = d;
    p->nk = (d + kBoxK - 1) / kBoxK;
    p->NT = choose_tile_rows(R, MT == 2 ? 128 : 256);
    const int a_rows = MT == 2 ? 128 : mc;                      // rows of the h box (rows past M arrive as zeros)
    p->a_tx = (uint32_t)a_rows * 128u;
    p->b_tx = (uint32_t)p->NT * 128u;
    p->a_slot = (p->a_tx + 1023u) & ~1023u;
    p->b_slot = (p->b_tx + 1023u) & ~1023u;
    // instruction descriptor: D fp32, A and B bf16, both K-major, N = NT, M = 128
    p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p->NT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const int n_epi = 4 * MT;
    const size_t park_bytes = (size_t)n_epi * kRowsChunk * 32 * 4;
    const size_t list_bytes = topk_list_regs(k) == 0 ? (size_t)k * n_epi * 32 * 8 : 0;
    const size_t bar_bytes = (size_t)(2 * kRowsMaxWStages + 2 * kRowsMaxHStages + 5) * 8 + 16;
    // An MMA reads 128 A rows = 16 KB from its A slot whatever the box delivered: what the last slot of the h ring
    // reads past the ring's end must still lie inside the allocation (it lands in the scratch that follows).
    const size_t overhang = p->a_slot >= 16384 ? 0 : 16384 - p->a_slot;
    const size_t tail = std::max(park_bytes + list_bytes + bar_bytes + 128, overhang);
    // The weights come from HBM, whose latency under load (2-3 us) times the SM's share of the bandwidth asks for
    // 130 KB and more in flight; h comes from L2 and needs only enough blocks to cover that shorter round trip.
    // So h gets a shallow ring of its own and everything else goes to the weights.
    const size_t h_blk = (size_t)MT * p->a_slot;
    p->h_stages = std::min(kRowsMaxHStages, std::max(MT == 2 ? 3 : 2, std::min(p->nk, (int)(65536 / h_blk))));
    p->kbw = std::max(1, std::min(std::min(4, p->nk), (int)((28 * 1024 + p->b_slot / 2) / p->b_slot)));
    const size_t w_stage = (size_t)p->kbw * p->b_slot;
    if ((size_t)kMaxDynSmem < 1024 + tail + (size_t)p->h_stages * h_blk + 2 * w_stage) return false;
    const size_t avail = (size_t)kMaxDynSmem - 1024 - tail - (size_t)p->h_stages * h_blk;
    p->w_stages = (int)std::min<size_t>(kRowsMaxWStages, avail / w_stage);
    const size_t w_ring = (size_t)p->w_stages * w_stage;
    p->h_off = (uint32_t)w_ring;
    const size_t h_end = w_ring + (size_t)p->h_stages * h_blk;
    p->park_off = (uint32_t)h_end;
    p->list_off = (uint32_t)(h_end + park_bytes);
    p->bar_off = (uint32_t)((p->list_off + list_bytes + 127) & ~(size_t)127);
    const size_t need = std::max((size_t)p->bar_off + bar_bytes, h_end + overhang);
    p->total_smem = (uint32_t)(need + 1024);
    return p->total_smem <= (uint32_t)kMaxDynSmem;
}

template <int KR>
static vt_status launch_rows(const CUtensorMap& tmW, const CUtensorMap& tmH, const RowsParams& p, int grid, cudaStream_t st) {
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(head_rows_kernel<KR>), kMaxDynSmem, &smem_configured);
        rc != VT_OK)
        return rc;
    cudaError_t e = launch_pdl(head_rows_kernel<KR>, grid, (4 * p.MT + 3) * 32, p.total_smem, st, tmW, tmH, p);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

vt_status launch_head_mma(const HeadCall& c, cudaStream_t st, int* grid_out) {
    int sms = 0;
    vt_status r = device_sm_count(&sms);
    if (r != VT_OK) return r;
    const int grid = head_grid(sms, c.Vt, 16);
    *grid_out = grid;
    const int KR = topk_list_regs(c.out.k);
    // passes of up to 256 draft rows (two A tiles), else 128; every pass must fit before anything is launched
    auto pass_rows = [&](int m0, RowsParams* q) -> int {
        const int left = c.M - m0;
        if (left > 128 && rows_plan(std::min(256, left), 2, c.d, c.Vt, c.out.k, grid, q)) return std::min(256, left);
        if (rows_plan(std::min(128, left), 1, c.d, c.Vt, c.out.k, grid, q)) return std::min(128, left);
        return 0;
    };
    for (int m0 = 0; m0 < c.M;) {
        RowsParams q{};
        const int mc = pass_rows(m0, &q);
        if (mc == 0) return VT_ERR_UNSUPPORTED;
        m0 += mc;
    }
    for (int m0 = 0; m0 < c.M;) {
        RowsParams p{};
        const int mc = pass_rows(m0, &p);
        p.out = c.out;
        p.m_begin = m0;
        CUtensorMap tmW, tmH;
        r = make_tensor_map_bf16(&tmW, c.W, c.Vt, c.d, p.NT);
        if (r != VT_OK) return r;
        r = make_tensor_map_bf16(&tmH, c.h, c.M, c.d, (int)(p.a_tx / 128u));
        if (r != VT_OK) return r;
        switch (KR) {
            case 4: r = launch_rows<4>(tmW, tmH, p, grid, st); break;
            case 8: r = launch_rows<8>(tmW, tmH, p, grid, st); break;
            case 10: r = launch_rows<10>(tmW, tmH, p, grid, st); break;
            case 16: r = launch_rows<16>(tmW, tmH, p, grid, st); break;
            default: r = launch_rows<0>(tmW, tmH, p, grid, st); break;
        }
        if (r != VT_OK) return r;
        m0 += mc;
    }
    return c.out.store_only ? VT_OK : launch_merge_rowmajor(c.out, grid, st);
}

}  // namespace vt
