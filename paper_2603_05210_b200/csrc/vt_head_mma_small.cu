// Draft head, tensor-core path with the vocabulary rows on the TMEM lanes (any M, 128 or 256 draft rows per launch).
//
//   D[i, m] = sum_j W_trim[row0 + i, j] * h[m, j]       (the d -> k linear head, 2*d*k FLOPs per draft row)
//
// Operand roles: A = a tile of up to 128 vocabulary rows of W_trim (K-major as stored), B = h (N = M rounded up
// to 16, at most 128 rows: the draft rows, zero-filled or don't-care beyond M), D = fp32 accumulator of 128 lanes
// x N columns in tensor memory.  tcgen05.ld then hands each of 128 epilogue threads one vocabulary row and its
// logits for 16 draft rows, so reading a tile out is cheap whatever M is, and a weight tile needs no padding rows:
// the tile height is the CTA's row count split evenly (<= 128), rows of the MMA past it compute on stale shared
// memory and land in lanes nobody reads.  Each k-block of h rides in the ring next to its weights (it comes from
// L2: every CTA reads the same h); only with M <= 8 and short tiles does h stay in shared memory for the whole
// kernel instead.
//   warps 0-7   (0-15 when M > 8) the epilogue.  Warps 0-3 read TMEM (warp q: lanes 32q..32q+31) and lay the tile's
//               logits out per draft row in shared memory, 32 draft rows at a time.  Warp w owns draft rows w,
//               w + 8 (16), ...: running (max, sum-exp) and top-k of the row over the tile (warp_topk_update), at
//               the end the row's record, and with at most 16 draft rows its arrival ticket and, for the warp that
//               arrives last of all CTAs, the row's final merge (merge_row_global): no CTA-wide barrier and no CTA
//               ever waits for another.  With more rows a warp owns several, and merging them one after the other
//               would put several round trips to L2 per row on the critical path: the kernel then only writes
//               the records and a one-warp-per-row merge kernel follows it.
//               From 17 draft rows on (from 9 or 13 when a CTA has a single tile, see small_plan) the epilogue is
//               thread-per-row instead (KR > 0 below): warps 0-3 scan, warps 4-7 sum, records only; and with more
//               than 64 draft rows on single-tile CTAs two such groups of eight warps take alternate passes of 64
//               draft rows while pairs of CTAs share each MMA (PAIR below).
//   next warp   TMA producer: boxes of 64 columns x tile-height rows of W (and the k-block of h) into a
//               shared-memory ring
//   last warp   MMA issuer: four K=16 tcgen05.mma (M=128, N) per 64-column k-block, tcgen05.commit frees the ring
//               stage; two accumulator buffers in TMEM
// Short tiles (a CTA with at most 64 rows: V_trim up to about 9,500) would waste the MMA: it costs the same 60-80
// cycles for 28 live rows as for 128, and 4 * nk of them per tile is then what the call takes.  The kernel then
// folds G = 4 (2) k-blocks into one MMA instead: TMEM lanes 32g..32g+31 (64g..) hold the tile's rows for
// k-block G*j + g, and since the blocks of h for consecutive k-blocks lie one after the other (resident or in the
// ring), a B operand of N = G * (rows of a block) rows is the matching k-blocks of h.  Lane group g against column
// group g is the wanted partial sum (the other G - 1 column groups are cross terms nobody reads); the readers add
// the G partial sums through shared memory.  G times fewer MMAs per tile.
// The weight stream is the bound (arithmetic intensity = M FLOP/B).
#include <cuda.h>

#include "vt_common.cuh"
#include "vt_launch.h"
#include "vt_tc.cuh"

namespace vt {

constexpr int kSmMaxEpiWarps = 16;            // warps 0-7, or 0-15 when there are more than 8 draft rows; 0-3 also read TMEM
constexpr int kSmThreads = (kSmMaxEpiWarps + 2) * 32;     // at most: the epilogue warps, then the producer, then the MMA issuer
constexpr int kSmMaxM = 128;                  // draft rows per launch = MMA N
constexpr int kSmMaxMChunked = 256;           // ... when a CTA has one tile and the thread-per-row epilogue takes it 64 draft rows at a time
constexpr int kChunkRows = 64;
constexpr int kLgRows = 32;                   // draft rows whose tile logits shared memory holds at a time
constexpr int kSmMaxStages = 32;
constexpr int kLgPitch = 132;                 // floats between draft rows of the tile's logits in shared memory
constexpr int kHParts = 4;                    // h arrives in this many parts so the first MMAs need not wait for all of it
constexpr int kSmCand = 128 + VT_MAX_K;       // candidate keys per epilogue warp (one tile's columns + the list)

struct SmallParams {
    HeadOut out;
    int M;                    // draft rows of this launch, <= kSmMaxM (<= kSmMaxMChunked with chunked thread-per-row)
    int m_begin;              // first of them among the call's draft rows
    int merge_in_kernel;      // 1: one draft row per epilogue warp, merged by the last warp to publish it; 0: a merge kernel follows
    int n_epi;                // epilogue warps: 8, or 16 when M > 8 with the warp-per-row epilogue; the block has
                              // two more (producer, MMA issuer)
    int lg_rows;              // draft rows whose tile logits shared memory holds at a time: kLgRows with warp-per-row;
                              // with thread-per-row all of them, or 64 at a time when the CTA has a single tile
    uint32_t scratch_stride;  // bytes of one epilogue warp's candidate buffer: (128 + k) keys
    int N;                    // MMA N: M rounded up to a multiple of 16
    int h_resident;           // 1: h sits in shared memory for the whole kernel (h_off); 0: one block per k-block in the ring
    uint32_t tmem_cols;       // allocation: 2 accumulators of N columns, a power of two >= 32
    int d, nk;                // nk = 64-column k-blocks
    int G;                    // k-blocks folded into one MMA: 128 / (tile height rounded up to 32 or 64), or 1
    int NG;                   // accumulator columns per folded k-block = rows of an h block: 8 (M <= 8), else M rounded up to 16
    int nsb;                  // MMA steps along d: ceil(nk / G) "super-blocks" of G k-blocks
    int TH;                   // vocabulary rows per tile (<= 128)
    int kb_per_stage;         // k-blocks one ring stage holds
    int n_stages;
    uint32_t slot_bytes;      // one k-block of a tile in the ring: TH rounded up to whole 8-row groups x 128 B
    uint32_t sub_bytes;       // with folded k-blocks: bytes between the k-blocks of one MMA step in a slot (128 / G rows x 128 B)
    uint32_t part_off;        // with folded k-blocks: the readers' partial sums [G][NG][64] floats
    uint32_t blk_bytes;       // slot_bytes, plus h_blk when h rides in the ring (the h block follows the weights)
    uint32_t stage_bytes;
    uint32_t w_tx;            // bytes one W box delivers (TH * 128)
    uint32_t h_blk;           // bytes of one k-block of h: 8 rows (M <= 8) or N rows x 128 B
    uint32_t h_off, lg_off, list_off, scratch_off, bar_off, total_smem;   // from the 1024-aligned base
    int acce_count;           // arrivals that free an accumulator buffer: the reading warps of the CTA (of both CTAs of a pair)
    uint32_t lg_bytes;        // one logits buffer (chunked thread-per-row has two, one per group of eight epilogue warps)
    uint32_t idesc;
};

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr) : "memory");
}
// Barrier among the four TMEM-reading warps.
__device__ __forceinline__ void reader_barrier() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
// Barrier among the epilogue warps only (the producer and the MMA issuer never join it).
__device__ __forceinline__ void epi_barrier(int threads) { asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory"); }
__device__ __forceinline__ void epi_barrier(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }

// KR == 0: the warp-per-row epilogue (any k).  KR > 0: the thread-per-row epilogue (more than 16 draft rows, fewer on
// single-tile CTAs), with a register list of KR >= k entries per thread.
// PAIR: launched as clusters of two CTAs that share one MMA of 256 lanes (thread-per-row in passes of 64 draft rows
// only): each CTA streams its own vocabulary rows and HALF of every k-block of h, so h crosses from L2 to the SMs
// 74 times instead of 148 - with 128 and more draft rows that traffic, not the weight stream, was the bound.
template <int KR, bool PAIR>
__global__ void __launch_bounds__(kSmThreads, 1)
head_mma_small_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH,
                      const SmallParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int producer_warp = p.n_epi, mma_warp = p.n_epi + 1;     // the block has n_epi + 2 warps
    const int G = gridDim.x, cta = blockIdx.x;
    const int Vt = p.out.Vt, k = p.out.k, M = p.M, TH = p.TH, S = p.n_stages, nk = p.nk, KF = p.G, nsb = p.nsb;   // KF: k-blocks folded into one MMA
    const int row_begin = (int)((long long)cta * Vt / G);
    const int row_end = (int)((long long)(cta + 1) * Vt / G);
    const int nrows = row_end - row_begin;
    const int ntiles = (nrows + TH - 1) / TH;
    const int h_part = (nk + kHParts - 1) / kHParts;          // k-blocks per part of h
    const uint32_t pair_rank = PAIR ? cluster_cta_rank() : 0u;
    const bool leader = pair_rank == 0u;                      // issues the MMAs (always true without pairs)

    float* lg = reinterpret_cast<float*>(smem + p.lg_off);                                  // [M][kLgPitch]
    unsigned long long* lists = reinterpret_cast<unsigned long long*>(smem + p.list_off);   // [M][k]
    float2* ms_s = reinterpret_cast<float2*>(lists + (size_t)M * k);                         // [kSmMaxM]
    float* tau_s = reinterpret_cast<float*>(ms_s + kSmMaxM);                                 // [kSmMaxM] k-th best logit so far
    unsigned char* scratch = smem + p.scratch_off + (uint32_t)(warp & (kSmMaxEpiWarps - 1)) * p.scratch_stride;
    const uint32_t bar_full = base + p.bar_off, bar_empty = bar_full + 8u * S;
    const uint32_t bar_accf = bar_empty + 8u * S, bar_acce = bar_accf + 16u;
    const uint32_t bar_h = bar_acce + 16u, bar_drain = bar_h + 8u * kHParts;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + p.bar_off + 8u * (2 * S + 4 + kHParts + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (warp == producer_warp && lane == 0) {      // descriptor fetches overlap the barrier set-up below
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmH) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_accf + 8u * b, 1);
            mbar_init(bar_acce + 8u * b, (uint32_t)p.acce_count);
        }
        for (int j = 0; j < kHParts; ++j) mbar_init(bar_h + 8u * j, 1);
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (KR == 0) {
        for (int i = tid; i < M * k; i += blockDim.x) lists[i] = 0ull;
        if (tid < kSmMaxM) {
            ms_s[tid] = make_float2(-INFINITY, 0.0f);
            tau_s[tid] = -INFINITY;
        }
    }
    // With 8 rows of h per k-block the MMA's rows 8-15 alias whatever follows the block (the next k-block of a
    // resident h, the next ring slot otherwise): accumulator columns nobody reads.  After the last block of a
    // resident h that is this pad.
    // With folded k-blocks the last MMA step may name k-blocks past d: zeros here, zeros (out-of-range boxes)
    // from the TMA on the weight side.
    if (p.h_resident)
        for (int i = tid; i < 256 * KF; i += blockDim.x)
            reinterpret_cast<uint32_t*>(smem + p.h_off + (uint32_t)nk * p.h_blk)[i] = 0u;
    if (warp == mma_warp) {
        if constexpr (PAIR) {     // the same warp of both CTAs
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"(p.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"(p.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    fence_proxy_async();          // the zeroed pad is read by the tensor core (async proxy)
    tc_fence_before();
    if constexpr (PAIR) cluster_sync_all();      // the other CTA's barriers are initialised before anything arrives on them
    else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched only shared memory, tensor memory and kernel parameters, so under programmatic
    // dependent launch it overlaps the previous kernel's tail.  Every thread now waits until the previous kernel
    // has completed and its writes are visible; no global memory is touched before that.  (Requesting weight tiles ahead of this wait, for weights the caller declares constant,
    // was measured to cost 1-4 % here: the early requests compete with the previous call's last tiles.)
    grid_dependency_wait();
    if (tid == 0) grid_launch_dependents();

    auto fail = [&]() {
        *abort_flag = 1;
        atomicOr(&p.out.hdr->status, kStatusTimeout);
    };

    if (warp == producer_warp) {
        // ------------------------------------------------------------------ TMA producer: the weight stream
        if (lane == 0) {
            const int kbs = p.kb_per_stage;
            const int spt = (nsb + kbs - 1) / kbs;          // ring stages per tile
            const int total = ntiles * spt;                 // ring stages of this CTA, in issue order
            const uint64_t stream_once = l2_policy_evict_first();
            const uint32_t h_tx = p.h_resident ? 0u : p.h_blk;
            const int h_row0 = p.m_begin + (PAIR ? (int)pair_rank * (p.N >> 1) : 0);     // a pair's CTAs hold N/2 rows of h each
            // stage q of the CTA's sequence into ring slot s: the weight boxes and the matching blocks of h
            auto issue = [&](int q, int s) {
                const int t = q / spt, ks = (q - t * spt) * kbs;
                const int row0 = row_begin + t * TH;
                const int nb = min(kbs, nsb - ks);
                const uint32_t bar = bar_full + 8u * s;
                if constexpr (PAIR) {
                    // both CTAs' bytes are counted on the leader's barrier, which its producer arms
                    if (leader) mbar_arrive_expect_tx(bar, 2u * (uint32_t)nb * (p.w_tx + h_tx));
                    const uint32_t lbar = cluster_map_shared(bar, 0u);
                    for (int kb = 0; kb < nb; ++kb) {
                        const uint32_t dst = base + (uint32_t)s * p.stage_bytes + (uint32_t)kb * p.blk_bytes;
                        tma_load_2d_pair_hint(dst, &tmW, (ks + kb) * kBoxK, row0, lbar, stream_once);
                        tma_load_2d_pair(dst + p.slot_bytes, &tmH, (ks + kb) * kBoxK, h_row0, lbar);
                    }
                    return;
                }
                mbar_arrive_expect_tx(bar, (uint32_t)nb * (uint32_t)KF * (p.w_tx + h_tx));
                for (int kb = 0; kb < nb; ++kb) {
                    const uint32_t dst = base + (uint32_t)s * p.stage_bytes + (uint32_t)kb * p.blk_bytes;
                    // k-block KF * (ks + kb) + g goes to lanes g * (128 / KF) ...; one past d is all zero fill
                    for (int g = 0; g < KF; ++g)
                        tma_load_2d_hint(dst + (uint32_t)g * p.sub_bytes, &tmW, ((ks + kb) * KF + g) * kBoxK, row0, bar,
                                         stream_once);
                    if (!p.h_resident)                // the matching k-blocks of h, one block after the other behind the weights
                        for (int g = 0; g < KF; ++g)
                            tma_load_2d(dst + p.slot_bytes + (uint32_t)g * p.h_blk, &tmH, ((ks + kb) * KF + g) * kBoxK,
                                        h_row0, bar);
                }
            };
            int s = 0, issued = 0;
            uint32_t wrap = 0;          // times the ring has wrapped: stage s is free once its (wrap-1)-th use retired
            for (int q = 0; q < total; ++q) {
                if (wrap > 0 && !mbar_wait(bar_empty + 8u * s, (wrap - 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                issue(q, s);
                ++issued;
                if (++s == S) { s = 0; ++wrap; }
            }
            if (*abort_flag && leader) {   // let copies in flight land before the CTA gives its shared memory back
                // (in a pair the leader's barriers count both CTAs' copies, and the other CTA leaves only after
                // the leader has passed this point: the cluster-wide barrier at the end)
                const unsigned long long deadline = global_timer_ns() + kWaitLimitNs;
                for (int i = max(0, issued - S); i < issued; ++i)
                    (void)mbar_wait_until(bar_full + 8u * (i % S), (uint32_t)(i / S) & 1u, deadline);
            }
        }
    } else if (warp == mma_warp) {
        // ------------------------------------------------------------------ MMA issuer (in a pair: the leader's)
        if (lane == 0 && leader) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint64_t desc0 = smem_desc_sw128(base);                      // descriptor of the ring's first byte
            const uint64_t h_desc0 = smem_desc_sw128(base + p.h_off);
            const uint32_t stage_units = p.stage_bytes >> 4, slot_units = p.slot_bytes >> 4, h_units = p.h_blk >> 4;
            const uint32_t blk_units = p.blk_bytes >> 4;
            const int kbs = p.kb_per_stage;
            int h_ready = 0;                                                   // k-blocks of h known to have landed
            for (int t = 0; t < ntiles && ok; ++t) {
                const int buf = t & 1;
                if (t >= 2 && !mbar_wait(bar_acce + 8u * buf, (uint32_t)((t >> 1) - 1) & 1u)) { fail(); break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.N);
                for (int ks = 0; ks < nsb && ok; ks += kbs) {
                    const int nb = min(kbs, nsb - ks);
                    while (p.h_resident && h_ready < min(nk, (ks + nb) * KF)) {
                        if (!mbar_wait(bar_h + 8u * (uint32_t)(h_ready / h_part), 0u)) { fail(); ok = false; break; }
                        h_ready += h_part;
                    }
                    if (!ok) break;
                    if (!mbar_wait(bar_full + 8u * s, phase)) { fail(); ok = false; break; }
                    if (*abort_flag) { ok = false; break; }
                    tc_fence_after();
                    for (int kb = 0; kb < nb; ++kb) {
                        const uint64_t a_desc = desc0 + (uint64_t)((uint32_t)s * stage_units + (uint32_t)kb * blk_units);
                        const uint64_t b_desc = p.h_resident ? h_desc0 + (uint64_t)((uint32_t)((ks + kb) * KF) * h_units)
                                                             : a_desc + slot_units;
                        // 16 bf16 = 32 bytes = 2 descriptor address units per MMA along K
                        if constexpr (PAIR) {
                            tc_mma_bf16_pair(d_tmem, a_desc, b_desc, p.idesc, (ks | kb) != 0);
                            tc_mma_bf16_pair(d_tmem, a_desc + 2u, b_desc + 2u, p.idesc, 1u);
                            tc_mma_bf16_pair(d_tmem, a_desc + 4u, b_desc + 4u, p.idesc, 1u);
                            tc_mma_bf16_pair(d_tmem, a_desc + 6u, b_desc + 6u, p.idesc, 1u);
                        } else {
                            tc_mma_bf16(d_tmem, a_desc, b_desc, p.idesc, (ks | kb) != 0);
                            tc_mma_bf16(d_tmem, a_desc + 2u, b_desc + 2u, p.idesc, 1u);
                            tc_mma_bf16(d_tmem, a_desc + 4u, b_desc + 4u, p.idesc, 1u);
                            tc_mma_bf16(d_tmem, a_desc + 6u, b_desc + 6u, p.idesc, 1u);
                        }
                    }
                    // the stage is free (in both CTAs of a pair) once these MMAs have read it
                    if constexpr (PAIR) tc_commit_pair_both(bar_empty + 8u * s);
                    else tc_commit(bar_empty + 8u * s);
                    if (++s == S) { s = 0; phase ^= 1u; }
                }
                if (ok) {
                    if constexpr (PAIR) tc_commit_pair_both(bar_accf + 8u * buf);
                    else tc_commit(bar_accf + 8u * buf);
                }
            }
            if (*abort_flag) {   // every MMA issued so far must retire before TMEM is freed
                if constexpr (PAIR) tc_commit_pair(bar_drain);
                else tc_commit(bar_drain);
                (void)mbar_wait(bar_drain, 0u);
            }
        }
    } else if (KR > 0 && warp < p.n_epi) {
        // ------------------------------------------------------------------ epilogue, one draft row per thread
        // Warps 0-3 read a finished tile out of TMEM (lane = vocabulary row, 16 draft rows per load) and lay it
        // out per draft row in shared memory.  Then each of their threads owns ONE draft row (and, with fewer than
        // 128 draft rows, one of several column ranges of it) and scans its logits alone, keeping a sorted list
        // of the KR best (logit, index) pairs in registers - no shuffle, no ballot, no barrier between threads.
        // A row's first scan bounds the candidates first: the KR-th largest of the maxima of groups of 4 or 8
        // logits has at least KR logits at or above it, so nothing below it can be among the KR best; the few
        // logits that pass are marked in a bit mask and inserted one per turn of a loop that runs for the busiest
        // lane's count.  Later tiles are filtered by the list's own last entry.  Warps 4-7 mirror that thread
        // assignment and fold the same logits into the rows' running (max, sum-exp): the two kinds of work use
        // different pipes (compare/select against multiply-add and exp2) and hide each other's latencies.
        constexpr int KL = KR > 0 ? KR : 1;
        // A CTA with a single tile takes its draft rows CH = 64 at a time and writes their records right away:
        // shared memory then holds 64 rows of logits per pass instead of all of them and the ring gets the
        // difference.  Two groups of eight warps then work side by side, each with its own buffers and barrier,
        // on every other pass: the scans wait on latencies more than on issue slots, so twice the warps finish
        // in nearly half the time.
        const int grp = warp >> 3, ngrp = p.n_epi >> 3;                // this warp's group; groups
        const int wg = warp & 7;                                       // the warp within its group
        const int gtid = tid & 255;
        const int bar_id = 1 + 2 * grp;                                // named barriers 1 and 3 (2: the readers')
        float* lg = reinterpret_cast<float*>(smem + p.lg_off + (uint32_t)grp * p.lg_bytes);
        const bool scanner = wg < 4;
        const int w4 = warp & 3;
        const int CH = p.lg_rows;                                      // draft rows per pass of the epilogue
        const int nch = (M + CH - 1) / CH;                             // 1 unless the CTA has a single tile
        const int RG = (min(M, CH) + 31) >> 5;                         // groups of 32 draft rows: 1 .. 4
        const int Q = RG == 1 ? 4 : RG == 2 ? 2 : 1;                   // column ranges a row is split into
        const int rg = w4 % RG, part = w4 / RG;
        const bool works = part < Q;                                   // warp-uniform
        const int m_own = rg * 32 + lane;                              // the thread's draft row of this pass
        const int xs = RG * 32;
        float v[KL];
        int ix[KL];
#pragma unroll
        for (int j = 0; j < KL; ++j) { v[j] = -INFINITY; ix[j] = -1; }
        float mx = -INFINITY, ssum = 0.0f;
        int seen = 0;                                                  // logits this thread has scanned (the same in every lane of a warp)
        unsigned long long* xl = reinterpret_cast<unsigned long long*>(lg);      // [(part * RG * 32 + row) * (KL + 1)], see below
        for (int t = 0; t < ntiles; ++t) {
            const int buf = t & 1;
            const int row0 = row_begin + t * TH;
            const int nv = min(TH, row_end - row0);
            bool got = false;
            if (scanner) {
                // warp-uniform decisions: tcgen05.ld needs the whole warp
                if (!__any_sync(0xFFFFFFFFu, *abort_flag != 0)) {
                    got = __all_sync(0xFFFFFFFFu, mbar_wait(bar_accf + 8u * buf, (uint32_t)(t >> 1) & 1u));
                    if (!got) fail();
                }
            }
            for (int ch = grp; ch < nch; ch += ngrp) {
                const int m0 = ch * CH, Mc = min(CH, M - m0);          // this pass: draft rows m0 .. m0 + Mc - 1 of the launch
                const float* rowp = lg + (size_t)min(m_own, Mc - 1) * kLgPitch;   // lanes past the last row re-read it and keep nothing
                if (scanner) {
                    const uint32_t taddr = tmem_base + ((uint32_t)(w4 * 32) << 16) + (uint32_t)(buf * p.N);
                    if (KF > 1) {
                        // Folded k-blocks (never with several passes): this warp's lanes are k-group g of tile rows
                        // r0 + lane, and columns NG*g .. NG*g + NG - 1 of the accumulator are their partial logits
                        // for the draft rows.
                        const int SR = 128 / KF, NG = p.NG, g = (w4 * 32) / SR, r = w4 * 32 + lane - g * SR;
                        float* partial = reinterpret_cast<float*>(smem + p.part_off);
                        if (got) {
                            tc_fence_after();
                            for (int c0 = 0; c0 < NG; c0 += 16) {
                                uint32_t u[16];
                                tc_ld16(taddr + (uint32_t)(NG * g + c0), u);
                                tc_wait_ld();
#pragma unroll
                                for (int m = 0; m < 16; ++m) partial[(g * NG + c0 + m) * 64 + r] = __uint_as_float(u[m]);
                            }
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_acce + 8u * buf);
                        }
                        reader_barrier();                              // all four readers' partial sums are in place
                        for (int e = gtid; e < M * SR; e += 128) {
                            const int m = e >> (KF == 4 ? 5 : 6), rr = e & (SR - 1);            // SR = 128 / KF is 32 or 64
                            if (rr >= nv) continue;
                            float sum = 0.0f;
                            for (int gg = 0; gg < KF; ++gg) sum += partial[(gg * p.NG + m) * 64 + rr];
                            lg[m * kLgPitch + rr] = sum;
                            if (wants_logits(p.out)) store_logit(p.out, p.m_begin + m, row0 + rr, sum);
                        }
                    } else if (got) {
                        const int i = w4 * 32 + lane;                  // TMEM lane = vocabulary row of the tile
                        if (ch == grp) tc_fence_after();
                        for (int c1 = 0; c1 < Mc; c1 += 16) {          // 16 draft rows per load
                            uint32_t u[16];
                            tc_ld16(taddr + (uint32_t)(m0 + c1), u);
                            tc_wait_ld();
                            if (i < nv) {
#pragma unroll
                                for (int m = 0; m < 16; ++m)
                                    if (c1 + m < Mc) lg[(c1 + m) * kLgPitch + i] = __uint_as_float(u[m]);
                                if (wants_logits(p.out)) {
#pragma unroll
                                    for (int m = 0; m < 16; ++m)
                                        if (c1 + m < Mc)
                                            store_logit(p.out, p.m_begin + m0 + c1 + m, row0 + i, __uint_as_float(u[m]));
                                }
                            }
                        }
                        if (ch + ngrp >= nch) {                        // this group has read its share of the accumulator
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) {                           // the MMAs of the tile after next may start
                                if constexpr (PAIR) mbar_arrive_cluster(cluster_map_shared(bar_acce + 8u * buf, 0u));
                                else mbar_arrive(bar_acce + 8u * buf);
                            }
                        }
                    }
                }
                // A later tile of a CTA that works in passes: the rows' records so far (this CTA's own, from L2) join
                // the merge below as one more list.  The summing threads fetch them now, under the scans.
                constexpr int PV = (KL + 1) / 2;                       // keys of the old record per summing thread (Q = 2)
                unsigned long long prevk[PV], prevms = 0ull;
#pragma unroll
                for (int i = 0; i < PV; ++i) prevk[i] = 0ull;
                const bool carry = nch > 1 && t > 0;
                if (carry && !scanner && works && m_own < Mc && !p.out.store_only) {
                    const int row = p.m_begin + m0 + m_own;
#pragma unroll
                    for (int i = 0; i < PV; ++i) {
                        const int j = part + Q * i;
                        prevk[i] = j < k ? __ldcg(VT_ROW_KEYS(p.out, row, j) + cta) : 0ull;
                    }
                    if (part == 0) prevms = __ldcg(VT_ROW_MS(p.out, row) + cta);
                }
                epi_barrier(bar_id, 256);                                      // the pass's logits are in shared memory
                // ---- the thread's own columns [cb, ce) of its draft row.  After a wait ran out the buffer holds
                // older logits: whatever is computed from them belongs to a call that reports the time-out.
                const int seg = (((nv + Q - 1) / Q) + 3) & ~3;         // multiples of 4: 16-byte loads
                const int cb = part * seg, ce = min(nv, cb + seg), n = ce - cb;
                if (works && n > 0 && !p.out.store_only) {
                    if (scanner) row_scan_topk<KL>(rowp, cb, ce, row0, seen >= KL, v, ix, smem + p.scratch_off + (uint32_t)grp * (kRowQueue * 128) + gtid);
                    else row_scan_lse(rowp, cb, ce, mx, ssum);
                }
                seen += max(n, 0);
                epi_barrier(bar_id, 256);                                      // the buffer may be overwritten
                if (nch == 1 && t + 1 < ntiles) continue;              // lists and sums carry over to the next tile
                // ---- the rows' records: best k keys and (max, sum-exp).  The logits buffer is free now: it takes
                // every thread's list (or sums); the range-0 scanner of a row merges its column ranges and writes
                // the record.
                if (works) {
                    unsigned long long* mine = xl + (size_t)(part * xs + m_own) * (KL + 1);
                    if (scanner) {
#pragma unroll
                        for (int j = 0; j < KL; ++j) mine[j] = ix[j] >= 0 ? make_key(v[j], ix[j]) : 0ull;
                    } else {
                        mine[KL] = pack_ms(mx, ssum);
                        if (carry && m_own < Mc) {                             // list Q: the record of the earlier tiles
                            unsigned long long* old = xl + (size_t)(Q * xs + m_own) * (KL + 1);
#pragma unroll
                            for (int i = 0; i < PV; ++i)
                                if (part + Q * i < KL) old[part + Q * i] = prevk[i];
                            if (part == 0) old[KL] = prevms;
                        }
                    }
                }
                epi_barrier(bar_id, 256);
                const int NL = Q + (carry ? 1 : 0);                            // sorted lists per row
                if (scanner && part == 0 && m_own < Mc && !p.out.store_only) {
                    const int row = p.m_begin + m0 + m_own;                    // among the call's draft rows
                    // NL sorted lists: the best remaining key is the largest head, k times
                    int pos[4] = {0, 0, 0, 0};
                    for (int j = 0; j < k; ++j) {
                        unsigned long long best = 0ull;
                        int bq = 0;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (q < NL && pos[q] < KL) {
                                const unsigned long long key = xl[(size_t)(q * xs + m_own) * (KL + 1) + pos[q]];
                                if (key > best) { best = key; bq = q; }
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) pos[q] += (q == bq && best != 0ull) ? 1 : 0;
                        VT_ROW_KEYS(p.out, row, j)[cta] = best;
                    }
                    float cmx = -INFINITY;
                    for (int q = 0; q < NL; ++q) cmx = fmaxf(cmx, unpack_ms(xl[(size_t)(q * xs + m_own) * (KL + 1) + KL]).x);
                    float cs = 0.0f;
                    for (int q = 0; q < NL; ++q) {
                        const float2 ms = unpack_ms(xl[(size_t)(q * xs + m_own) * (KL + 1) + KL]);
                        if (ms.y > 0.0f) cs += ms.y * __expf(ms.x - cmx);
                    }
                    VT_ROW_MS(p.out, row)[cta] = pack_ms(cmx, cs);
                }
                if (ch + ngrp < nch || t + 1 < ntiles) {
                    // the group's next pass starts from empty lists, once the exchange buffer has been read
#pragma unroll
                    for (int j = 0; j < KL; ++j) { v[j] = -INFINITY; ix[j] = -1; }
                    mx = -INFINITY;
                    ssum = 0.0f;
                    seen = 0;
                    epi_barrier(bar_id, 256);
                }
            }
        }
    } else if (KR == 0 && warp < p.n_epi) {
        // ------------------------------------------------------------------ epilogue warps
        const int n_epi = p.n_epi;
        if (warp == n_epi - 1 && lane == 0 && ntiles > 0 && p.h_resident) {
            // h, fetched once: every CTA needs all of it, one box per k-block, in kHParts parts
            for (int j = 0; j < kHParts; ++j) {
                const int k0 = j * h_part, k1 = min(nk, k0 + h_part);
                if (k0 >= k1) break;
                mbar_arrive_expect_tx(bar_h + 8u * j, (uint32_t)(k1 - k0) * p.h_blk);
                for (int kb = k0; kb < k1; ++kb)
                    tma_load_2d(base + p.h_off + (uint32_t)kb * p.h_blk, &tmH, kb * kBoxK, p.m_begin, bar_h + 8u * j);
            }
        }
        __syncwarp();
        unsigned long long* cbuf = reinterpret_cast<unsigned long long*>(scratch);
        // Every epilogue warp passes the same barriers per tile whatever happens, so none can be left waiting at
        // one: after a wait has run out the remaining tiles only skip their work.
        for (int t = 0; t < ntiles; ++t) {
            const int buf = t & 1;
            const int row0 = row_begin + t * TH;
            const int nv = min(TH, row_end - row0);
            bool got_tile = false;
            if (warp < 4) {
                // warp-uniform decisions: tcgen05.ld needs the whole warp
                bool got = false;
                if (!__any_sync(0xFFFFFFFFu, *abort_flag != 0)) {
                    got = __all_sync(0xFFFFFFFFu, mbar_wait(bar_accf + 8u * buf, (uint32_t)(t >> 1) & 1u));
                    if (!got) fail();
                }
                const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * p.N);
                if (KF > 1) {
                    // Folded k-blocks: this warp's lanes are k-group g of tile rows r0 + lane, and columns
                    // NG*g .. NG*g + NG - 1 of the accumulator are their partial logits for the draft rows.
                    const int SR = 128 / KF, NG = p.NG, g = (warp * 32) / SR, r = warp * 32 + lane - g * SR;
                    float* part = reinterpret_cast<float*>(smem + p.part_off);
                    if (got) {
                        tc_fence_after();
                        if (NG == 8) {
                            uint32_t v[8];
                            tc_ld8(taddr + (uint32_t)(8 * g), v);
                            tc_wait_ld();
#pragma unroll
                            for (int m = 0; m < 8; ++m) part[(g * 8 + m) * 64 + r] = __uint_as_float(v[m]);
                        } else {
                            for (int c0 = 0; c0 < NG; c0 += 16) {
                                uint32_t v[16];
                                tc_ld16(taddr + (uint32_t)(NG * g + c0), v);
                                tc_wait_ld();
#pragma unroll
                                for (int m = 0; m < 16; ++m) part[(g * NG + c0 + m) * 64 + r] = __uint_as_float(v[m]);
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_acce + 8u * buf);
                    }
                    reader_barrier();                                  // all four readers' partial sums are in place
                    for (int e = tid; e < M * SR; e += 128) {
                        const int m = e >> (KF == 4 ? 5 : 6), rr = e & (SR - 1);            // SR = 128 / KF is 32 or 64
                        if (rr >= nv) continue;
                        float sum = 0.0f;
                        for (int gg = 0; gg < KF; ++gg) sum += part[(gg * p.NG + m) * 64 + rr];
                        lg[m * kLgPitch + rr] = sum;
                        if (wants_logits(p.out)) store_logit(p.out, p.m_begin + m, row0 + rr, sum);
                    }
                }
                got_tile = got;
            }
            // The tile's logits go through shared memory kLgRows draft rows at a time: readers lay a chunk out per
            // draft row, every epilogue warp folds its rows of the chunk, and the buffer is free for the next chunk.
            for (int c0 = 0; c0 < M; c0 += kLgRows) {
                const int mc = min(kLgRows, M - c0);
                if (warp < 4 && KF == 1 && got_tile) {
                    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * p.N + c0);
                    const int i = warp * 32 + lane;                    // TMEM lane = vocabulary row of the tile
                    if (c0 == 0) tc_fence_after();
                    for (int c1 = 0; c1 < mc; c1 += 16) {              // 16 draft rows per load
                        uint32_t r[16];
                        tc_ld16(taddr + (uint32_t)c1, r);
                        tc_wait_ld();
                        if (i < nv) {
#pragma unroll
                            for (int m = 0; m < 16; ++m)
                                if (c1 + m < mc) lg[(c1 + m) * kLgPitch + i] = __uint_as_float(r[m]);
                            if (wants_logits(p.out)) {
#pragma unroll
                                for (int m = 0; m < 16; ++m)
                                    if (c1 + m < mc) store_logit(p.out, p.m_begin + c0 + c1 + m, row0 + i, __uint_as_float(r[m]));
                            }
                        }
                    }
                    if (c0 + kLgRows >= M) {                           // the accumulator is read out
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_acce + 8u * buf);   // the MMAs of the tile after next may start
                    }
                }
                epi_barrier(n_epi * 32);                               // the chunk's logits are in shared memory
                for (int m = c0 + warp; m < c0 + mc && !p.out.store_only; m += n_epi) {
                    const float tau = warp_topk_update<4>(lg + (m - c0) * kLgPitch, nv, row0, lists + (size_t)m * k, k,
                                                          tau_s[m], cbuf, ms_s + m, lane);
                    __syncwarp();
                    if (lane == 0) tau_s[m] = tau;
                    __syncwarp();
                }
                epi_barrier(n_epi * 32);                               // ... and may be overwritten
            }
        }
        // ------------------------------------------------------------------ publish, and merge if last
        // The warp owns its rows from the first tile to the outputs: record -> fence -> ticket; the warp that
        // draws the last ticket of a row (over all CTAs) merges that row.  No CTA-wide step in between.
        for (int m = warp; m < M && !p.out.store_only; m += n_epi) {
            const int row = p.m_begin + m;                             // among the call's draft rows
            const unsigned long long* list = lists + (size_t)m * k;
            for (int j = lane; j < k; j += 32) VT_ROW_KEYS(p.out, row, j)[cta] = list[j];
            if (lane == 0) {
                const float2 ms = ms_s[m];
                VT_ROW_MS(p.out, row)[cta] = pack_ms(ms.x, ms.y);
            }
            if (!p.merge_in_kernel) continue;      // the records are complete when the kernel is
            __threadfence();
            __syncwarp();
            unsigned int ticket = 0;
            if (lane == 0) ticket = atomicAdd(&p.out.hdr->row_ticket[row], 1u);
            ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
            if (ticket == (unsigned int)G - 1u) {
                __threadfence();
                merge_row_global(p.out, G, row, cbuf);
                if (lane == 0) p.out.hdr->row_ticket[row] = 0u;        // ready for the next call
            }
        }
        if (warp == n_epi - 1 && lane == 0 && ntiles > 0 && p.h_resident && *abort_flag) {
            // let the copies of h land before the CTA gives its shared memory back
            const unsigned long long deadline = global_timer_ns() + kWaitLimitNs;
            for (int j = 0; j < kHParts && j * h_part < nk; ++j) (void)mbar_wait_until(bar_h + 8u * j, 0u, deadline);
        }
    }

    tc_fence_before();
    if constexpr (PAIR) cluster_sync_all();      // neither CTA leaves while the other's MMAs or arrivals may still reach it
    else __syncthreads();
    tc_fence_after();
    if (warp == mma_warp) {
        if constexpr (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------ host
// Tile geometry and shared-memory layout for a shape; false if it does not fit.
static bool small_plan(int M, int d, int Vt, int k, int grid, bool pairs_ok, SmallParams* p, int* list_regs, bool* pair_out) {
    if (M < 1 || M > kSmMaxMChunked) return false;
    const int R = (Vt + grid - 1) / grid;                    // most rows a CTA owns
    const int nt = (R + 127) / 128;
    // More than 16 draft rows: one thread per draft row, as long as a register list holds k entries.  With four
    // and more tiles per CTA and at most 64 draft rows the warp-per-row epilogue hides behind the stream as well
    // and leaves more shared memory to the ring (measured at V_trim = 128256: 180 against 194 us).  With one tile
    // per CTA nothing hides the epilogue, and thread-per-row is the faster one from 13 draft rows on, from 9 when
    // k > 8 (measured at d = 4096, V_trim = 16384, k = 10: M = 16 37.3 -> 33.0 us, M = 9 36.0 -> 33.4 us; k = 8:
    // M = 16 32.4 -> 31.5 us, M = 9..12 equal) although the rows are then merged by a second launch.
    const bool many = M > 16 && !(M <= 64 && nt >= 4);
    const bool few_single_tile = nt == 1 && (M > 12 || (M > 8 && k > 8));
    const int KR = (many || few_single_tile) ? topk_list_regs(k) : 0;
    *list_regs = KR;
    // More than 64 draft rows: the epilogue takes a tile 64 draft rows at a time and writes (from the second tile on:
    // merges into) their records at once, so nothing but the records carries over between passes; that halves the
    // logits buffer at 128 draft rows and lets one launch take 256.
    // With several tiles per CTA and at most 96 draft rows one pass per tile with the lists kept in registers is as
    // good or better (measured at V_trim = 128256, M = 65: 181 against 202 us; M = 100: equal; V_trim = 32000, M = 100:
    // 72 against 64 us).
    const bool chunked = KR > 0 && M > kChunkRows && (nt == 1 || M > 96);
    if (M > kSmMaxM && !chunked) return false;
    // ... and then two CTAs share each MMA, each fetching half of h
    const bool pair = chunked && pairs_ok && (grid & 1) == 0;
    *pair_out = pair;
    const int n_round = pair ? 32 : 16;                      // MMA N: a pair's CTAs hold whole 16-row blocks of h each
    p->M = M;
    p->d = d;
    p->nk = (d + kBoxK - 1) / kBoxK;
    p->TH = (R + nt - 1) / nt;
    p->w_tx = (uint32_t)p->TH * 128u;
    p->h_blk = M <= 8 ? 1024u : (uint32_t)(((M + n_round - 1) / n_round) * n_round) * (pair ? 64u : 128u);
    p->lg_rows = chunked ? kChunkRows : KR > 0 ? ((M + 15) / 16) * 16 : std::min(M, kLgRows);
    // thread-per-row: all of the tile's draft rows at once, and room for the column ranges' lists at the end
    const size_t lg_bytes = KR > 0 ? (std::max((size_t)p->lg_rows * kLgPitch * 4, (size_t)128 * (KR + 1) * 8) + 127) & ~(size_t)127
                                   : ((size_t)p->lg_rows * kLgPitch * 4 + 127) & ~(size_t)127;
    const size_t list_bytes = KR > 0 ? 0 : (((size_t)M * k * 8 + (size_t)kSmMaxM * 12) + 127) & ~(size_t)127;
    p->n_epi = KR > 0 ? (chunked ? 16 : 8) : M > 8 ? kSmMaxEpiWarps : 8;
    p->acce_count = chunked ? (pair ? 16 : 8) : 4;
    p->merge_in_kernel = KR == 0 && M <= p->n_epi;
    p->scratch_stride = (uint32_t)(kSmCand - VT_MAX_K + k) * 8u;
    // thread-per-row: the scanners' candidate queues, kRowQueue entries of one byte for each of 128 threads
    const size_t scratch_bytes = KR > 0 ? (size_t)kRowQueue * 128 * (chunked ? 2 : 1) : ((size_t)p->n_epi * p->scratch_stride + 127) & ~(size_t)127;
    const size_t bar_bytes = (size_t)(2 * kSmMaxStages + 4 + kHParts + 1) * 8 + 16;
    p->lg_bytes = (uint32_t)lg_bytes;
    const size_t lg_total = lg_bytes * (chunked ? 2 : 1);
    const size_t common = 1024 + lg_total + list_bytes + scratch_bytes + bar_bytes + 128;
    // h resident only for M <= 8 (8 rows per k-block) and short tiles, where little is streamed and the fold by two
    // wants it; otherwise it rides in the ring: measured 1-3 % faster at 109-row tiles once the ring (then six
    // stages instead of five) is filled ahead of the dependency wait.
    for (int attempt = (M <= 8 && R <= 64) ? 0 : 1; attempt < 3; ++attempt) {
        const int resident = attempt == 0;
        // short tiles: fold G k-blocks into each MMA, as far as the accumulator (G * NG columns) and the partial sums allow
        p->NG = M <= 8 ? 8 : ((M + 15) / 16) * 16;            // = rows of one h block
        p->G = p->TH <= 32 ? 4 : p->TH <= 64 ? 2 : 1;
        // measured at d = 4096 with h in the ring: G = 4 gains (M = 16, 32 at 28 rows per CTA), G = 2 loses (M = 32 at 56
        // rows, M = 48 and 64 at 28), so there it is four or nothing
        if (!resident && (p->G < 4 || 4 * p->NG > 128)) p->G = 1;
        p->nsb = (p->nk + p->G - 1) / p->G;
        p->N = p->G > 1 ? p->NG * p->G : ((M + n_round - 1) / n_round) * n_round;
        p->sub_bytes = (uint32_t)(128 / p->G) * 128u;
        p->slot_bytes = p->G > 1 ? 16384u : (uint32_t)((p->TH + 7) / 8) * 1024u;
        p->tmem_cols = 32;
        while (p->tmem_cols < 2u * (uint32_t)p->N) p->tmem_cols *= 2;
        // instruction descriptor: D fp32, A and B bf16, both K-major, N, M = 128
        // (a pair's MMA: M = 256, 128 lanes in either CTA)
        p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p->N >> 3) << 17) | ((uint32_t)((pair ? 256 : 128) >> 4) << 24);
        const size_t part_bytes = p->G > 1 ? (size_t)p->G * p->NG * 64 * 4 : 0;
        // + zeros for what the last MMA step reads past h: rows 8-15 of an unfolded step, whole k-blocks of a folded one
        const size_t h_bytes = resident ? (size_t)p->nk * p->h_blk + 1024 * (size_t)p->G : 0;
        p->h_resident = resident;
        p->blk_bytes = p->slot_bytes + (resident ? 0u : (uint32_t)p->G * p->h_blk);
        // Every hand-over of a stage costs the issuing thread some 300 cycles beside its MMAs, and that thread is what
        // limits how fast an SM can take weights: two k-blocks per stage at least (24-32 KB), and three where four
        // such stages still fit and the tiles are tall (measured at 109-row tiles, d = 4096: 1-5 % faster than two;
        // with only three stages left, or with folded short tiles, slower), one only as the last resort.
        p->kb_per_stage = std::max(2, std::min(4, (int)((28 * 1024 + p->blk_bytes / 2) / p->blk_bytes)));
        if (p->G == 1 && p->kb_per_stage == 2 && p->nk >= 6 &&
            common + h_bytes + part_bytes + 4 * (size_t)(3 * p->blk_bytes) <= (size_t)kMaxDynSmem)
            p->kb_per_stage = 3;
        if (attempt == 2) p->kb_per_stage = 1;
        p->kb_per_stage = std::min(p->kb_per_stage, p->nsb);
        p->stage_bytes = p->blk_bytes * (uint32_t)p->kb_per_stage;
        const size_t fixed = common + h_bytes + part_bytes;
        if (fixed + 3 * (size_t)p->stage_bytes > (size_t)kMaxDynSmem) continue;
        const int S = (int)std::min<size_t>(kSmMaxStages, ((size_t)kMaxDynSmem - fixed) / p->stage_bytes);
        if (S < (resident && p->G == 1 ? 4 : 3)) continue;
        const size_t ring = (size_t)S * p->stage_bytes;
        p->n_stages = S;
        p->h_off = (uint32_t)ring;                                            // stages are multiples of 1024 bytes
        p->part_off = (uint32_t)(ring + h_bytes);
        p->lg_off = (uint32_t)(p->part_off + part_bytes);
        p->list_off = (uint32_t)(p->lg_off + lg_total);
        p->scratch_off = (uint32_t)(p->list_off + list_bytes);
        p->bar_off = (uint32_t)(p->scratch_off + scratch_bytes);
        // An MMA always reads 128 A rows = 16 KB from its slot's first byte and N B rows from its h block's: past
        // a short tile or an 8-row h block that is whatever follows in shared memory, which must still be inside
        // the allocation.
        const size_t need = std::max((size_t)p->bar_off + bar_bytes, ring + 16384);
        p->total_smem = (uint32_t)(need + 1024);
        if (p->total_smem <= (uint32_t)kMaxDynSmem) return true;
    }
    return false;
}

template <int KR, bool PAIR>
static vt_status launch_small(const CUtensorMap& tmW, const CUtensorMap& tmH, const SmallParams& p, int grid, cudaStream_t st) {
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(head_mma_small_kernel<KR, PAIR>), kMaxDynSmem, &smem_configured);
        rc != VT_OK)
        return rc;
    cudaError_t e = PAIR ? launch_pdl_cluster2(head_mma_small_kernel<KR, PAIR>, grid, (p.n_epi + 2) * 32, p.total_smem, st, tmW, tmH, p)
                         : launch_pdl(head_mma_small_kernel<KR, PAIR>, grid, (p.n_epi + 2) * 32, p.total_smem, st, tmW, tmH, p);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

// Whether `grid` CTAs of the pair kernel with the largest shared-memory request can all be resident as clusters of
// two (asked once per process; the answer does not depend on the list length).
static bool pairs_schedulable(int grid) {
    static std::atomic<int> cached{-1};          // most clusters the device holds at once
    int n = cached.load(std::memory_order_acquire);
    if (n < 0) {
        static std::atomic<unsigned long long> smem_configured{0};
        if (ensure_max_dyn_smem(reinterpret_cast<const void*>(head_mma_small_kernel<10, true>), kMaxDynSmem, &smem_configured) != VT_OK)
            return false;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3((unsigned)(10 * 32));
        cfg.dynamicSmemBytes = kMaxDynSmem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, head_mma_small_kernel<10, true>, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            clusters = 0;
        }
        n = clusters;
        cached.store(n, std::memory_order_release);
    }
    return 2 * n >= grid;
}

vt_status launch_head_mma_small(const HeadCall& c, cudaStream_t st, int* grid_out) {
    int sms = 0;
    vt_status r = device_sm_count(&sms);
    if (r != VT_OK) return r;
    const int grid = head_grid(sms, c.Vt, 16);
    *grid_out = grid;
    const bool pairs_ok = c.M > kChunkRows && (grid & 1) == 0 && pairs_schedulable(grid);
    // draft rows per pass: 256 where the plan takes them (one tile per CTA, thread-per-row), else 128
    int KR = 0, pass = kSmMaxM;
    bool pair = false;
    if (c.M > kSmMaxM) {
        SmallParams q{};
        if (small_plan(std::min(kSmMaxMChunked, c.M), c.d, c.Vt, c.out.k, grid, pairs_ok, &q, &KR, &pair)) pass = kSmMaxMChunked;
    }
    // every pass must fit before anything is launched
    for (int m0 = 0; m0 < c.M; m0 += pass) {
        SmallParams q{};
        if (!small_plan(std::min(pass, c.M - m0), c.d, c.Vt, c.out.k, grid, pairs_ok, &q, &KR, &pair)) return VT_ERR_UNSUPPORTED;
    }
    bool merge_after = false;
    for (int m0 = 0; m0 < c.M; m0 += pass) {           // each pass streams the weights once for its draft rows
        SmallParams p{};
        small_plan(std::min(pass, c.M - m0), c.d, c.Vt, c.out.k, grid, pairs_ok, &p, &KR, &pair);
        p.out = c.out;
        p.m_begin = m0;
        if (c.M > pass) p.merge_in_kernel = 0;          // row tickets serve single-pass calls only
        merge_after = !p.merge_in_kernel;
        CUtensorMap tmW, tmH;
        r = make_tensor_map_bf16(&tmW, c.W, c.Vt, c.d, p.TH);
        if (r != VT_OK) return r;
        r = make_tensor_map_bf16(&tmH, c.h, c.M, c.d, (int)(p.h_blk / 128u));
        if (r != VT_OK) return r;
        if (pair) {
            switch (KR) {
                case 4: r = launch_small<4, true>(tmW, tmH, p, grid, st); break;
                case 8: r = launch_small<8, true>(tmW, tmH, p, grid, st); break;
                case 10: r = launch_small<10, true>(tmW, tmH, p, grid, st); break;
                default: r = launch_small<16, true>(tmW, tmH, p, grid, st); break;
            }
        } else {
            switch (KR) {
                case 4: r = launch_small<4, false>(tmW, tmH, p, grid, st); break;
                case 8: r = launch_small<8, false>(tmW, tmH, p, grid, st); break;
                case 10: r = launch_small<10, false>(tmW, tmH, p, grid, st); break;
                case 16: r = launch_small<16, false>(tmW, tmH, p, grid, st); break;
                default: r = launch_small<0, false>(tmW, tmH, p, grid, st); break;
            }
        }
        if (r != VT_OK) return r;
    }
    return merge_after && !c.out.store_only ? launch_merge_rowmajor(c.out, grid, st) : VT_OK;
}

}  // namespace vt
