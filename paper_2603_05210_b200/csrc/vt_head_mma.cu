// Draft head, tensor-core path: the head contraction as a tcgen05 GEMM with TMEM accumulators.
//
//   D[m, i] = sum_j h[m, j] * W_trim[i, j]       (the d -> k linear head, 2*d*k FLOPs per draft row)
//
// Operand roles: A = h (up to 128 draft rows = the 128 TMEM lanes), B = a tile of NT vocabulary rows
// of W_trim (K-major as stored), D = fp32 accumulator of 128 lanes x NT columns in tensor memory.
// With draft rows on the lanes, tcgen05.ld hands every epilogue thread one draft row and a run of
// consecutive vocabulary logits, so the running (max, sum-exp) and the top-k list are thread-private
// and need no shuffles.  One persistent CTA per SM owns a contiguous range of vocabulary rows:
//   warp 4   TMA producer: per 64-column k-step one box of h and one box of W into a shared-memory ring
//   warp 6   fetches h once into shared memory when it fits (else warp 4 streams it per k-step)
//   warp 5   MMA issuer: four K=16 tcgen05.mma per k-step, tcgen05.commit frees the ring slot;
//            two accumulator buffers in TMEM so the epilogue of tile t overlaps the MMAs of tile t+1
//   warps 0-3 epilogue: warp q reads TMEM lanes 32q..32q+31 (draft rows), never stores a logit
// The weight stream is the bound (arithmetic intensity = M FLOP/B), so the design spends its
// shared memory on bytes in flight rather than on operand reuse.
#include <cuda.h>

#include "vt_common.cuh"
#include "vt_launch.h"
#include "vt_tc.cuh"

namespace vt {

constexpr int kMmaThreads = 384;               // warps 0-3 epilogue, 4 TMA, 5 MMA; the rest only join the final merge
constexpr int kMaxStages = 32;
constexpr size_t kResidentHMax = 96 * 1024;   // h stays in shared memory when its A blocks fit in this
constexpr int kAccStride = 256;              // TMEM columns between the two accumulator buffers

struct MmaParams {
    HeadOut out;
    int m_begin, m_count;     // draft rows of this pass
    int d;
    int NT;                   // vocabulary rows per tile (multiple of 16, <= 256)
    int nk;                   // 64-column k-blocks per tile
    int kb_per_stage;         // k-blocks one ring stage holds (one barrier hand-over per stage)
    uint32_t blk_bytes;       // bytes of one k-block in a stage: (A slot +) B slot, multiple of 1024
    int n_stages;
    uint32_t stage_bytes;     // A slot + B slot, multiple of 1024
    uint32_t a_slot;          // bytes of the A slot: the pass's rows rounded up to whole 8-row groups
    uint32_t a_tx, b_tx;      // bytes each TMA box delivers
    int h_resident;           // 1: all of h sits in shared memory for the whole kernel (h_off), one A block per k-step
    uint32_t h_off;
    uint32_t idesc;
    int batch_cols;           // vocabulary columns per top-k selection batch (multiple of 32, <= 256)
    uint32_t tile_floats;     // floats of one warp's transpose buffer
    uint32_t list_off, bar_off, total_smem;   // offsets from the 1024-aligned base
};

// ------------------------------------------------------------------------------------------ kernel
constexpr int kMaxBatchCols = 256;            // vocabulary columns the top-k selection takes at a time

// Epilogue in two layouts.  tcgen05.ld gives lane = draft row, registers = 32 consecutive vocabulary
// logits: the running (max, sum-exp) is kept there, thread-private.  For the top-k the logits are turned
// through shared memory so that a whole warp works on one draft row at a time (warp_topk_update), which
// keeps all 32 lanes busy when there are only a few draft rows.
__global__ void __launch_bounds__(kMmaThreads, 1)
head_mma_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH, const MmaParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int Vt = p.out.Vt, k = p.out.k, NT = p.NT, S = p.n_stages, nk = p.nk;
    const int row_begin = (int)((long long)cta * Vt / G);
    const int row_end = (int)((long long)(cta + 1) * Vt / G);
    const int nrows = row_end - row_begin;
    const int ntiles = (nrows + NT - 1) / NT;

    unsigned long long* epi = reinterpret_cast<unsigned long long*>(smem + p.list_off);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + p.bar_off);
    const uint32_t bar_full = base + p.bar_off, bar_empty = bar_full + 8u * S;
    const uint32_t bar_accf = bar_empty + 8u * S, bar_acce = bar_accf + 16u, bar_drain = bar_acce + 16u;
    const uint32_t bar_merge = bar_drain + 8u, bar_h = bar_merge + 8u;
    const uint32_t bar_sel_ready = bar_h + 8u, bar_sel_done = bar_sel_ready + 8u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 9);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* last_flag = const_cast<int*>(abort_flag) + 1;

    const int n_epi_warps = (p.m_count + 31) / 32;
    if (warp == 4 && lane == 0) {      // descriptor fetches overlap the barrier set-up below
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
            mbar_init(bar_acce + 8u * b, n_epi_warps);
        }
        mbar_init(bar_drain, 1);
        mbar_init(bar_merge, 1);
        mbar_init(bar_h, 1);
        mbar_init(bar_sel_ready, n_epi_warps);
        mbar_init(bar_sel_done, n_epi_warps + (4 - n_epi_warps) + (kMmaThreads / 32 - 7));
        *abort_flag = 0;
        fence_mbar_init();
    }
    // epilogue scratch: lists [warps * 32][k] keys | candidate staging per warp | transpose buffer per warp
    for (int i = tid; i < n_epi_warps * 32 * k; i += blockDim.x) epi[i] = 0ull;
    const int n_cbuf = 4 + (kMmaThreads / 32 - 7);  // one candidate buffer per team member (readers and helpers)
    unsigned long long* cands = epi + (size_t)n_epi_warps * 32 * k;
    float* thr_s = reinterpret_cast<float*>(cands + (size_t)n_cbuf * (kMaxBatchCols + VT_MAX_K));   // [warps * 32]
    float2* ms_s = reinterpret_cast<float2*>(thr_s + n_epi_warps * 32);                               // [warps * 32]
    float* tiles = reinterpret_cast<float*>(ms_s + n_epi_warps * 32);
    for (int i = tid; i < n_epi_warps * 32; i += blockDim.x) {
        thr_s[i] = -INFINITY;
        ms_s[i] = make_float2(-INFINITY, 0.0f);
    }
    // The MMA always reads 128 A rows; rows past the pass's last row hold whatever follows the A block in
    // shared memory.  They only feed TMEM lanes that no thread reads, so they are left as they are.
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // everything above touched only shared memory, tensor memory and kernel parameters
    grid_dependency_wait();
    if (tid == 0) grid_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    auto fail = [&]() {
        *abort_flag = 1;
        atomicOr(&p.out.hdr->status, kStatusTimeout);
    };

    if (warp == 6) {
        // ------------------------------------------------------------------ resident h: fetched once
        // Every CTA needs all of h.  One fetch per CTA spreads the 148 CTAs' requests for its lines over
        // the L2 slices and keeps h out of the per-k-step path.
        if (lane == 0 && p.h_resident && ntiles > 0) {
            mbar_arrive_expect_tx(bar_h, p.a_tx * (uint32_t)nk);
            for (int ks = 0; ks < nk; ++ks)
                tma_load_2d(base + p.h_off + (uint32_t)ks * p.a_slot, &tmH, ks * kBoxK, p.m_begin, bar_h);
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0, issued = 0;
            uint32_t wrap = 0;          // times the ring has wrapped: stage s is free once its (wrap-1)-th use retired
            bool ok = true;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int row0 = row_begin + t * NT;
                const CUtensorMap* mapW = &tmW;
                const uint32_t b_tx = p.b_tx;
                const int kbs = p.kb_per_stage;
                const uint32_t blk = p.blk_bytes;
                for (int ks = 0; ks < nk; ks += kbs) {
                    if (wrap > 0 && !mbar_wait(bar_empty + 8u * s, (wrap - 1) & 1u)) { fail(); ok = false; break; }
                    if (*abort_flag) { ok = false; break; }
                    const int nb = min(kbs, nk - ks);
                    const uint32_t bar = bar_full + 8u * s;
                    mbar_arrive_expect_tx(bar, (uint32_t)nb * (p.h_resident ? b_tx : p.a_tx + b_tx));
                    for (int kb = 0; kb < nb; ++kb) {
                        const uint32_t dst = base + (uint32_t)s * p.stage_bytes + (uint32_t)kb * blk;
                        if (p.h_resident) {
                            tma_load_2d(dst, mapW, (ks + kb) * kBoxK, row0, bar);
                        } else {
                            tma_load_2d(dst, &tmH, (ks + kb) * kBoxK, p.m_begin, bar);
                            tma_load_2d(dst + p.a_slot, mapW, (ks + kb) * kBoxK, row0, bar);
                        }
                    }
                    ++issued;
                    if (++s == S) { s = 0; ++wrap; }
                }
            }
            if (*abort_flag) {   // let copies in flight land before the CTA gives its shared memory back
                for (int i = max(0, issued - S); i < issued; ++i)
                    (void)mbar_wait(bar_full + 8u * (i % S), (uint32_t)(i / S) & 1u);
                if (p.h_resident && ntiles > 0) (void)mbar_wait(bar_h, 0u);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            if (p.h_resident && ntiles > 0 && !mbar_wait(bar_h, 0u)) { fail(); ok = false; }
            const uint64_t desc0 = smem_desc_sw128(base);                      // descriptor of the ring's first byte
            const uint64_t h_desc0 = smem_desc_sw128(base + p.h_off);
            const uint32_t stage_units = p.stage_bytes >> 4, a_units = p.a_slot >> 4;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int buf = t & 1;
                if (t >= 2 && !mbar_wait(bar_acce + 8u * buf, (uint32_t)((t >> 1) - 1) & 1u)) { fail(); break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kAccStride);
                const uint32_t idesc = p.idesc;
                const int kbs = p.kb_per_stage;
                const uint32_t blk_units = p.blk_bytes >> 4;
                for (int ks = 0; ks < nk; ks += kbs) {
                    if (!mbar_wait(bar_full + 8u * s, phase)) { fail(); ok = false; break; }
                    if (*abort_flag) { ok = false; break; }
                    tc_fence_after();
                    const int nb = min(kbs, nk - ks);
                    for (int kb = 0; kb < nb; ++kb) {
                        const uint64_t blk_desc = desc0 + (uint64_t)((uint32_t)s * stage_units + (uint32_t)kb * blk_units);
                        const uint64_t a_desc = p.h_resident ? h_desc0 + (uint64_t)((uint32_t)(ks + kb) * a_units) : blk_desc;
                        const uint64_t b_desc = p.h_resident ? blk_desc : blk_desc + a_units;
                        // 16 bf16 = 32 bytes = 2 descriptor address units per MMA along K
                        tc_mma_bf16(d_tmem, a_desc, b_desc, idesc, (ks | kb) != 0);
                        tc_mma_bf16(d_tmem, a_desc + 2u, b_desc + 2u, idesc, 1u);
                        tc_mma_bf16(d_tmem, a_desc + 4u, b_desc + 4u, idesc, 1u);
                        tc_mma_bf16(d_tmem, a_desc + 6u, b_desc + 6u, idesc, 1u);
                    }
                    tc_commit(bar_empty + 8u * s);
                    if (++s == S) { s = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(bar_accf + 8u * buf);
            }
            if (*abort_flag) {   // every MMA issued so far must retire before TMEM is freed
                tc_commit(bar_drain);
                (void)mbar_wait(bar_drain, 0u);
            }
        }
    } else if (warp < n_epi_warps || warp >= 7 || warp < 4) {
        // ------------------------------------------------------------------ epilogue team
        // Readers (warps 0 .. n_epi_warps-1) own a quarter of the TMEM lanes each and turn their draft rows'
        // logits into the transpose buffers; then every team member - the readers and the otherwise idle
        // warps (the other warps below 4, and warps 7-11) - takes every team-th draft row of the batch.
        // Helpers replay the readers' batch sequence, which depends only on the tile geometry.
        const bool reader = warp < n_epi_warps;
        const int n_help = (4 - n_epi_warps) + (kMmaThreads / 32 - 7);
        const int team = n_epi_warps + n_help;
        const int member = reader ? warp : (warp < 4 ? warp : n_epi_warps + (4 - n_epi_warps) + (warp - 7));
        const int m_local = warp * 32 + lane;
        const bool live = reader && m_local < p.m_count;
        const int EB = p.batch_cols, EBP = EB + 1;                     // odd row pitch: conflict-free both ways
        float* my_tbuf = tiles + (size_t)warp * p.tile_floats;         // reader: tbuf[row * EBP + column in batch]
        unsigned long long* cbuf = cands + (size_t)member * (kMaxBatchCols + VT_MAX_K);
        uint32_t batch_no = 0;
        bool ok = true;

        for (int t = 0; t < ntiles && ok; ++t) {
            const int buf = t & 1;
            if (reader) {
                if (!mbar_wait(bar_accf + 8u * buf, (uint32_t)(t >> 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                tc_fence_after();
            }
            const int row0 = row_begin + t * NT;
            const int ncols = min(NT, row_end - row0);
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * kAccStride);
            for (int c0 = 0; c0 < ncols; c0 += 32) {
                const int nv = min(32, ncols - c0);
                const int cb = c0 % EB;                                // column of this chunk inside the batch
                const bool tile_end = c0 + 32 >= ncols;
                if (reader) {
                    uint32_t r[32];
                    tc_ld32(taddr + (uint32_t)c0, r);
                    tc_wait_ld();
                    // lane = draft row; columns past the CTA's rows are not its logits
                    if (live) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            my_tbuf[lane * EBP + cb + c] = c < nv ? __uint_as_float(r[c]) : -INFINITY;
                        if (p.out.logits) {
                            float* dst = p.out.logits + (size_t)(p.m_begin + m_local) * Vt + row0 + c0;
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c < nv) dst[c] = __uint_as_float(r[c]);
                        }
                    }
                }
                if (!(cb + 32 >= EB || tile_end)) continue;
                // a batch is complete (EB columns, or the tile's last chunk)
                if (reader) {
                    if (tile_end) {                  // TMEM is read out: the MMAs of the tile after next may start
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_acce + 8u * buf);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_sel_ready);
                }
                if (!mbar_wait(bar_sel_ready, batch_no & 1u)) { fail(); ok = false; break; }
                if (*abort_flag) { ok = false; break; }
                const int bvalid = min(min(cb + 32, EB), ncols - (c0 - cb));   // valid columns of the batch
                const int bcol0 = row0 + c0 - cb;                              // vocabulary row of its first column
                for (int m = member; m < p.m_count; m += team) {
                    const float* vals = tiles + (size_t)(m >> 5) * p.tile_floats + (size_t)(m & 31) * EBP;
                    const float t2 = warp_topk_update<kMaxBatchCols / 32>(vals, bvalid, bcol0, epi + (size_t)m * k, k, thr_s[m], cbuf,
                                                      ms_s + m, lane);
                    if (lane == 0) thr_s[m] = t2;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sel_done);
                // the transpose buffers are rewritten only after the whole team is done with them
                if (reader && !mbar_wait(bar_sel_done, batch_no & 1u)) { fail(); ok = false; break; }
                ++batch_no;
            }
        }
        if (reader) {
            // records: a row's list is contiguous in shared memory, so k lanes copy it out together.  Rows
            // another member kept are visible: its arrival on bar_sel_done released them.
            const int rows_here = min(32, p.m_count - warp * 32);
            for (int row = 0; row < rows_here; ++row) {
                const int m = warp * 32 + row;
                unsigned long long* rec = VT_REC(p.out, cta, p.m_begin + m);
                for (int j = lane; j < k; j += 32) rec[j] = epi[(size_t)m * k + j];
            }
            if (live) {
                const float2 ms = ms_s[m_local];
                VT_REC(p.out, cta, p.m_begin + m_local)[k] = pack_ms(ms.x, ms.y);
            }
        }
    }

    // ---------------------------------------------------------------------- publish + merge
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 5)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    if (!p.out.fused_merge) return;
    if (publish_and_check_last(p.out.hdr, last_flag)) {
        merge_rows(p.out, G, p.m_begin, p.m_count, smem, p.h_off, bar_merge);   // the ring is free now
        if (tid == 0) p.out.hdr->ticket = 0u;                                    // ready for the next call
    }
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static vt_status get_encode(EncodeTiledFn* out) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q);
        if (e != cudaSuccess) return cuda_fail(e);
        if (q != cudaDriverEntryPointSuccess || !ptr) return cuda_fail(cudaErrorSymbolNotFound);
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    *out = fn;
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

// Tile height for the most rows a CTA owns: a multiple of 16, at least 96 unless the CTA has fewer rows
// (every ring stage costs a barrier hand-over and every MMA 45 cycles however few rows it covers), with the
// least padding - rows a tile loads past the CTA's range are wasted HBM traffic - and, among equals, the
// height nearest 128 from below: with two or more tiles per CTA all epilogues but the last hide behind the
// stream, and the last one is short (measured: 2 x 112 beats 1 x 224; tiles of 48-64 rows stream too slowly).
static int choose_tile_rows(int rows) {
    if (rows <= 96) return ((rows + 15) / 16) * 16;
    int best = 256, best_cost = 1 << 30;
    for (int nt = 96; nt <= 256; nt += 16) {
        const int pad = (rows + nt - 1) / nt * nt - rows;
        const int cost = pad * 1024 + (nt <= 128 ? 128 - nt : nt);
        if (cost < best_cost) {
            best_cost = cost;
            best = nt;
        }
    }
    return best;
}

vt_status launch_head_mma(const HeadCall& c, cudaStream_t st, int* grid_out) {
    int sms = 0;
    vt_status r = device_sm_count(&sms);
    if (r != VT_OK) return r;
    const int grid = head_grid(sms, c.Vt, 16);
    *grid_out = grid;
    const int rows_per_cta = (c.Vt + grid - 1) / grid;
    const int NT = choose_tile_rows(rows_per_cta);

    static int configured_device = -1;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail(cudaGetLastError());
    if (configured_device != dev) {
        cudaError_t e = cudaFuncSetAttribute(head_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        configured_device = dev;
    }

    CUtensorMap tmW;
    r = make_tensor_map_bf16(&tmW, c.W, c.Vt, c.d, NT);
    if (r != VT_OK) return r;

    for (int m0 = 0; m0 < c.M; m0 += 128) {
        const int mc = std::min(128, c.M - m0);
        CUtensorMap tmH;
        r = make_tensor_map_bf16(&tmH, c.h, c.M, c.d, mc);
        if (r != VT_OK) return r;

        MmaParams p{};
        p.out = c.out;
        p.m_begin = m0;
        p.m_count = mc;
        p.d = c.d;
        p.NT = NT;
        p.nk = (c.d + kBoxK - 1) / kBoxK;
        p.a_tx = (uint32_t)mc * 128u;
        p.b_tx = (uint32_t)NT * 128u;
        p.a_slot = (((uint32_t)mc * 128u) + 1023u) & ~1023u;
        const uint32_t b_slot = ((uint32_t)NT * 128u + 1023u) & ~1023u;
        const size_t h_bytes = (size_t)p.nk * p.a_slot;
        p.h_resident = h_bytes <= kResidentHMax;
        p.blk_bytes = p.h_resident ? b_slot : p.a_slot + b_slot;
        // a stage of 24-32 KB amortises the per-stage barrier hand-over whatever the tile height
        p.kb_per_stage = std::max(1, std::min(4, (int)((28 * 1024 + p.blk_bytes / 2) / p.blk_bytes)));
        p.kb_per_stage = std::min(p.kb_per_stage, p.nk);
        p.stage_bytes = p.blk_bytes * p.kb_per_stage;
        // instruction descriptor: D fp32, A and B bf16, both K-major, N = NT, M = 128
        p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        // epilogue scratch: lists, candidate staging and a transpose buffer per epilogue warp; the fewer draft
        // rows a warp has, the more columns it can afford to select from at a time
        const int epi_warps = (mc + 31) / 32;
        const int rows_w = std::min(mc, 32);
        int batch = ((NT + 31) / 32) * 32;
        while (batch > 32 && (size_t)rows_w * (batch + 1) * 4 > 17 * 1024) batch -= 32;
        p.batch_cols = batch;
        p.tile_floats = (uint32_t)(rows_w * (batch + 1));
        const int n_cbuf = 4 + (kMmaThreads / 32 - 7);
        const size_t list_bytes = (((size_t)epi_warps * 32 * c.out.k * 8 + (size_t)n_cbuf * (kMaxBatchCols + VT_MAX_K) * 8 +
                                    (size_t)epi_warps * 32 * 12 + (size_t)epi_warps * p.tile_floats * 4) + 127) & ~(size_t)127;
        const size_t bar_bytes = (size_t)(2 * kMaxStages + 9) * 8 + 16;  // sized for the largest stage count
        const size_t merge_bytes = (size_t)grid * (ws_slots(c.out.k) * 8 + 16) + (size_t)(kMmaThreads / 32) * kMergeCand * 8;
        // Layout from the 1024-aligned base: ring | resident h | 16 KB the MMA may read past the last A block
        // (it always reads 128 A rows) | lists | barriers.  The pad is never written.
        const size_t fixed = 1024 + (p.h_resident ? h_bytes : 0) + 16384 + list_bytes + bar_bytes + 256;
        if (fixed + 2 * (size_t)p.stage_bytes > (size_t)kMaxDynSmem) return VT_ERR_UNSUPPORTED;
        int S = (int)std::min<size_t>(kMaxStages, ((size_t)kMaxDynSmem - fixed) / p.stage_bytes);
        size_t ring = (size_t)S * p.stage_bytes;
        if (ring < merge_bytes) ring = (merge_bytes + 1023) & ~(size_t)1023;
        if (ring + fixed > (size_t)kMaxDynSmem) return VT_ERR_UNSUPPORTED;
        p.n_stages = S;
        p.h_off = (uint32_t)ring;
        p.list_off = (uint32_t)(ring + (p.h_resident ? h_bytes : 0) + 16384);
        p.bar_off = (uint32_t)((p.list_off + list_bytes + 127) & ~(size_t)127);
        p.total_smem = (uint32_t)(p.bar_off + bar_bytes + 1024);

        cudaError_t e = launch_pdl(head_mma_kernel, grid, kMmaThreads, p.total_smem, st, tmW, tmH, p);
        count_launch();
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return VT_OK;
}

}  // namespace vt
