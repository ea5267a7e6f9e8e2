// Draft head, small-M path: a bandwidth-bound streaming GEMV on the CUDA cores.
//
//   x[m, i] = sum_j h[m, j] * W_trim[i, j]          (the d -> k linear head, 2*d*k FLOPs per row)
//
// One persistent CTA per SM owns a contiguous range of vocabulary rows.  A producer thread streams
// that range through a ring of shared-memory stages with 1-D bulk copies (whole rows are contiguous
// in W_trim).  Each stage holds a few complete rows and is consumed by ONE warp: its lanes stride
// over the row in 16-byte chunks, multiply with the bf16 hidden states kept in shared memory using
// packed fp32x2 FMAs, and fold the lane partials with a transposing shuffle reduction.  The lane
// that ends up with a logit keeps that (row slot, draft row)'s running (max, sum-exp) and top-k
// list, so no logit is written to memory and no warp waits for another.  When the range is done
// the CTA folds its warps' lists into one record per draft row; the warp that publishes a row last of all
// CTAs merges it (or the row-wise merge kernel does, for many draft rows).
//
// The FP32 pipe bounds this path: every weight costs M fused multiply-adds, which the CUDA cores
// keep up with only for M <= 4; larger M belongs to the tensor-core path.
#include "vt_common.cuh"
#include "vt_launch.h"

namespace vt {

constexpr int kGemvPrefill = 4;     // ring stages the producer starts before the dependency wait (measured: 4-8 gain, 16 lose)

constexpr int kGemvWarps = 16;                 // 1 producer + 15 consumers
constexpr int kGemvConsumers = kGemvWarps - 1;
constexpr int kGemvThreads = kGemvWarps * 32;
constexpr int kGemvR = 2;                      // vocabulary rows a warp accumulates together
constexpr int kGemvMaxM = 4;                   // draft rows per pass

struct GemvParams {
    const uint16_t* h;       // [M, d] bf16 (already offset to the first row of this pass)
    const uint16_t* W;       // [Vt, d] bf16
    HeadOut out;
    int m_begin, m_count;    // draft rows of this pass
    int early_weights;       // 1: the first stages may be requested before the dependency wait (W_trim declared constant)
    int d;
    int rows_per_stage;      // multiple of kGemvR
    int n_stages;            // multiple of n_cons, so a stage is always consumed by the same warp
    int n_cons;              // consumer warps that take tiles (<= kGemvConsumers)
    uint32_t stage_bytes;
    uint32_t h_off, list_off, fold_off, bar_off, total_smem;   // fold_off: candidate buffers of the per-row fold
};

// Folds NV per-lane values over the 32 lanes of a warp with NV-1 + log2(32/NV) shuffles.
// Afterwards every lane holds the warp total of value index (lane >> (5 - log2 NV)).
template <int N, int OFF>
__device__ __forceinline__ void fold_step(float* v, int lane) {
    if constexpr (N > 1) {
        constexpr int H = N / 2;
        const bool up = (lane & OFF) != 0;
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const float send = up ? v[i] : v[i + H];
            const float keep = up ? v[i + H] : v[i];
            v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, OFF);
        }
        fold_step<H, OFF / 2>(v, lane);
    } else if constexpr (OFF > 0) {
        v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], OFF);
        fold_step<1, OFF / 2>(v, lane);
    }
}

template <int N> struct Log2 { static constexpr int value = 1 + Log2<N / 2>::value; };
template <> struct Log2<1> { static constexpr int value = 0; };

__device__ __forceinline__ float2 bf16x2_to_f32x2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

// MP: draft rows per pass padded to a power of two.
template <int MP>
__global__ void __launch_bounds__(kGemvThreads, 1) head_gemv_kernel(const GemvParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int R = kGemvR;
    constexpr int NV = R * MP;                         // logits a warp finishes per fold
    constexpr int SHIFT = 5 - Log2<NV>::value;         // owner lane of value index i is i << SHIFT

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int Vt = p.out.Vt, d = p.d, k = p.out.k;
    const int row_begin = (int)((long long)cta * Vt / G);
    const int row_end = (int)((long long)(cta + 1) * Vt / G);
    const int nrows = row_end - row_begin;
    const int SR = p.rows_per_stage, S = p.n_stages;
    const int ntiles = (nrows + SR - 1) / SR;
    const int KS = ((k + 2) & ~1);

    unsigned char* hs = smem + p.h_off;                                                      // [MP][d] bf16
    unsigned long long* lists = reinterpret_cast<unsigned long long*>(smem + p.list_off);   // [consumer][NV][KS]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + p.bar_off);
    // bars: full[S], empty[S], one spare; then the abort flag
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * S;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * S + 1);

    auto fail = [&]() {
        *abort_flag = 1;
        atomicOr(&p.out.hdr->status, kStatusTimeout);
    };
    auto issue_tile = [&](int t) {     // tile t of this CTA's rows into stage t % S
        const int s = t % S;
        const int rows = min(SR, nrows - t * SR);
        const uint32_t bytes = (uint32_t)rows * (uint32_t)d * 2u;
        mbar_arrive_expect_tx(bar_full + 8u * s, bytes);
        bulk_g2s(smem_u32(smem) + (uint32_t)s * p.stage_bytes, p.W + (size_t)(row_begin + t * SR) * d, bytes,
                 bar_full + 8u * s);
    };
    // The producing thread sets the ring up and starts the stream before it joins the CTA's set-up barrier: the
    // first bytes take two microseconds to arrive and need nothing else of the set-up.  It waits for the previous
    // kernel in the stream first - except that, when the caller has declared W_trim a constant of the model, the
    // first few stages are requested even before that, while the previous kernel finishes.  h, the workspace and
    // the outputs are only touched after the wait.
    const int first_fill = min(min(S, ntiles), kGemvPrefill);     // a few stages only: the CTA waits for this thread at the barrier below
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
        const int early = p.early_weights ? min(first_fill, kGemvPrefill) : 0;
        for (int t = 0; t < early; ++t) issue_tile(t);
        grid_dependency_wait();
        for (int t = early; t < first_fill; ++t) issue_tile(t);
    }
    for (int i = tid; i < kGemvConsumers * NV * KS; i += blockDim.x) lists[i] = 0ull;
    __syncthreads();                   // the barriers are initialised and the ring is being filled
    grid_dependency_wait();
    if (tid == 0) grid_launch_dependents();
    {   // hidden states of this pass; pad rows (m >= m_count) repeat the last real row and are never read out
        const int nchunks = d >> 3;
        for (int i = tid; i < MP * nchunks; i += blockDim.x) {
            const int m = i / nchunks, c = i - m * nchunks;
            const int msrc = min(m, p.m_count - 1);
            reinterpret_cast<uint4*>(hs)[i] = __ldg(reinterpret_cast<const uint4*>(p.h + (size_t)msrc * d) + c);
        }
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int issued = first_fill;
            for (int t = first_fill; t < ntiles; ++t) {
                const int s = t % S, n = t / S;
                if (n > 0 && !mbar_wait(bar_empty + 8u * s, (uint32_t)(n - 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                issue_tile(t);
                issued = t + 1;
            }
            if (*abort_flag) {   // let copies in flight land before the CTA gives its shared memory back
                const unsigned long long deadline = global_timer_ns() + kWaitLimitNs;
                for (int t = max(0, issued - S); t < issued; ++t)
                    (void)mbar_wait_until(bar_full + 8u * (t % S), (uint32_t)(t / S) & 1u, deadline);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers: one warp per stage
        const int cw = warp - 1;
        const int nchunks = d >> 3;
        const int my_idx = lane >> SHIFT;                       // value index this lane ends up holding
        const bool owner = (lane & ((1 << SHIFT) - 1)) == 0;
        const int my_r = my_idx / MP, my_m = my_idx % MP;
        const bool live = owner && my_m < p.m_count;
        unsigned long long* my_list = lists + (size_t)(cw * NV + my_idx) * KS;
        float mx = -INFINITY, ssum = 0.0f, thr_x = -INFINITY;
        int filled = 0;
        // Tile t lives in stage t % S and belongs to warp t % n_cons.  S is a multiple of n_cons, so one warp sees
        // every phase of the stages it uses, in order (a parity wait may lag its barrier by one phase at most).
        for (int t = cw; t < ntiles && cw < p.n_cons; t += p.n_cons) {
            const int s = t % S;
            if (!mbar_wait(bar_full + 8u * s, (uint32_t)(t / S) & 1u)) { fail(); break; }
            if (*abort_flag) break;
            const int rows = min(SR, nrows - t * SR);
            const unsigned char* stage = smem + (size_t)s * p.stage_bytes;
            for (int g0 = 0; g0 < rows; g0 += R) {
                float2 acc[R][MP];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int m = 0; m < MP; ++m) acc[r][m] = make_float2(0.0f, 0.0f);
                // a row slot past the tile's last row re-reads the last row; its result is dropped below
                const unsigned char* wrow[R];
#pragma unroll
                for (int r = 0; r < R; ++r) wrow[r] = stage + (size_t)min(g0 + r, rows - 1) * d * 2;
                for (int c = lane; c < nchunks; c += 32) {
                    uint4 w[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) w[r] = *reinterpret_cast<const uint4*>(wrow[r] + (size_t)c * 16);
#pragma unroll
                    for (int m = 0; m < MP; ++m) {
                        const uint4 hv = *reinterpret_cast<const uint4*>(hs + ((size_t)m * d + (size_t)c * 8) * 2);
                        const float2 h0 = bf16x2_to_f32x2(hv.x), h1 = bf16x2_to_f32x2(hv.y);
                        const float2 h2 = bf16x2_to_f32x2(hv.z), h3 = bf16x2_to_f32x2(hv.w);
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            acc[r][m] = __ffma2_rn(bf16x2_to_f32x2(w[r].x), h0, acc[r][m]);
                            acc[r][m] = __ffma2_rn(bf16x2_to_f32x2(w[r].y), h1, acc[r][m]);
                            acc[r][m] = __ffma2_rn(bf16x2_to_f32x2(w[r].z), h2, acc[r][m]);
                            acc[r][m] = __ffma2_rn(bf16x2_to_f32x2(w[r].w), h3, acc[r][m]);
                        }
                    }
                }
                float v[NV];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int m = 0; m < MP; ++m) v[r * MP + m] = acc[r][m].x + acc[r][m].y;
                fold_step<NV, 16>(v, lane);
                if (live && g0 + my_r < rows) {
                    const float x = v[0];
                    const int row = row_begin + t * SR + g0 + my_r;
                    if (!p.out.store_only) {
                        lse_update(mx, ssum, x);
                        if (x > thr_x || filled < k) {     // rows reach this lane in ascending order: ties lose
                            const unsigned long long kth = list_insert(my_list, 1, k, make_key(x, row));
                            if (filled < k) ++filled;
                            if (filled == k) thr_x = key_logit(kth);
                        }
                    }
                    if (wants_logits(p.out)) store_logit(p.out, p.m_begin + my_m, row, x);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8u * s);
        }
        if (owner) my_list[k] = pack_ms(mx, ssum);
    }
    __syncthreads();

    // ---------------------------------------------------------------------- fold the CTA's lists: one warp per draft row
    if (warp < p.m_count && !p.out.store_only) {
        // lists of draft row `warp`: index (cw * NV + r * MP + warp), i.e. P1 = consumers * R lists, KS apart * MP
        const int m = warp;
        const int P1 = kGemvConsumers * R;
        const unsigned long long* rec0 = lists + (size_t)m * KS;
        const int stride = MP * KS;
        const float2 ms = warp_merge_ms(rec0, stride, P1, k);
        unsigned long long* cbuf = reinterpret_cast<unsigned long long*>(smem + p.fold_off) + (size_t)warp * kMergeCand;
        // Row-major record; with few draft rows then the row's ticket: the warp that draws the last one (over all
        // CTAs) merges the row at once, straight from global memory, with no CTA-wide step between the fold and
        // the outputs.  With many draft rows the row-wise merge kernel follows instead.
        const int row = p.m_begin + m;
        auto to_record = [&](int j, unsigned long long best) { VT_ROW_KEYS(p.out, row, j)[cta] = best; };
        if (P1 <= 32 && k <= kSelectLanesMaxK) warp_select_topk_lanes(rec0, stride, P1, k, cbuf, to_record);
        else warp_select_topk(rec0, stride, P1, k, cbuf, to_record);
        if (lane == 0) VT_ROW_MS(p.out, row)[cta] = pack_ms(ms.x, ms.y);
        if (p.out.fused_merge) {
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
    }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
template <int MP>
static vt_status launch_one(const GemvParams& p, int grid, cudaStream_t st) {
    auto kern = head_gemv_kernel<MP>;
    static std::atomic<unsigned long long> smem_configured{0};
    if (vt_status rc = ensure_max_dyn_smem(reinterpret_cast<const void*>(kern), (int)(kMaxDynSmem), &smem_configured); rc != VT_OK)
        return rc;
    cudaError_t e = launch_pdl(kern, grid, kGemvThreads, p.total_smem, st, p);
    count_launch();
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

bool gemv_supports(int d) { return d >= 8 && d % 8 == 0 && d <= 8192; }

vt_status launch_head_gemv(const HeadCall& c, cudaStream_t st, int* grid_out) {
    if (!gemv_supports(c.d)) return VT_ERR_UNSUPPORTED;
    int sms = 0;
    vt_status rs = device_sm_count(&sms);
    if (rs != VT_OK) return rs;
    const int grid = head_grid(sms, c.Vt);
    *grid_out = grid;
    const int KS = ((c.out.k + 2) & ~1);

    for (int m0 = 0; m0 < c.M; m0 += kGemvMaxM) {
        const int mc = std::min(kGemvMaxM, c.M - m0);
        const int MP = mc <= 1 ? 1 : mc <= 2 ? 2 : 4;

        GemvParams p{};
        p.h = reinterpret_cast<const uint16_t*>(c.h) + (size_t)m0 * c.d;
        p.W = reinterpret_cast<const uint16_t*>(c.W);
        p.out = c.out;
        p.m_begin = m0;
        p.m_count = mc;
        p.early_weights = c.static_weights;
        p.d = c.d;
        int sr = 16384 / (2 * c.d);
        sr = std::max(kGemvR, std::min(16, sr) / kGemvR * kGemvR);
        p.rows_per_stage = sr;
        p.stage_bytes = (uint32_t)sr * c.d * 2;
        const size_t h_bytes = ((size_t)MP * c.d * 2 + 127) & ~(size_t)127;
        const size_t list_bytes = ((size_t)kGemvConsumers * kGemvR * MP * KS * 8 + 127) & ~(size_t)127;
        const size_t bar_bytes = (size_t)(2 * 32 + 1) * 8 + 16;
        const size_t fold_bytes = (size_t)kGemvMaxM * kMergeCand * 8;
        const size_t fixed = h_bytes + list_bytes + fold_bytes + bar_bytes;
        if (fixed + 2 * (size_t)p.stage_bytes > (size_t)kMaxDynSmem) return VT_ERR_UNSUPPORTED;
        int S = (int)std::min<size_t>(32, ((size_t)kMaxDynSmem - fixed) / p.stage_bytes);
        p.n_cons = std::min(kGemvConsumers, S);
        S = S / p.n_cons * p.n_cons;
        size_t off = (size_t)S * p.stage_bytes;
        p.n_stages = S;
        p.h_off = (uint32_t)off;
        off += h_bytes;
        p.list_off = (uint32_t)off;
        off += list_bytes;
        p.fold_off = (uint32_t)off;
        off += fold_bytes;
        p.bar_off = (uint32_t)off;
        p.total_smem = (uint32_t)(off + bar_bytes);
        if (p.total_smem > (uint32_t)kMaxDynSmem) return VT_ERR_UNSUPPORTED;

        vt_status r = MP == 1 ? launch_one<1>(p, grid, st) : MP == 2 ? launch_one<2>(p, grid, st)
                                                                      : launch_one<4>(p, grid, st);
        if (r != VT_OK) return r;
    }
    return VT_OK;
}

}  // namespace vt
