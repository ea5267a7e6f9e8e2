// Draft head, small-M path: a bandwidth-bound streaming GEMV on the CUDA cores.
//
//   x[m, i] = sum_j h[m, j] * W_trim[i, j]          (the d -> k linear head, 2*d*k FLOPs per row)
//
// One persistent CTA per SM owns a contiguous range of vocabulary rows.  A producer thread
// streams that range through a ring of shared-memory stages with 1-D bulk copies (whole rows are
// contiguous in W_trim), consumer warps hold their column slice of h in registers, multiply with
// packed fp32x2 FMAs and fold the per-lane partial sums with a transposing shuffle reduction, and
// one epilogue warp finishes each logit, keeps a running (max, sum-exp) and a top-k list per draft
// row, and never writes a logit to memory.  The last CTA to publish its partials merges them.
#include "vt_common.cuh"
#include "vt_launch.h"

namespace vt {

struct GemvParams {
    const uint16_t* h;       // [M, d] bf16 (already offset to the first row of this pass)
    const uint16_t* W;       // [Vt, d] bf16
    HeadOut out;
    int m_begin;             // first draft row of this pass (index into out.*)
    int m_count;             // rows in this pass, <= MP
    int d;
    int rows_per_stage;
    int n_stages;
    int ncw;                 // consumer warps
    uint32_t stage_bytes;
    uint32_t red_off, list_off, bar_off, total_smem;
};

__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

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

// MP: draft rows per pass padded to a power of two; CPT: 16-byte column chunks per consumer thread;
// R: vocabulary rows accumulated together before a fold; MAXT: launch bound.
template <int MP, int CPT, int R, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) head_gemv_kernel(const GemvParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int NV = R * MP;
    static_assert(NV <= 32 && (NV & (NV - 1)) == 0, "fold width");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int Vt = p.out.Vt, d = p.d, k = p.out.k, M = p.out.M;
    const int row_begin = (int)((long long)cta * Vt / G);
    const int row_end = (int)((long long)(cta + 1) * Vt / G);
    const int nrows = row_end - row_begin;
    const int SR = p.rows_per_stage, S = p.n_stages, ncw = p.ncw;
    const int ntiles = (nrows + SR - 1) / SR;

    float* red = reinterpret_cast<float*>(smem + p.red_off);                       // [2][SR][ncw][MP]
    unsigned long long* lists = reinterpret_cast<unsigned long long*>(smem + p.list_off);   // [k][MP]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + p.bar_off);
    // bars: full[S], empty[S], red_full[2], red_empty[2]; then two ints: abort flag, last flag
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * S;
    const uint32_t bar_rfull = bar_empty + 8u * S, bar_rempty = bar_rfull + 16u;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * S + 4);
    int* last_flag = const_cast<int*>(abort_flag) + 1;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, ncw);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_rfull + 8u * b, ncw);
            mbar_init(bar_rempty + 8u * b, 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    for (int i = tid; i < k * MP; i += blockDim.x) lists[i] = 0ull;
    __syncthreads();

    auto fail = [&]() {
        *abort_flag = 1;
        atomicOr(&p.out.hdr->status, kStatusTimeout);
    };

    float mx = -INFINITY, ssum = 0.0f;     // epilogue state of lane m < m_count

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int issued = 0;
            for (int t = 0; t < ntiles; ++t) {
                const int s = t % S, n = t / S;
                if (n > 0 && !mbar_wait(bar_empty + 8u * s, (uint32_t)(n - 1) & 1u)) { fail(); break; }
                if (*abort_flag) break;
                const int rows = min(SR, nrows - t * SR);
                const uint32_t bytes = (uint32_t)rows * (uint32_t)d * 2u;
                mbar_arrive_expect_tx(bar_full + 8u * s, bytes);
                bulk_g2s(smem_u32(smem) + (uint32_t)s * p.stage_bytes,
                         p.W + (size_t)(row_begin + t * SR) * d, bytes, bar_full + 8u * s);
                issued = t + 1;
            }
            if (*abort_flag) {   // let copies in flight land before the CTA gives its shared memory back
                for (int t = max(0, issued - S); t < issued; ++t)
                    (void)mbar_wait(bar_full + 8u * (t % S), (uint32_t)(t / S) & 1u);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ epilogue warp
        constexpr int NPARTS = 32 / MP;
        const int m = lane % MP, part = lane / MP;
        const bool owner = (part == 0) && (m < p.m_count);
        unsigned long long thr = 0ull;
        for (int t = 0; t < ntiles; ++t) {
            const int buf = t & 1;
            if (!mbar_wait(bar_rfull + 8u * buf, (uint32_t)(t >> 1) & 1u)) { fail(); break; }
            if (*abort_flag) break;
            const int rows = min(SR, nrows - t * SR);
            for (int r = 0; r < rows; ++r) {
                const float* src = red + ((size_t)(buf * SR + r) * ncw) * MP + m;
                float x = 0.0f;
                for (int cw = part; cw < ncw; cw += NPARTS) x += src[cw * MP];
#pragma unroll
                for (int o = MP; o < 32; o <<= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
                if (owner) {
                    const int row = row_begin + t * SR + r;
                    lse_update(mx, ssum, x);
                    const unsigned long long key = make_key(x, row);
                    if (key > thr) thr = list_insert(lists + m, MP, k, key);
                    if (p.out.logits) p.out.logits[(size_t)(p.m_begin + m) * Vt + row] = x;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_rempty + 8u * buf);
        }
        __syncwarp();
        if (owner) {
            const size_t slot = (size_t)cta * M + p.m_begin + m;
            for (int j = 0; j < k; ++j) p.out.keys[slot * k + j] = lists[j * MP + m];
            p.out.ms[slot] = make_float2(mx, ssum);
        }
    } else if (warp - 2 < ncw) {
        // ------------------------------------------------------------------ consumers
        const int cw = warp - 2;
        const int nchunks = d >> 3;
        float2 hp[CPT][4][MP];
        int chunk[CPT];
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
            chunk[q] = cw * 32 + lane + q * ncw * 32;
            const bool valid = chunk[q] < nchunks;
#pragma unroll
            for (int m = 0; m < MP; ++m) {
                uint4 w = make_uint4(0u, 0u, 0u, 0u);
                if (valid && m < p.m_count)
                    w = __ldg(reinterpret_cast<const uint4*>(p.h + (size_t)m * d + (size_t)chunk[q] * 8));
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    hp[q][jj][m] = make_float2(__uint_as_float(ww[jj] << 16), __uint_as_float(ww[jj] & 0xFFFF0000u));
            }
            if (!valid) chunk[q] = -1;
        }
        constexpr int SHIFT = 5 - Log2<NV>::value;
        for (int t = 0; t < ntiles; ++t) {
            const int s = t % S, buf = t & 1;
            if (!mbar_wait(bar_full + 8u * s, (uint32_t)(t / S) & 1u)) { fail(); break; }
            if (t >= 2 && !mbar_wait(bar_rempty + 8u * buf, (uint32_t)((t >> 1) - 1) & 1u)) { fail(); break; }
            if (*abort_flag) break;
            const int rows = min(SR, nrows - t * SR);
            const unsigned char* stage = smem + (size_t)s * p.stage_bytes;
            for (int g0 = 0; g0 < rows; g0 += R) {
                float2 acc[R][MP];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int m = 0; m < MP; ++m) acc[r][m] = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (g0 + r < rows) {
#pragma unroll
                        for (int q = 0; q < CPT; ++q) {
                            if (chunk[q] >= 0) {
                                const uint4 w = *reinterpret_cast<const uint4*>(
                                    stage + ((size_t)(g0 + r) * d + (size_t)chunk[q] * 8) * 2);
                                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                                for (int jj = 0; jj < 4; ++jj) {
                                    const float2 wp = make_float2(__uint_as_float(ww[jj] << 16),
                                                                  __uint_as_float(ww[jj] & 0xFFFF0000u));
#pragma unroll
                                    for (int m = 0; m < MP; ++m) acc[r][m] = ffma2(wp, hp[q][jj][m], acc[r][m]);
                                }
                            }
                        }
                    }
                }
                float v[NV];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int m = 0; m < MP; ++m) v[r * MP + m] = acc[r][m].x + acc[r][m].y;
                fold_step<NV, 16>(v, lane);
                if ((lane & ((1 << SHIFT) - 1)) == 0) {
                    const int idx = lane >> SHIFT;
                    const int r = idx / MP, m = idx % MP;
                    if (g0 + r < rows) red[((size_t)(buf * SR + g0 + r) * ncw + cw) * MP + m] = v[0];
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_empty + 8u * s);
                mbar_arrive(bar_rfull + 8u * buf);
            }
        }
    }

    // ---------------------------------------------------------------------- publish + merge
    if (publish_and_check_last(p.out.hdr, last_flag))
        merge_rows(p.out, G, p.m_begin, p.m_count, smem, p.bar_off);   // ring, red and lists are free now
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
template <int MP, int CPT, int R, int MAXT>
static vt_status launch_one(const GemvParams& p, int grid, int threads, cudaStream_t st) {
    auto kern = head_gemv_kernel<MP, CPT, R, MAXT>;
    static int configured_device = -1;   // per instantiation
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail(cudaGetLastError());
    if (configured_device != dev) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        configured_device = dev;
    }
    kern<<<grid, threads, p.total_smem, st>>>(p);
    count_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_OK : cuda_fail(e);
}

bool gemv_supports(int d) { return d >= 8 && d % 8 == 0 && d <= 8192; }

vt_status launch_head_gemv(const HeadCall& c, cudaStream_t st) {
    if (!gemv_supports(c.d)) return VT_ERR_UNSUPPORTED;
    const int nchunks = c.d / 8;
    int sms = 0;
    vt_status rs = device_sm_count(&sms);
    if (rs != VT_OK) return rs;
    const int grid = std::max(1, std::min(std::min(sms, kMaxParts), c.Vt));

    for (int m0 = 0; m0 < c.M; m0 += 8) {
        const int mc = std::min(8, c.M - m0);
        const int MP = mc <= 1 ? 1 : mc <= 2 ? 2 : mc <= 4 ? 4 : 8;
        // consumer warps and chunks per thread: MP = 8 keeps its h slice in 64 registers, so one chunk only
        int cpt = 1, ncw = (nchunks + 31) / 32;
        if (ncw > 16) {
            if (MP == 8 || ncw > 20) { cpt = 2; ncw = (nchunks + 63) / 64; }
        }
        if (MP == 8 && cpt == 2) return VT_ERR_UNSUPPORTED;   // h slice would not fit the register file
        const int R = (MP == 8) ? 2 : 4;
        const int threads = (ncw + 2) * 32;

        GemvParams p{};
        p.h = reinterpret_cast<const uint16_t*>(c.h) + (size_t)m0 * c.d;
        p.W = reinterpret_cast<const uint16_t*>(c.W);
        p.out = c.out;
        p.m_begin = m0;
        p.m_count = mc;
        p.d = c.d;
        p.ncw = ncw;
        int sr = 32768 / (2 * c.d);
        sr = std::max(R, std::min(16, sr) / R * R);
        p.rows_per_stage = sr;
        p.stage_bytes = (uint32_t)sr * c.d * 2;
        const size_t red_bytes = (size_t)2 * sr * ncw * MP * 4;
        const size_t list_bytes = (size_t)c.out.k * MP * 8;
        const size_t bar_bytes = 0;   // sized below, needs n_stages
        (void)bar_bytes;
        const size_t merge_bytes = (size_t)grid * (c.out.k + 1) * 8;
        // stages: as many as fit next to the small buffers, at most 8
        int S = 8;
        size_t ring, total;
        for (;; --S) {
            ring = (size_t)S * p.stage_bytes;
            size_t off = (ring + 127) & ~(size_t)127;
            p.red_off = (uint32_t)off;
            off += (red_bytes + 127) & ~(size_t)127;
            p.list_off = (uint32_t)off;
            off += (list_bytes + 127) & ~(size_t)127;
            if (off < merge_bytes) off = (merge_bytes + 127) & ~(size_t)127;   // merge staging reuses [0, bar_off)
            p.bar_off = (uint32_t)off;
            total = off + (size_t)(2 * S + 4) * 8 + 16;
            if (total <= (size_t)kMaxDynSmem || S == 2) break;
        }
        if (total > (size_t)kMaxDynSmem) return VT_ERR_UNSUPPORTED;
        p.n_stages = S;
        p.total_smem = (uint32_t)total;

        vt_status r = VT_ERR_UNSUPPORTED;
#define VT_GEMV_CASE(MP_, CPT_, R_)                                                            \
        if (MP == MP_ && cpt == CPT_) {                                                        \
            r = (threads <= 576) ? launch_one<MP_, CPT_, R_, 576>(p, grid, threads, st)        \
                                 : launch_one<MP_, CPT_, R_, 704>(p, grid, threads, st);       \
        }
        VT_GEMV_CASE(1, 1, 4)
        VT_GEMV_CASE(2, 1, 4)
        VT_GEMV_CASE(4, 1, 4)
        VT_GEMV_CASE(1, 2, 4)
        VT_GEMV_CASE(2, 2, 4)
        VT_GEMV_CASE(4, 2, 4)
#undef VT_GEMV_CASE
        if (MP == 8 && cpt == 1) {
            if (threads > 576) return VT_ERR_UNSUPPORTED;
            r = launch_one<8, 1, 2, 576>(p, grid, threads, st);
        }
        if (r != VT_OK) return r;
    }
    return VT_OK;
}

}  // namespace vt
