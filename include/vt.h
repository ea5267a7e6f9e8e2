/*
 * vt.h - C boundary of the trimmed-vocabulary draft head for NVIDIA B200 (sm_100a).
 *
 * The library computes, on one GPU, the part of a speculative-decoding draft step that
 * vocabulary trimming makes cheaper: the draft model's language-modelling head restricted to
 * a kept set V_d of V_trim token rows (the paper's k = |V_d|, Section 2.1), whose cost is the
 * 2*d*k term of the paper's cost model (Section 2.3, Eq. 3).
 *
 * Conventions that hold for every entry point
 *  - "dev" pointers are device memory of the current CUDA device, "host" pointers are host
 *    memory.  The caller owns every buffer; the library allocates and frees nothing and keeps
 *    no pointer after a call returns.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Unless stated
 *    otherwise a call only enqueues work on that stream and returns without synchronising.
 *  - bf16 tensors are row-major arrays of 16-bit patterns; ids and indices are int32.
 *  - Errors are return codes.  Argument errors are detected on the host before anything is
 *    launched.  No entry point throws, aborts or traps the device.
 *  - A call must run on the device whose memory it is given; the library does not switch devices.
 */
#ifndef VT_H_
#define VT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum vt_status {
    VT_OK = 0,
    VT_ERR_NULL = 1,       /* a required pointer is NULL                                              */
    VT_ERR_SHAPE = 2,      /* d < 8, d % 8 != 0, M < 1, V_trim < 1, V_trim > V_full, k < 1, k > V_trim,
                              k > VT_MAX_K, N < 0, a size beyond what an entry point states it takes  */
    VT_ERR_ALIGN = 3,      /* a bf16 matrix pointer is not 16-byte aligned, an id pointer not 4-byte  */
    VT_ERR_RANGE = 4,      /* a keep id lies outside [0, V_full)                                      */
    VT_ERR_DUP = 5,        /* keep_ids names an id twice (V_d is a set, Section 2.1)                  */
    VT_ERR_EMPTY = 6,      /* vt_coverage with N == 0: Eq. 2 would be 0/0                             */
    VT_ERR_WORKSPACE = 7,  /* workspace NULL, misaligned (256 B) or smaller than the size function says */
    VT_ERR_TIMEOUT = 8,    /* a bounded device-side wait ran out; outputs of that call are invalid    */
    VT_ERR_CUDA = 9,       /* a CUDA runtime or driver call failed (see vt_last_cuda_error)           */
    VT_ERR_UNSUPPORTED = 10 /* the requested path cannot run this shape (only with a forced path)     */
} vt_status;

#define VT_MAX_K 64        /* largest top-k per draft row */

/* Which contraction kernel vt_draft_head_path / vt_debug_logits run. */
typedef enum vt_path {
    VT_PATH_AUTO = 0,      /* chosen from M and d                                                     */
    VT_PATH_GEMV = 1,      /* CUDA-core streaming GEMV; 4 draft rows per pass, d <= 8192              */
    VT_PATH_MMA = 2,       /* tcgen05 tensor-core GEMM, draft rows on the TMEM lanes; any M            */
    VT_PATH_MMA_SMALL = 3  /* tcgen05 tensor-core GEMM, vocabulary rows on the TMEM lanes; any M, in passes
                              of 128 draft rows; of 256 when k <= 16 and M > 96 (M > 64 where a CTA owns at
                              most 128 vocabulary rows): pairs of CTAs then share each MMA            */
} vt_path;

#define VT_PATH_MASK 0xFF  /* the vt_path part of an `options` argument */

/* Option bits for vt_draft_head_path, ORed onto the vt_path value. */
#define VT_HEAD_STATIC_WEIGHTS 0x100 /* the caller declares W_trim a constant of the model: nothing earlier in the
                                        stream writes it (see vt_draft_head).  The kernels may then request weights
                                        ahead of the stream-order dependency wait.                                 */
#define VT_HEAD_D2T_OFFSETS    0x200 /* d2t holds offsets instead of ids: target id = draft index + d2t[draft index],
                                        the form an EAGLE-3 style checkpoint stores (Section 1)                     */

/* Text for a status code (static storage). */
const char* vt_strerror(vt_status s);

/* The last CUDA error code (cudaError_t or CUresult as int) this thread's calls ran into; 0 if none. */
int vt_last_cuda_error(void);

/* ------------------------------------------------------------------------------------------
 * Head compaction (Section 2.1: the draft vocabulary V_d is the kept tokens; the head keeps
 * only their rows).
 *
 *   W_trim[i, :] = W_full[keep_ids[i], :]      for i in [0, V_trim),  a bit copy of bf16 rows
 *
 *   W_full   dev  [V_full, d] bf16 row-major, 16-byte aligned
 *   keep_ids dev  [V_trim] int32, each in [0, V_full), pairwise distinct.  This call does not check that
 *                 (vt_validate_keep_ids does, and synchronises to do so); a row whose id is out of range
 *                 is left unwritten
 *   W_trim   dev  [V_trim, d] bf16 row-major, caller-allocated, 16-byte aligned, must not
 *                 overlap W_full
 * Asynchronous.  VT_ERR_NULL / VT_ERR_SHAPE / VT_ERR_ALIGN / VT_ERR_CUDA.
 */
vt_status vt_compact_head(const void* W_full, int V_full, int d,
                          const int32_t* keep_ids, int V_trim,
                          void* W_trim, void* stream);

/* Bytes of scratch vt_validate_keep_ids and vt_coverage need for a vocabulary of V_full ids
 * (a membership bitmap plus counters).  Returns 0 if V_full < 1. */
size_t vt_coverage_workspace_bytes(int V_full);

/* Checks that keep_ids is a set inside [0, V_full) (Section 2.1).  Builds the membership
 * bitmap in `workspace` (dev, 256-byte aligned, vt_coverage_workspace_bytes(V_full)) and
 * SYNCHRONISES the stream to read two counters back.
 * Returns VT_ERR_RANGE if any id is out of range, else VT_ERR_DUP if any id repeats, else VT_OK. */
vt_status vt_validate_keep_ids(const int32_t* keep_ids, int V_trim, int V_full,
                               void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Draft head over the trimmed vocabulary (Section 2.3: the d -> k linear head, the only
 * vocabulary-dependent cost of an EAGLE-style draft; Section 1: the draft-to-target buffer).
 *
 * For each draft row m in [0, M):
 *   x[m, i]   = sum_j h[m, j] * W_trim[i, j]            fp32 accumulation of exact bf16 products
 *   lse[m]    = log sum_{i < V_trim} exp(x[m, i])       natural log, over the kept rows only
 *   the k largest x[m, :] in descending order, equal logits ordered by ascending draft index
 *   logprobs[m, j]   = x[m, i_j] - lse[m]
 *   target_ids[m, j] = d2t[i_j]                         d2t holds absolute target-vocabulary ids
 * The logits are never written to memory.
 *
 *   h          dev [M, d] bf16, 16-byte aligned          W_trim dev [V_trim, d] bf16, 16-byte aligned
 *   d2t        dev [V_trim] int32
 *   target_ids dev [M, k] int32 (out)                    logprobs dev [M, k] float (out)
 *   draft_ids  dev [M, k] int32 (out) or NULL            lse      dev [M] float (out) or NULL
 *   workspace  dev, 256-byte aligned, at least vt_workspace_bytes(M, k) bytes, zero-filled once
 *              by vt_workspace_init before its first use.  It carries per-CTA partial results,
 *              an arrival counter and a status word; calls that share a workspace must be
 *              ordered on one stream.
 * d % 8 == 0, d >= 8; 1 <= k <= min(V_trim, VT_MAX_K); any M >= 1.  Inputs must be finite.
 * Stream order: the kernels are launched with programmatic dependent launch, i.e. their CTAs may become
 *   resident while the stream's previous kernel is finishing (for this library's own head kernels: while
 *   their last rows are still being merged).  They set up shared and tensor memory and then wait for that
 *   kernel to complete before they touch h, W_trim, d2t, the workspace or the outputs, so every input may be
 *   produced by earlier work on the same stream, whatever kind of kernel produced it.
 *   vt_draft_head_path with VT_HEAD_STATIC_WEIGHTS relaxes this for W_trim only: the caller declares that
 *   nothing earlier in the stream writes W_trim (it was written once, e.g. by vt_compact_head, and the
 *   stream or device was synchronised afterwards - the usual state of model weights in a serving loop).
 *   A kernel may then request weight tiles before the wait, which hides the first memory round trip behind
 *   the previous call's tail (the CUDA-core path for one or two draft rows does; the tensor-core paths
 *   measured no gain and ignore the option).  h, d2t, the workspace and the outputs keep full stream-order
 *   semantics.
 * Asynchronous: no host synchronisation.  A device-side wait that ran out is reported by
 * vt_last_status on the same workspace; after VT_ERR_TIMEOUT run vt_workspace_init again before
 * the workspace is reused (arrival counters may be left mid-count).
 */
size_t    vt_workspace_bytes(int M, int k);
vt_status vt_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

vt_status vt_draft_head(const void* h, const void* W_trim, const int32_t* d2t,
                        int M, int d, int V_trim, int k,
                        int32_t* target_ids, float* logprobs,
                        int32_t* draft_ids, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Same call with options: `options` = a vt_path value (a forced contraction kernel returns
 * VT_ERR_UNSUPPORTED if it cannot take the shape; VT_PATH_AUTO is what vt_draft_head uses), optionally ORed
 * with VT_HEAD_STATIC_WEIGHTS and / or VT_HEAD_D2T_OFFSETS.  vt_draft_head is this call with options = 0.
 * Unknown option bits give VT_ERR_SHAPE. */
vt_status vt_draft_head_path(const void* h, const void* W_trim, const int32_t* d2t,
                             int M, int d, int V_trim, int k,
                             int32_t* target_ids, float* logprobs,
                             int32_t* draft_ids, float* lse,
                             void* workspace, size_t workspace_bytes, void* stream, int options);

/* End-to-end form of vt_draft_head for callers whose per-step data lives on the host:
 * h_host (host [M, d] bf16, ideally pinned) is copied to the device, the head runs, and
 * target_ids_host / logprobs_host (host [M, k]) are copied back, all on `stream`; the call
 * SYNCHRONISES the stream before returning so the host outputs are valid.  W_trim and d2t
 * stay device-resident (they are model state, not per-step input).  Pinned (page-locked, mapped) output
 * buffers are written by the kernel directly; pageable ones are filled by two copies after it.  Which kind a
 * buffer is is looked up once per buffer address and thread and remembered: keep an output buffer's kind
 * for as long as its address is passed.
 * workspace: dev, vt_host_workspace_bytes(M, d, k) bytes, initialised with vt_workspace_init. */
size_t    vt_host_workspace_bytes(int M, int d, int k);
vt_status vt_draft_head_host(const void* h_host, const void* W_trim, const int32_t* d2t,
                             int M, int d, int V_trim, int k,
                             int32_t* target_ids_host, float* logprobs_host,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Reads the status word of a draft-head workspace.  SYNCHRONISES the stream.  Returns VT_OK,
 * VT_ERR_TIMEOUT, or VT_ERR_CUDA, and clears the word. */
vt_status vt_last_status(void* workspace, void* stream);

/* ------------------------------------------------------------------------------------------
 * Feature fusion of an EAGLE-style draft (Section 2.3, component 1: the layer that projects the concatenated
 * hidden states of several target-model layers into the hidden dimension; Table 1, first row, 2 * 3d * d
 * FLOPs - part of the fixed cost F_fixed of Eq. 3, independent of the vocabulary):
 *
 *   fused[m, i] = bf16( sum_j h3[m, j] * W_fuse[i, j] )     fp32 accumulation of exact bf16 products, rounded
 *                                                           once, to nearest-even
 *
 *   h3      dev [M, d_in]  bf16, 16-byte aligned (d_in = 3d for three concatenated layers)
 *   W_fuse  dev [d_out, d_in] bf16, 16-byte aligned, row-major (one row per output feature)
 *   fused   dev [M, d_out] bf16 (out)
 *   workspace  a draft-head workspace of at least vt_workspace_bytes(M, 1) bytes (only its status word is used)
 * d_in % 8 == 0, d_in >= 8.  It runs the head's contraction kernels with an epilogue that only stores, so the
 * fixed part of a draft step can be timed on the same footing as the vocabulary-dependent part.
 * Asynchronous; stream order as for vt_draft_head. */
vt_status vt_fuse_features(const void* h3, const void* W_fuse, int M, int d_in, int d_out,
                           void* fused, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Cross-row candidate selection of a tree-style draft step (Section 1 describes the draft proposing candidate
 * tokens that the target verifies; the paper gives no formula for expanding several rows at once, so this is the
 * plain reading, stated here in full):
 *
 *   score[m, j] = parent_scores[m] + logprobs[m, j]        one fp32 addition
 *   the T largest scores over all M * k pairs, in descending order; equal scores by ascending m * k + j
 *   out_rows[t], out_slots[t] = the pair (m, j);  out_tokens[t] = target_ids[m, j];  out_scores[t] = its score
 *
 *   logprobs, target_ids  dev [M, k] (the outputs of vt_draft_head)      parent_scores  dev [M] float
 *   out_rows, out_slots, out_tokens  dev [T] int32 (out)                 out_scores     dev [T] float (out)
 * M * k <= 8192, 1 <= T <= M * k.  Asynchronous. */
vt_status vt_tree_select(const float* logprobs, const int32_t* target_ids, const float* parent_scores,
                         int M, int k, int T,
                         int32_t* out_rows, int32_t* out_slots, int32_t* out_tokens, float* out_scores,
                         void* stream);

/* ------------------------------------------------------------------------------------------
 * Coverage of a token stream by the kept set (Eq. 2 with f(v) = occurrences of v in the
 * stream; the "frequency coverage" of Table 4):
 *
 *   covered = #{ t in [0, N) : token_ids[t] in keep_ids },   fraction = covered / N
 *
 *   token_ids dev [N] int32; ids outside [0, V_full) count in N and are never covered
 *   keep_ids  dev [V_trim] int32 in [0, V_full) (out-of-range entries are ignored)
 *   covered_out, fraction_out: host (either may be NULL)
 *   workspace dev, 256-byte aligned, vt_coverage_workspace_bytes(V_full) bytes; contents are
 *             overwritten, no initialisation needed
 * SYNCHRONISES the stream once to return the count.  N == 0 gives VT_ERR_EMPTY.
 */
vt_status vt_coverage(const int32_t* token_ids, int64_t N,
                      const int32_t* keep_ids, int V_trim, int V_full,
                      uint64_t* covered_out, double* fraction_out,
                      void* workspace, size_t workspace_bytes, void* stream);

/* The same count (Eq. 2) in two steps, for callers that must not synchronise where the work is enqueued:
 * vt_coverage_enqueue puts the bitmap build and the count on the stream and returns at once (same arguments and
 * errors as vt_coverage, minus the outputs); vt_coverage_result SYNCHRONISES the stream and reads the count
 * that the last enqueue on this workspace left in it (N = that call's N, for the fraction). */
vt_status vt_coverage_enqueue(const int32_t* token_ids, int64_t N,
                              const int32_t* keep_ids, int V_trim, int V_full,
                              void* workspace, size_t workspace_bytes, void* stream);
vt_status vt_coverage_result(void* workspace, int64_t N,
                             uint64_t* covered_out, double* fraction_out, void* stream);

/* ------------------------------------------------------------------------------------------
 * Vocabulary-size selection (the paper's method, Sections 2.1-2.5), as an exhaustive scan over k:
 *
 *   f(v)  = occurrences of id v in token_ids (the stream is taken as already restricted to assistant
 *           tokens, Section 2.2); ids outside [0, V_full) are ignored
 *   order = ids by (f descending, id ascending)                     top-k most frequent, Section 2.1
 *   C(k)  = (sum of the k largest f) / (sum of all f)               Eq. 2
 *   R(k)  = 1 - (F_fixed + 2 d k) / (F_fixed + 2 d V_full)          Eq. 3
 *   U(k)  = alpha C(k) + (1 - alpha) R(k);  U~(k) = U(k) if C(k) >= c_min, else -1       Eq. 4, 5
 *   k*    = argmax of U~(k) over k_min <= k <= k_max, the smallest k among equal maxima   Eq. 1
 *
 * The paper searches k with 100 trials of a TPE optimiser; every k is evaluated here, which gives the exact
 * optimum of the same objective.  All arithmetic is IEEE double without fused multiply-add.
 *
 *   token_ids  dev [N] int32            ranked_ids dev [V_full] int32 (out): ranked_ids[:k*] is the draft
 *                                       vocabulary, i.e. keep_ids / d2t for the calls above
 *   cum_counts dev [V_full] uint64 (out) or NULL: cum_counts[k-1] = occurrences covered by the top k
 *   k_star     host (out);  C_star, R_star, U_star  host (out), each may be NULL
 *   unique_star host (out) or NULL: of the distinct ids that occur in the stream, the fraction that the top k*
 *              keeps (the "unique coverage" Table 4 reports beside Eq. 2's frequency-weighted coverage)
 *   workspace  dev, 256-byte aligned, vt_select_workspace_bytes(V_full); contents are overwritten
 * 1 <= k_min <= k_max <= V_full, 0 <= alpha <= 1, F_fixed >= 0, d >= 1, N < 2^32 (frequencies are counted in
 * 32 bits; a longer stream gives VT_ERR_SHAPE).  SYNCHRONISES the stream.
 * VT_ERR_EMPTY if N == 0 or no id falls inside [0, V_full). */
size_t    vt_select_workspace_bytes(int V_full);
vt_status vt_select_vocab(const int32_t* token_ids, int64_t N, int V_full, int d, double F_fixed,
                          double alpha, double c_min, int k_min, int k_max,
                          int32_t* ranked_ids, uint64_t* cum_counts,
                          int* k_star, double* C_star, double* R_star, double* U_star, double* unique_star,
                          void* workspace, size_t workspace_bytes, void* stream);

/* vt_coverage for callers that must not allocate device memory.  (The paper has no counterpart: this
 * entry point exists for integration, not for the method.)
 *
 * Who needs it: code that runs inside someone else's serving loop - an engine plugin that is handed a
 * stream and device pointers but does not own an allocator, or a process whose memory pool has been
 * reserved up front so that a late cudaMalloc would either fail or stall every stream on the device
 * while it runs.  vt_coverage asks such a caller for a scratch buffer it cannot provide; this variant
 * keeps the membership bitmap and the counters in a fixed array inside the library instead, and makes
 * no cudaMalloc / cudaFree call of its own.
 *
 * Same arguments, results and errors as vt_coverage, minus the workspace, with these differences:
 *  - V_full may be at most 262,144 (the built-in bitmap is 32 KiB; with its counters the array takes
 *    33,024 bytes on every device that loads the library, until the process ends).  A larger V_full
 *    returns VT_ERR_SHAPE and launches nothing.
 *  - The first call on a device looks up the array's device address and remembers it.
 *  - Every call ends by synchronising the stream to read the count back, so it cannot be part of a stream
 *    capture at all (neither can vt_coverage).
 *  - All calls on a device share the one array.  Each call clears it before use, so results do not
 *    depend on earlier calls, but two calls whose GPU work can overlap (different streams, different
 *    host threads) race on it: keep them ordered.
 * SYNCHRONISES the stream once to return the count, like vt_coverage. */
vt_status vt_coverage_static(const int32_t* token_ids, int64_t N,
                             const int32_t* keep_ids, int V_trim, int V_full,
                             uint64_t* covered_out, double* fraction_out, void* stream);

/* ------------------------------------------------------------------------------------------
 * Test and inspection entry points (same kernels as the calls above).
 */

/* The head contraction alone (Section 2.3), with the epilogue storing x[m, i] as fp32:
 * logits dev [M, V_trim] row-major (out).  Runs the same contraction code as vt_draft_head
 * on the chosen path; workspace as for vt_draft_head with k = 2 (vt_workspace_bytes(M, 2)). */
vt_status vt_debug_logits(const void* h, const void* W_trim, int M, int d, int V_trim,
                          float* logits, void* workspace, size_t workspace_bytes,
                          void* stream, int path);

/* The draft-to-target map alone (Section 1): target_ids[t] = d2t[draft_ids[t]] for t < n.
 * A draft id outside [0, V_trim) writes -1.  All pointers dev. */
vt_status vt_remap(const int32_t* draft_ids, const int32_t* d2t, int64_t n, int V_trim,
                   int32_t* target_ids, void* stream);

/* The two index buffers an EAGLE-3 style draft stores with its weights (the draft-to-target and the
 * target-to-draft map of Section 1), derived from keep_ids:
 *   d2t_offsets[i] = keep_ids[i] - i        (target id = draft index + offset), dev [V_trim] int32 or NULL
 *   t2d_mask[v]    = 1 if v is kept else 0,                                      dev [V_full] uint8 or NULL
 * At least one output must be given.  The head calls above take absolute ids (keep_ids itself as d2t) unless
 * VT_HEAD_D2T_OFFSETS is set, in which case they take the d2t_offsets this call writes.  Asynchronous. */
vt_status vt_vocab_maps(const int32_t* keep_ids, int V_trim, int V_full,
                        int32_t* d2t_offsets, uint8_t* t2d_mask, void* stream);

/* Number of kernels the last call of this thread launched (for launch accounting). */
int vt_last_launch_count(void);

/* Failure-path probe: one tiny kernel posts an mbarrier transaction that no copy will ever complete and
 * waits on it with the same bounded wait the head kernels use, limited to `limit_us` microseconds
 * (1 .. 1,000,000).  When the limit runs out it sets the time-out bit in the workspace's status word and
 * exits normally - nothing is in flight, nothing faults - so vt_last_status(workspace) then reports
 * VT_ERR_TIMEOUT, exactly as after a head call whose wait ran out.  workspace: a draft-head workspace.
 * Asynchronous. */
vt_status vt_test_timeout_probe(void* workspace, int limit_us, void* stream);

/* Stream-order probe: a kernel that releases its programmatic dependents at once, idles for `delay_us`
 * microseconds (0 .. 10,000) and only then copies n_bytes (a multiple of 16; dev pointers, 16-byte aligned)
 * from src to dst.  A head call enqueued right behind it must still see the copied bytes. Asynchronous. */
vt_status vt_test_late_copy(void* dst, const void* src, size_t n_bytes, int delay_us, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VT_H_ */
