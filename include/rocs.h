/*
 * rocs.h -- C ABI of the B200 (sm_100a) In-Kernel Broadcast Optimization library.
 *
 * The library evaluates the candidate-side hot path of ROCS request-candidate layers:
 * request tensors stay at batch size R (B_r in the paper), candidate tensors at batch
 * size N (B_c), and each kernel resolves the request of a candidate inside the kernel
 * (Section 4, "In-Kernel Broadcast Optimization"); nothing is replicated per candidate.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.  The caller owns
 *     all buffers; the library allocates only what a plan holds.
 *   - Matrices are row-major, innermost dimension last.  `ld_*` are row strides in
 *     ELEMENTS.  Every base pointer must be 16-byte aligned and every row stride must
 *     be a multiple of 16 bytes (the memory-alignment rule of Section 4.2.4 made
 *     explicit; rocs_padded_ld gives the zero-padded stride).
 *   - Candidates of one request are stored consecutively: request r owns candidate
 *     rows cand_offsets[r] .. cand_offsets[r+1]-1.  This is the index map m of
 *     Section 4.1 in segment form.  Empty requests are legal.
 *   - Work is enqueued on `stream` (a cudaStream_t, NULL = default stream) and the call
 *     returns without synchronising, except where stated.  The tensor-core kernels are
 *     launched as programmatic dependents of the kernel in front of them on the stream: they
 *     may set up their own on-chip state while that kernel ends, and wait for its completion
 *     before they read or write global memory, so the ordering a stream guarantees is kept.
 *   - Errors are return codes.  Arguments are validated before anything is enqueued: every
 *     code except ROCS_ERR_CUDA means that the call launched nothing.
 *   - dtype names the storage type of all X / W / Q / K / V / output tensors of a call.
 *     ROCS_BF16: bf16 storage, fp32 accumulation (tensor cores where the shape allows),
 *     softmax in fp32, results rounded to bf16 (nearest even).  ROCS_F32: fp32 storage
 *     and plain fp32 FMA arithmetic.
 *   - Results are run-to-run bitwise deterministic, and a candidate's output bits do not
 *     depend on any other candidate's inputs (the GLM invariant, Eq. 1).
 */
#ifndef ROCS_H_
#define ROCS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ROCS_OK = 0,
  ROCS_ERR_INVALID_ARG = -1, /* null pointer, negative or inconsistent size            */
  ROCS_ERR_ALIGNMENT = -2,   /* base pointer or row stride not a multiple of 16 bytes  */
  ROCS_ERR_UNSUPPORTED = -3, /* shape outside what the kernels handle                  */
  ROCS_ERR_SEGMENTS = -4,    /* offsets not non-decreasing / wrong end points          */
  ROCS_ERR_WORKSPACE = -5,   /* workspace NULL, misaligned or too small                */
  ROCS_ERR_CUDA = -6,        /* a CUDA runtime or driver call failed                   */
  ROCS_ERR_TIMEOUT = -7,     /* a bounded device-side wait expired (see rocs_last_device_status) */
  ROCS_ERR_STATIC_LIMIT = -8 /* problem larger than the fixed scratch of rocs_ikbo_linear_static */
} rocs_status_t;

typedef enum { ROCS_BF16 = 0, ROCS_F32 = 1 } rocs_dtype_t;
typedef enum { ROCS_ACT_NONE = 0, ROCS_ACT_RELU = 1 } rocs_act_t;

/* Which kernels a ROCS_BF16 call may use.  AUTO picks the tcgen05 tensor-core kernels when
 * the shape qualifies and the general kernels otherwise; GENERAL forces the general
 * (CUDA-core, fp32 FMA) kernels, which accept every legal shape. */
typedef enum { ROCS_PATH_AUTO = 0, ROCS_PATH_GENERAL = 1 } rocs_path_t;

typedef struct rocs_plan rocs_plan_t; /* opaque; owned by the library */

const char* rocs_status_string(rocs_status_t status);

/* Smallest row stride (in elements) >= n whose byte size is a multiple of 16
 * (Section 4.2.4, memory alignment). */
int64_t rocs_padded_ld(int64_t n, rocs_dtype_t dtype);

/* Process-wide kernel-path selector (default ROCS_PATH_AUTO).  Not thread-safe against
 * concurrent calls of the compute entry points. */
rocs_status_t rocs_set_path(rocs_path_t path);

/*
 * Segment plan (Section 4.1: the request-candidate map m).  Built once per batch and
 * shared by every layer that uses the same cand_offsets.
 *   R, N               number of requests and of candidates (N < 2^31)
 *   cand_offsets       [R+1] device int32, non-decreasing, [0] = 0, [R] = N; must stay
 *                      valid and unchanged for the plan's lifetime
 *   cand_offsets_host  optional host copy of the same array.  When given, validation and
 *                      tile planning use it and the call does not synchronise; when NULL
 *                      the offsets are copied back from the device (the call synchronises
 *                      `stream`).
 * The plan owns device arrays of O(N + number of tiles) int32, allocated and freed in stream
 * order on `stream` (from a memory pool of the library's own, which keeps what a destroyed plan
 * frees for the next plan instead of returning it to the driver); use the plan on that stream, or order other streams
 * behind it yourself.  Tile lists for a given number of rows per candidate are created on
 * first use by the attention / interaction calls (one allocation + copy) and cached.
 * Errors: INVALID_ARG, SEGMENTS, CUDA.
 */
rocs_status_t rocs_plan_create(rocs_plan_t** out, int32_t R, int64_t N,
                               const int32_t* cand_offsets,
                               const int32_t* cand_offsets_host, void* stream);
rocs_status_t rocs_plan_destroy(rocs_plan_t* plan);

/*
 * GLM linear layer, candidate side, with the request half broadcast inside the kernel
 * (Eq. 4 for two groups; decomposition of Section 4.1; Eq. 14; fused epilogue of
 * Section 4.2.1):
 *     Z   = X^R W_CR^T + bias                 once per request, fp32, in `workspace`
 *     Y_i = act( Z[m_i] + X^C_i W_CC^T )      for every candidate i
 *   XR   [R, d_req], ld_xr       request features   (ignored when d_req == 0)
 *   XC   [N, d_cand], ld_xc      candidate features
 *   W_CR [d_out, d_req], ld_wcr  request block of the masked weight row [W_CR | W_CC];
 *   W_CC [d_out, d_cand], ld_wcc the two may alias one [d_out, d_req+d_cand] matrix
 *                                (W_CR = W, W_CC = W + d_req, both strides d_req+d_cand)
 *   bias [d_out] fp32 or NULL
 *   Y    [N, d_out], ld_y        output, storage type `dtype`
 *   workspace                    >= rocs_ikbo_linear_workspace(plan, d_out) bytes, 256-byte
 *                                aligned; contents are overwritten; unused when d_req == 0
 * d_req == 0 gives the plain one-group layer Y = act(X^C W_CC^T + bias).
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.
 */
size_t rocs_ikbo_linear_workspace(const rocs_plan_t* plan, int32_t d_out);
rocs_status_t rocs_ikbo_linear(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t d_req,
                               int32_t d_cand, int32_t d_out, const void* XR, int64_t ld_xr,
                               const void* XC, int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                               const void* W_CC, int64_t ld_wcc, const float* bias,
                               rocs_act_t act, void* Y, int64_t ld_y, void* workspace,
                               size_t workspace_bytes, void* stream);

/*
 * The same layer for callers that cannot allocate device memory while they score a batch --
 * a serving thread whose allocator is frozen after start-up, a plugin living inside another
 * component's memory budget, a path where an allocation's possible synchronisation is not
 * acceptable.  (The paper has no counterpart; this entry point exists for such hosts only.)
 * It needs no plan and no workspace: the request half Z and the candidate->request map live in
 * one fixed array inside the library image (5 MiB of device memory held by every GPU context
 * that loads the library, until the process exits).  The call performs no cudaMalloc, cudaFree
 * or other allocating routine.
 *   Limits: R * d_out <= rocs_ikbo_linear_static_max_z_elems()      (1 Mi fp32 values)
 *           N         <= rocs_ikbo_linear_static_max_candidates()   (256 Ki candidates)
 *           beyond either, the call returns ROCS_ERR_STATIC_LIMIT and launches nothing.
 *   cand_offsets [R+1] device int32 as for rocs_plan_create; its contents are not validated
 *   (they live on the device).  d_req, d_cand, d_out > 0.  Other arguments as above.
 *   The first call on a device looks up the array's device address (cudaGetSymbolAddress);
 *   make that first call outside any stream capture.  The CUDA runtime itself loads a kernel's
 *   code the first time that kernel is launched, which can allocate: which kernels run depends
 *   on the shape class (dtype, small or large N, width of d_out), so a host with a frozen
 *   allocator should send one warm-up call per shape class it will use at start-up (or run with
 *   CUDA_MODULE_LOADING=EAGER).  rocs_set_path does not apply to this entry point: it always
 *   takes the tensor-core kernels where the shape allows.
 *   All calls share the one array, and it keeps whatever the previous call left.  Each call
 *   overwrites every word it later reads, so stale contents are harmless, but two calls whose
 *   kernels overlap on the GPU (different streams, no ordering between them) race on it:
 *   serialise them.
 * Errors: INVALID_ARG, ALIGNMENT, STATIC_LIMIT, CUDA.
 */
size_t rocs_ikbo_linear_static_max_z_elems(void);
size_t rocs_ikbo_linear_static_max_candidates(void);
rocs_status_t rocs_ikbo_linear_static(rocs_dtype_t dtype, int32_t R, int64_t N,
                                      const int32_t* cand_offsets, int32_t d_req, int32_t d_cand,
                                      int32_t d_out, const void* XR, int64_t ld_xr, const void* XC,
                                      int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                                      const void* W_CC, int64_t ld_wcc, const float* bias,
                                      rocs_act_t act, void* Y, int64_t ld_y, void* stream);

/*
 * One-group linear layer Y = act(X W^T + bias) on M rows (Eq. 4 with a single group):
 * the plain layers that follow a split layer, and request-side products at batch size R.
 *   X [M, d_in], ld_x;  W [d_out, d_in], ld_w;  bias [d_out] fp32 or NULL;  Y [M, d_out], ld_y.
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, CUDA.
 */
rocs_status_t rocs_linear(rocs_dtype_t dtype, int64_t M, int32_t d_in, int32_t d_out,
                          const void* X, int64_t ld_x, const void* W, int64_t ld_w,
                          const float* bias, rocs_act_t act, void* Y, int64_t ld_y,
                          void* stream);

/*
 * Group-wise cross attention, candidate side (Eq. 13, second line; K/V sharing of
 * Section 4.3.1): every query row of candidate i attends over the sequence of its own
 * request m_i, whose keys and values exist once:
 *     O[i,t,h,:] = sum_j softmax_j( scale * <Q[i,t,h,:], K[s_r + j, h, :]> ) V[s_r + j, h, :]
 * with r = m_i, s_r = seq_offsets[r], j over the L_r = seq_offsets[r+1]-seq_offsets[r]
 * positions of that request.  No mask, no dropout, no output projection.
 *   Q [N, n_q, H, dh] dense;  K, V [T, H, dh] dense;  O [N, n_q, H, dh]
 *   T            number of sequence rows in K and V; must equal seq_offsets[R] (T < 2^31)
 *   seq_offsets  [R+1] device int32, non-decreasing, [0] = 0 (contents are not validated)
 *   scale <= 0 selects 1/sqrt(dh)
 *   dh * sizeof(element) must be a multiple of 16; dh <= 256
 * bf16 with dh in {32, 64, 128} and n_q <= 128 runs on the tensor cores; anything else on a
 * general kernel.  Values of one request never reach another request's rows, NaN and Inf
 * included (the invariant of Eq. 1): a NaN in K or V of request r shows in rows of r only.
 * A request with L_r = 0 yields zero rows.  `workspace` may be NULL when
 * rocs_dca_attention_workspace returns 0.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.
 */
size_t rocs_dca_attention_workspace(const rocs_plan_t* plan, int32_t n_q, int32_t H, int32_t dh);
rocs_status_t rocs_dca_attention(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_q,
                                 int32_t H, int32_t dh, float scale, const void* Q,
                                 const void* K, const void* V, int64_t T,
                                 const int32_t* seq_offsets, void* O, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * GLM factorization machine for two groups (Eq. 9-10) with the optional ROCSified
 * linear compression on the row axis (Eq. 5-6), n = n_r + n_c:
 *     YR[r] = [ X^R_r X^R_r^T , 0 ]                         [R, n_r, n]   once per request
 *     YC[i] = [ X^C_i X^R_{m_i}^T , X^C_i X^C_i^T ]         [N, n_c, n]
 *     OR[r] = W_RR YR[r]                                    [R, n_ro, n]
 *     OC[i] = W_CR YR[m_i] + W_CC YC[i]                     [N, n_co, n]
 * where W = [[W_RR, *], [W_CR, W_CC]] is [n_ro + n_co, n] dense row-major and its
 * upper-right block W[0:n_ro, n_r:n] is never read (the mask of Eq. 3).  The request
 * term W_CR YR[r] is formed once per request (fp32, in `workspace`) and added to each
 * candidate of r inside the candidate kernel.
 *   XR [R, n_r, d] dense;  XC [N, n_c, d] dense;  d * sizeof(element) multiple of 16
 *   W == NULL: no compression; OR_ and OC must be NULL, n_ro = n_co = 0
 *   YR, YC: raw interaction blocks, either may be NULL (not written)
 *   OR_, OC: compressed outputs, either may be NULL (not written)
 *   workspace >= rocs_glm_interaction_workspace(...) bytes, 256-byte aligned
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.
 */
size_t rocs_glm_interaction_workspace(const rocs_plan_t* plan, int32_t n_r, int32_t n_c,
                                      int32_t n_co);
rocs_status_t rocs_glm_interaction(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_r,
                                   int32_t n_c, int32_t d, const void* XR, const void* XC,
                                   const void* W, int32_t n_ro, int32_t n_co, void* YR,
                                   void* YC, void* OR_, void* OC, void* workspace,
                                   size_t workspace_bytes, void* stream);

/*
 * GLM factorization machine for two groups (Eq. 9-10) followed by a projection of the
 * interaction matrix's column axis to k columns (the compression an FM block applies to its
 * n x n output; the paper names the dimension k but prints no formula, so this entry point
 * takes the reading F = G P).  With n = n_r + n_c, P = [P_R; P_C] in R^{n x k}:
 *     FR[r] = X^R_r X^R_r^T P_R                                      [R, n_r, k]  once per request
 *     FC[i] = X^C_i X^R_{m_i}^T P_R + X^C_i X^C_i^T P_C              [N, n_c, k]
 * evaluated as FC[i] = X^C_i (T[m_i] + X^C_i^T P_C) with T[r] = X^R_r^T P_R formed once per
 * request (fp32, in `workspace`): no request tensor is replicated per candidate.
 *   XR [R, n_r, d] dense;  XC [N, n_c, d] dense;  P [n_r + n_c, k] dense row-major
 *   FR, FC: either may be NULL (not written);  d * sizeof(element) multiple of 16
 *   workspace >= rocs_glm_fm_projection_workspace(...) bytes, 256-byte aligned
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.
 */
size_t rocs_glm_fm_projection_workspace(const rocs_plan_t* plan, int32_t d, int32_t k);
rocs_status_t rocs_glm_fm_projection(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_r,
                                     int32_t n_c, int32_t d, int32_t k, const void* XR,
                                     const void* XC, const void* P, void* FR, void* FC,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Group-local normalisation (Eq. 7): y = Norm(x) on ONE group's tensor, every row over its own d
 * coordinates, so no statistic spans two groups (normalise the request rows and the candidate rows
 * with separate calls; statistics over concatenated groups would break the invariant of Eq. 1).
 *     ROCS_NORM_LAYER:  y = (x - mean) / sqrt(var + eps) * gamma + beta    (biased variance)
 *     ROCS_NORM_RMS:    y = x / sqrt(mean(x^2) + eps) * gamma              (beta is ignored)
 *   X [M, d] with row stride ld_x, Y [M, d] with row stride ld_y (elements; Y may alias X)
 *   gamma, beta [d] in the storage type, either may be NULL (1 and 0);  eps >= 0
 * Statistics are accumulated in fp32.  Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
typedef enum { ROCS_NORM_LAYER = 0, ROCS_NORM_RMS = 1 } rocs_norm_t;
rocs_status_t rocs_group_norm(rocs_dtype_t dtype, rocs_norm_t kind, int64_t M, int32_t d, const void* X,
                              int64_t ld_x, const void* gamma, const void* beta, float eps, void* Y,
                              int64_t ld_y, void* stream);

/*
 * Group-local normalisation folded into the layers around it (Eq. 7 together with the fused
 * epilogue of Section 4.2.1): for a row y and the layer that consumes norm(y),
 *     LayerNorm:  norm(y) W^T = sc (y W^T) + sh (W 1),   sc = 1 / sqrt(var(y) + eps), sh = -mean(y) sc
 *     RMSNorm:    norm(y) W^T = sc (y W^T),              sc = 1 / sqrt(mean(y^2) + eps)
 * so the normalised rows are never written: the layer that produces y leaves each row's sum and
 * sum of squares (rocs_ikbo_linear_stats), the layer that consumes it scales and shifts its own
 * accumulators (rocs_linear_normed).  A learned gain gamma and offset beta are folded by the caller:
 * pass W with its columns multiplied by gamma and bias + W beta.
 *
 * rocs_ikbo_linear_stats: rocs_ikbo_linear plus
 *   row_stats [N, 2] fp32   (sum, sum of squares) over the d_out outputs of each row (after the
 *                           activation; taken from the fp32 values before they are rounded)
 *   workspace               >= rocs_ikbo_linear_stats_workspace(plan, d_out) bytes, 256-byte aligned
 * rocs_weight_row_sums: wbar[n] = sum_k W[n, k] in fp32 (the W 1 of LayerNorm's shift).
 * rocs_linear_normed: Y = act(norm(X) W^T + bias) from X as stored, its row_stats [M, 2] and wbar
 *   (wbar may be NULL for ROCS_NORM_RMS).  The variance is taken as mean(x^2) - mean(x)^2 in fp32:
 *   rows whose mean is thousands of times their spread lose accuracy; rocs_group_norm has no such limit.
 *   bf16 rows on the wide-layer kernel only (M >= 2048, d_out >= 256 and a multiple of 8); other
 *   shapes return ROCS_ERR_UNSUPPORTED: normalise with rocs_group_norm, then call rocs_linear.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.
 */
size_t rocs_ikbo_linear_stats_workspace(const rocs_plan_t* plan, int32_t d_out);
rocs_status_t rocs_ikbo_linear_stats(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t d_req,
                                     int32_t d_cand, int32_t d_out, const void* XR, int64_t ld_xr,
                                     const void* XC, int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                                     const void* W_CC, int64_t ld_wcc, const float* bias,
                                     rocs_act_t act, void* Y, int64_t ld_y, float* row_stats,
                                     void* workspace, size_t workspace_bytes, void* stream);
rocs_status_t rocs_weight_row_sums(rocs_dtype_t dtype, int32_t d_out, int32_t d_in, const void* W,
                                   int64_t ld_w, float* wbar, void* stream);
rocs_status_t rocs_linear_normed(rocs_dtype_t dtype, rocs_norm_t kind, int64_t M, int32_t d_in,
                                 int32_t d_out, const void* X, int64_t ld_x, const float* row_stats,
                                 float eps, const void* W, int64_t ld_w, const float* wbar,
                                 const float* bias, rocs_act_t act, void* Y, int64_t ld_y,
                                 void* stream);

/*
 * Device-side status of the tensor-core kernels.  Their barrier waits are bounded; a wait
 * that expires records a code in a device word instead of spinning forever and the kernel
 * returns.  This call synchronises the device, reads the word, clears it and returns
 * ROCS_OK or ROCS_ERR_TIMEOUT; *detail_host (optional) receives the raw word.
 */
rocs_status_t rocs_last_device_status(uint32_t* detail_host);

#ifdef __cplusplus
}
#endif
#endif /* ROCS_H_ */
