// Internal declarations shared by the translation units of librocs.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <map>
#include <mutex>
#include <vector>

#include "../../include/rocs.h"

namespace rocs {

// One unit of work of the attention / interaction kernels: `count` consecutive candidates
// of request `req`, starting at candidate row `cand0`.  A tile never crosses a request.
struct Tile {
  int32_t req;
  int32_t cand0;
  int32_t count;
  int32_t pad;
};

struct TileList {
  Tile* dev = nullptr;
  int32_t num = 0;
};

// One unit of work of the tensor-core attention kernel: one head of up to two consecutive tiles
// (A and B) of the same request, which then share every K/V block that is loaded.
struct DcaItem {
  int32_t req;
  int32_t cand0;    // first candidate of tile A; tile B starts at cand0 + count_a
  int16_t count_a;  // candidates in tile A (>= 1)
  int16_t count_b;  // candidates in tile B (0 = no second tile)
  int32_t head;
};

struct DcaItemList {
  DcaItem* dev = nullptr;
  int32_t num = 0;
};

}  // namespace rocs

struct rocs_plan {
  int32_t R = 0;
  int64_t N = 0;
  const int32_t* cand_offsets = nullptr;  // device, borrowed
  int32_t* row2req = nullptr;             // device [N], m_i of Section 4.1
  std::vector<int32_t> offsets_host;      // [R+1]
  mutable std::mutex mu;
  mutable std::map<int32_t, rocs::TileList> tiles;  // key: candidates per tile
  mutable std::map<int64_t, rocs::DcaItemList> dca_items;  // key: (candidates per tile * 65536 + heads) * 2 + tiles per item - 1
  int device = 0;
  cudaStream_t stream = nullptr;  // stream the plan was created on; its memory is freed there
};

namespace rocs {

#define ROCS_CUDA_TRY(expr)                    \
  do {                                         \
    cudaError_t _e = (expr);                   \
    if (_e != cudaSuccess) return ROCS_ERR_CUDA; \
  } while (0)

inline size_t elem_size(rocs_dtype_t dt) { return dt == ROCS_BF16 ? 2 : 4; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Returns the cached tile list for `cands_per_tile`, building it on first use.
rocs_status_t plan_tiles(const rocs_plan* plan, int32_t cands_per_tile, cudaStream_t stream,
                         TileList* out);

// Work items for the attention kernel, ordered request, head, tile (or tile pair when tiles_per_item is 2);
// cached in the plan.
rocs_status_t plan_dca_items(const rocs_plan* plan, int32_t cands_per_tile, int32_t heads, int32_t tiles_per_item,
                             cudaStream_t stream, DcaItemList* out);

// ---- general (CUDA-core) kernels: simt_kernels.cu -------------------------------------
// Y[i, :] = act(add[row2req ? row2req[i] : -, :] + X[i, :] W^T + bias).  out_f32 selects an
// fp32 output regardless of the storage type (used for the request half Z).
rocs_status_t simt_linear(rocs_dtype_t dt, int64_t M, int32_t d_in, int32_t d_out, const void* X,
                          int64_t ld_x, const void* W, int64_t ld_w, const float* bias,
                          const float* add, int64_t ld_add, const int32_t* row2req, int act,
                          void* Y, int64_t ld_y, bool out_f32, cudaStream_t stream);
rocs_status_t simt_dca(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_q, int32_t H, int32_t dh,
                       float scale, const void* Q, const void* K, const void* V,
                       const int32_t* seq_offsets, void* O, cudaStream_t stream);
rocs_status_t simt_glm(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d,
                       const void* XR, const void* XC, const void* W, int32_t n_ro, int32_t n_co,
                       void* YR, void* YC, void* OR_, void* OC, float* zr_workspace,
                       cudaStream_t stream);

// ---- group-local normalisation (Eq. 7): group_norm.cu -------------------------------------
rocs_status_t group_norm(rocs_dtype_t dt, int kind, int64_t M, int32_t d, const void* X, int64_t ld_x,
                         const void* gamma, const void* beta, float eps, void* Y, int64_t ld_y, cudaStream_t stream);

// ---- projected factorization machine: fm_projection.cu ----------------------------------
// F = G P on the request-once form; tt_workspace [R, k, d] fp32 receives P_R^T X^R per request.
// allow_fast: use the bf16 streaming kernel for the candidate side where the shape allows it.
bool fm_projection_fast_supported(int32_t n_c, int32_t d, int32_t k);
rocs_status_t fm_projection(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, int32_t k,
                            const void* XR, const void* XC, const void* P, void* FR, void* FC, float* tt_workspace,
                            bool allow_fast, cudaStream_t stream);

// ---- tcgen05 tensor-core kernels (bf16): umma_*.cu -------------------------------------
bool umma_linear_supported(int64_t M, int32_t d_in, int32_t d_out, int64_t ld_x, int64_t ld_w,
                           int64_t ld_y, bool out_f32);
// add_rows: number of rows of `add` (the requests of the batch); 0 means one row per output row.
// add_from_previous_launch: `add` is written by the launch directly in front of this one on the
// stream (the request half) and nothing else this call reads is; the kernel may then overlap its
// set-up with that launch and waits for it only before it reads `add`.
rocs_status_t umma_linear(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x,
                          const void* W, int64_t ld_w, const float* bias, const float* add,
                          int64_t ld_add, const int32_t* row2req, int act, void* Y, int64_t ld_y,
                          bool out_f32, cudaStream_t stream, bool add_from_previous_launch = false,
                          float2* stat_partials = nullptr, int64_t add_rows = 0);
// Weight-stationary kernel on CTA pairs (cta_group::2) for d_in <= 256 and bf16 output: half a weight
// slice per SM, TMA-store epilogue (umma_linear picks it when it applies).
bool umma_linear_ws2_supported(int64_t M, int32_t d_in, int32_t d_out, bool out_f32);
rocs_status_t umma_linear_ws2(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x,
                              const void* W, int64_t ld_w, const float* bias, const float* add,
                              int64_t ld_add, const int32_t* row2req, int act, void* Y, int64_t ld_y,
                              cudaStream_t stream, bool add_from_previous_launch = false,
                              float2* stat_partials = nullptr, int64_t add_rows = 0);
// Number of (sum, sum of squares) partials per row the kernel above writes when asked to.
inline int32_t umma_linear_ws2_stat_partials(int32_t d_out) { return 2 * ((d_out + 255) / 256); }
// K-ring GEMM on CTA pairs for wide plain layers (no request term, bf16 output, many rows).
bool umma_linear_pair_supported(int64_t M, int32_t d_in, int32_t d_out, bool out_f32, bool has_add);
// norm (optional): the rows of X are to be normalised (Eq. 7) before the product; the kernel applies the
// row's scale and shift to its accumulators instead (see rocs_linear_normed).
struct RowNorm {
  const float2* row_stats = nullptr;  // [M] (sum, sum of squares) over the d_in columns of each row of X
  int kind = 0;                       // ROCS_NORM_LAYER / ROCS_NORM_RMS
  float eps = 0.f;
  const float* wbar = nullptr;        // [d_out] row sums of W (LayerNorm only)
};
rocs_status_t umma_linear_pair(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x,
                               const void* W, int64_t ld_w, const float* bias, int act, void* Y,
                               int64_t ld_y, cudaStream_t stream, const RowNorm* norm = nullptr);

// ---- per-row sums for a normalisation fused into the next layer: row_stats.cu ---------------------
rocs_status_t row_stats_from_partials(int64_t M, int32_t partials_per_row, const float2* partials, float2* row_stats,
                                      cudaStream_t stream);
rocs_status_t row_stats_direct(rocs_dtype_t dt, int64_t M, int32_t d, const void* Y, int64_t ld_y, float2* row_stats,
                               cudaStream_t stream);
rocs_status_t weight_row_sums(rocs_dtype_t dt, int32_t d_out, int32_t d_in, const void* W, int64_t ld_w, float* wbar,
                              cudaStream_t stream);
bool umma_dca_supported(int32_t n_q, int32_t H, int32_t dh);
rocs_status_t umma_dca(const rocs_plan* plan, int32_t n_q, int32_t H, int32_t dh, float scale,
                       const void* Q, const void* K, const void* V, const int32_t* seq_offsets,
                       int64_t T, void* O, cudaStream_t stream);
bool umma_glm_supported(int32_t n_r, int32_t n_c, int32_t d, int32_t n_ro, int32_t n_co);
rocs_status_t umma_glm(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, const void* XR,
                       const void* XC, const void* W, int32_t n_ro, int32_t n_co, void* YC,
                       void* OC, const float* zr_workspace, cudaStream_t stream);

// Request side of the interaction operator on warp-level tensor cores (bf16): YR, OR and the request
// term ZR of the compression, one block per request.
bool glm_request_mma_supported(int32_t n_r, int32_t d, int32_t n_ro, int32_t n_co);
rocs_status_t glm_request_mma(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, const void* XR,
                              const void* W, int32_t n_ro, int32_t n_co, void* YR, void* OR_, float* zr,
                              cudaStream_t stream);

// Device status word written by bounded waits of the tensor-core kernels.
uint32_t* device_status_word();

}  // namespace rocs
