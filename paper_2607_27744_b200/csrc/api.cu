// C ABI of librocs.so: argument validation, the segment plan, and dispatch to the kernels.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <map>
#include <mutex>
#include <new>

#include "rocs_internal.h"

namespace rocs {
namespace {

std::atomic<int> g_path{ROCS_PATH_AUTO};

// m_i of Section 4.1 from the segment offsets: one thread per candidate, binary search.
__global__ void fill_row2req_kernel(int32_t R, int64_t N, const int32_t* __restrict__ off,
                                    int32_t* __restrict__ row2req) {
  // the first layer's kernel may set itself up beside this one; it waits for this grid before it reads anything
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  int32_t lo = 0, hi = R;  // largest r with off[r] <= i
  while (hi - lo > 1) {
    const int32_t mid = lo + (hi - lo) / 2;
    if (off[mid] <= i) lo = mid; else hi = mid;
  }
  row2req[i] = lo;
}

bool row_stride_ok(int64_t ld, int64_t min_cols, rocs_dtype_t dt) {
  return ld >= min_cols && (ld * (int64_t)elem_size(dt)) % 16 == 0;
}

__device__ uint32_t g_device_status;

}  // namespace

// Stream-ordered allocations of the plan (request ids, work lists) come from a pool of the library's
// own that keeps freed memory instead of returning it to the driver at the next synchronisation: a
// serving loop builds and drops one plan per batch, and with the default pool's zero release
// threshold every batch would pay the driver's allocation path again.
static cudaError_t pool_alloc(void** ptr, size_t bytes, cudaStream_t stream) {
  static std::mutex mu;
  static std::map<int, cudaMemPool_t> pools;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  cudaMemPool_t pool = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = pools.find(dev);
    if (it == pools.end()) {
      cudaMemPoolProps props = {};
      props.allocType = cudaMemAllocationTypePinned;
      props.handleTypes = cudaMemHandleTypeNone;
      props.location.type = cudaMemLocationTypeDevice;
      props.location.id = dev;
      e = cudaMemPoolCreate(&pool, &props);
      if (e != cudaSuccess) return e;
      uint64_t keep = UINT64_MAX;
      cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
      pools[dev] = pool;
    } else {
      pool = it->second;
    }
  }
  return cudaMallocFromPoolAsync(ptr, bytes, pool, stream);
}

uint32_t* device_status_word() {
  uint32_t* p = nullptr;
  if (cudaGetSymbolAddress((void**)&p, g_device_status) != cudaSuccess) return nullptr;
  return p;
}

// Work lists are expanded on the device: the host only adds up the tile counts of the R requests
// (tile_base, R + 1 integers), every list entry then finds its request by binary search in that
// prefix array, so a batch with hundreds of thousands of entries costs one small copy and one launch.
__global__ void expand_tiles_kernel(int32_t R, int32_t total, int32_t cands_per_tile,
                                    const int32_t* __restrict__ off, const int32_t* __restrict__ tile_base,
                                    Tile* __restrict__ out) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int32_t lo = 0, hi = R;  // largest r with tile_base[r] <= i
  while (hi - lo > 1) {
    const int32_t mid = lo + (hi - lo) / 2;
    if (tile_base[mid] <= i) lo = mid; else hi = mid;
  }
  const int32_t c = off[lo] + (i - tile_base[lo]) * cands_per_tile;
  out[i] = Tile{lo, c, min(cands_per_tile, off[lo + 1] - c), 0};
}

// Attention items in the order request, head, tile (or tile pair).
__global__ void expand_dca_items_kernel(int32_t R, int32_t total, int32_t cands_per_tile, int32_t heads,
                                        int32_t tiles_per_item, const int32_t* __restrict__ off,
                                        const int32_t* __restrict__ item_base, DcaItem* __restrict__ out) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int32_t lo = 0, hi = R;  // largest r with item_base[r] * heads <= i
  while (hi - lo > 1) {
    const int32_t mid = lo + (hi - lo) / 2;
    if ((int64_t)item_base[mid] * heads <= i) lo = mid; else hi = mid;
  }
  const int32_t per_head = item_base[lo + 1] - item_base[lo];
  const int32_t local = i - item_base[lo] * heads;
  const int32_t h = local / per_head, t = local % per_head;
  const int32_t c = off[lo] + t * tiles_per_item * cands_per_tile, c_end = off[lo + 1];
  const int32_t a = min(cands_per_tile, c_end - c);
  const int32_t b = tiles_per_item == 2 ? min(cands_per_tile, c_end - c - a) : 0;
  out[i] = DcaItem{lo, c, (int16_t)a, (int16_t)b, h};
}

// Prefix sums of ceil(n_r / per_entry) over the requests, copied to the device.  Returns the total
// through *total; *base_dev is a stream-ordered allocation the caller frees after its kernel.
static rocs_status_t upload_entry_base(const rocs_plan* plan, int32_t per_entry, cudaStream_t stream,
                                       int32_t** base_dev, int64_t* total) {
  std::vector<int32_t> base((size_t)plan->R + 1);
  int64_t acc = 0;
  for (int32_t r = 0; r < plan->R; ++r) {
    base[r] = (int32_t)acc;
    const int64_t n = (int64_t)plan->offsets_host[r + 1] - plan->offsets_host[r];
    acc += (n + per_entry - 1) / per_entry;
    if (acc > 0x7fffffffLL) return ROCS_ERR_UNSUPPORTED;
  }
  base[plan->R] = (int32_t)acc;
  *total = acc;
  ROCS_CUDA_TRY(pool_alloc((void**)base_dev, sizeof(int32_t) * base.size(), stream));
  // Pageable source: the copy is staged before the call returns, so `base` may go away.
  if (cudaMemcpyAsync(*base_dev, base.data(), sizeof(int32_t) * base.size(), cudaMemcpyHostToDevice, stream) !=
      cudaSuccess) {
    cudaFreeAsync(*base_dev, stream);
    return ROCS_ERR_CUDA;
  }
  return ROCS_OK;
}

rocs_status_t plan_tiles(const rocs_plan* plan, int32_t cands_per_tile, cudaStream_t stream,
                         TileList* out) {
  if (cands_per_tile < 1) return ROCS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(plan->mu);
  auto it = plan->tiles.find(cands_per_tile);
  if (it != plan->tiles.end()) {
    *out = it->second;
    return ROCS_OK;
  }
  TileList tl;
  if (plan->N > 0) {
    int32_t* base_dev = nullptr;
    int64_t total = 0;
    rocs_status_t st = upload_entry_base(plan, cands_per_tile, stream, &base_dev, &total);
    if (st != ROCS_OK) return st;
    tl.num = (int32_t)total;
    cudaError_t e = pool_alloc((void**)&tl.dev, sizeof(Tile) * (size_t)total, stream);
    if (e == cudaSuccess) {
      expand_tiles_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(plan->R, tl.num, cands_per_tile,
                                                                              plan->cand_offsets, base_dev, tl.dev);
      e = cudaGetLastError();
      if (e != cudaSuccess) cudaFreeAsync(tl.dev, stream);
    }
    cudaFreeAsync(base_dev, stream);
    if (e != cudaSuccess) return ROCS_ERR_CUDA;
  }
  plan->tiles[cands_per_tile] = tl;
  *out = tl;
  return ROCS_OK;
}

rocs_status_t plan_dca_items(const rocs_plan* plan, int32_t cands_per_tile, int32_t heads, int32_t tiles_per_item,
                             cudaStream_t stream, DcaItemList* out) {
  if (cands_per_tile < 1 || cands_per_tile > 32767 || heads < 1 || heads > 65535 || tiles_per_item < 1 ||
      tiles_per_item > 2)
    return ROCS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(plan->mu);
  const int64_t key = ((int64_t)cands_per_tile * 65536 + heads) * 2 + (tiles_per_item - 1);
  auto it = plan->dca_items.find(key);
  if (it != plan->dca_items.end()) {
    *out = it->second;
    return ROCS_OK;
  }
  DcaItemList il;
  if (plan->N > 0) {
    int32_t* base_dev = nullptr;
    int64_t per_head = 0;
    rocs_status_t st = upload_entry_base(plan, cands_per_tile * tiles_per_item, stream, &base_dev, &per_head);
    if (st != ROCS_OK) return st;
    const int64_t total = per_head * heads;
    if (total > 0x7fffffffLL) {
      cudaFreeAsync(base_dev, stream);
      return ROCS_ERR_UNSUPPORTED;
    }
    il.num = (int32_t)total;
    cudaError_t e = pool_alloc((void**)&il.dev, sizeof(DcaItem) * (size_t)total, stream);
    if (e == cudaSuccess) {
      expand_dca_items_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
          plan->R, il.num, cands_per_tile, heads, tiles_per_item, plan->cand_offsets, base_dev, il.dev);
      e = cudaGetLastError();
      if (e != cudaSuccess) cudaFreeAsync(il.dev, stream);
    }
    cudaFreeAsync(base_dev, stream);
    if (e != cudaSuccess) return ROCS_ERR_CUDA;
  }
  plan->dca_items[key] = il;
  *out = il;
  return ROCS_OK;
}

}  // namespace rocs

using namespace rocs;

extern "C" {

const char* rocs_status_string(rocs_status_t s) {
  switch (s) {
    case ROCS_OK: return "ok";
    case ROCS_ERR_INVALID_ARG: return "invalid argument";
    case ROCS_ERR_ALIGNMENT: return "pointer or row stride not 16-byte aligned";
    case ROCS_ERR_UNSUPPORTED: return "unsupported shape";
    case ROCS_ERR_SEGMENTS: return "malformed segment offsets";
    case ROCS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case ROCS_ERR_CUDA: return "CUDA call failed";
    case ROCS_ERR_TIMEOUT: return "bounded device-side wait expired";
    case ROCS_ERR_STATIC_LIMIT: return "problem larger than the fixed scratch array of the no-allocation entry point";
  }
  return "unknown status";
}

int64_t rocs_padded_ld(int64_t n, rocs_dtype_t dtype) {
  const int64_t per16 = 16 / (int64_t)elem_size(dtype);
  return n <= 0 ? 0 : (n + per16 - 1) / per16 * per16;
}

rocs_status_t rocs_set_path(rocs_path_t path) {
  if (path != ROCS_PATH_AUTO && path != ROCS_PATH_GENERAL) return ROCS_ERR_INVALID_ARG;
  g_path.store(path);
  return ROCS_OK;
}

rocs_status_t rocs_plan_create(rocs_plan_t** out, int32_t R, int64_t N, const int32_t* cand_offsets,
                               const int32_t* cand_offsets_host, void* stream_) {
  if (!out) return ROCS_ERR_INVALID_ARG;
  *out = nullptr;
  if (R < 0 || N < 0 || N > 0x7fffffffLL || !cand_offsets) return ROCS_ERR_INVALID_ARG;
  if (R == 0 && N != 0) return ROCS_ERR_SEGMENTS;
  cudaStream_t stream = (cudaStream_t)stream_;
  rocs_plan* p = new (std::nothrow) rocs_plan();
  if (!p) return ROCS_ERR_INVALID_ARG;
  p->R = R;
  p->N = N;
  p->cand_offsets = cand_offsets;
  p->offsets_host.resize((size_t)R + 1);
  if (cand_offsets_host) {
    std::copy(cand_offsets_host, cand_offsets_host + R + 1, p->offsets_host.begin());
  } else {
    if (cudaMemcpyAsync(p->offsets_host.data(), cand_offsets, sizeof(int32_t) * ((size_t)R + 1),
                        cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
      delete p;
      return ROCS_ERR_CUDA;
    }
  }
  const auto& off = p->offsets_host;
  bool ok = off[0] == 0 && off[R] == N;
  for (int32_t r = 0; ok && r < R; ++r) ok = off[r + 1] >= off[r];
  if (!ok) {
    delete p;
    return ROCS_ERR_SEGMENTS;
  }
  if (cudaGetDevice(&p->device) != cudaSuccess) {
    delete p;
    return ROCS_ERR_CUDA;
  }
  {
    // Keep freed plan memory in the device's default pool instead of returning it to the driver
    // at every synchronisation (a per-process setting of the CUDA context, not of the GPU).
    static std::once_flag once[64];
    if (p->device >= 0 && p->device < 64)
      std::call_once(once[p->device], [&] {
        cudaMemPool_t pool;
        if (cudaDeviceGetDefaultMemPool(&pool, p->device) == cudaSuccess) {
          uint64_t keep = 1ull << 30;
          cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        }
      });
  }
  if (N > 0) {
    // Stream-ordered allocation: after the first batch the pool hands the block back without a
    // device synchronisation, so building a plan per batch stays off the critical path.
    if (pool_alloc((void**)&p->row2req, sizeof(int32_t) * (size_t)N, stream) != cudaSuccess) {
      delete p;
      return ROCS_ERR_CUDA;
    }
    fill_row2req_kernel<<<(unsigned)((N + 255) / 256), 256, 0, stream>>>(R, N, cand_offsets, p->row2req);
    if (cudaGetLastError() != cudaSuccess) {
      cudaFreeAsync(p->row2req, stream);
      delete p;
      return ROCS_ERR_CUDA;
    }
  }
  p->stream = stream;
  *out = p;
  return ROCS_OK;
}

rocs_status_t rocs_plan_destroy(rocs_plan_t* plan) {
  if (!plan) return ROCS_OK;
  rocs_status_t st = ROCS_OK;
  // Freed in stream order behind whatever the caller enqueued on the plan's stream.
  if (plan->row2req && cudaFreeAsync(plan->row2req, plan->stream) != cudaSuccess) st = ROCS_ERR_CUDA;
  for (auto& kv : plan->tiles)
    if (kv.second.dev && cudaFreeAsync(kv.second.dev, plan->stream) != cudaSuccess) st = ROCS_ERR_CUDA;
  for (auto& kv : plan->dca_items)
    if (kv.second.dev && cudaFreeAsync(kv.second.dev, plan->stream) != cudaSuccess) st = ROCS_ERR_CUDA;
  delete plan;
  return st;
}

size_t rocs_ikbo_linear_workspace(const rocs_plan_t* plan, int32_t d_out) {
  if (!plan || d_out <= 0) return 0;
  return round_up((size_t)plan->R * (size_t)d_out * sizeof(float), 256);
}

static rocs_status_t linear_dispatch(rocs_dtype_t dt, int64_t M, int32_t d_in, int32_t d_out,
                                     const void* X, int64_t ld_x, const void* W, int64_t ld_w,
                                     const float* bias, const float* add, int64_t ld_add,
                                     const int32_t* row2req, int act, void* Y, int64_t ld_y,
                                     bool out_f32, cudaStream_t stream,
                                     bool add_from_previous_launch = false, float2* stat_partials = nullptr,
                                     int64_t add_rows = 0) {
  if (dt == ROCS_BF16 && g_path.load() == ROCS_PATH_AUTO &&
      umma_linear_supported(M, d_in, d_out, ld_x, ld_w, ld_y, out_f32))
    return umma_linear(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y,
                       out_f32, stream, add_from_previous_launch, stat_partials, add_rows);
  return simt_linear(dt, M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y,
                     out_f32, stream);
}

// row_stats (optional): per-row (sum, sum of squares) of the output, for a normalisation folded into
// the next layer; its partials follow Z in the workspace.
static rocs_status_t ikbo_linear_impl(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t d_req,
                                      int32_t d_cand, int32_t d_out, const void* XR, int64_t ld_xr,
                                      const void* XC, int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                                      const void* W_CC, int64_t ld_wcc, const float* bias, rocs_act_t act,
                                      void* Y, int64_t ld_y, float* row_stats, void* workspace,
                                      size_t workspace_bytes, void* stream_) {
  if (!plan || (dtype != ROCS_BF16 && dtype != ROCS_F32)) return ROCS_ERR_INVALID_ARG;
  if (d_req < 0 || d_cand < 0 || d_out <= 0 || d_req + d_cand <= 0) return ROCS_ERR_INVALID_ARG;
  if (act != ROCS_ACT_NONE && act != ROCS_ACT_RELU) return ROCS_ERR_INVALID_ARG;
  if ((plan->N > 0 && (!Y || (d_cand > 0 && !XC))) || (d_cand > 0 && !W_CC) ||
      (d_req > 0 && (!W_CR || (plan->R > 0 && !XR))))
    return ROCS_ERR_INVALID_ARG;
  if (!aligned16(Y) || !aligned16(bias) || !row_stride_ok(ld_y, d_out, dtype)) return ROCS_ERR_ALIGNMENT;
  if (d_cand > 0 && (!aligned16(XC) || !aligned16(W_CC) || !row_stride_ok(ld_xc, d_cand, dtype) ||
                     !row_stride_ok(ld_wcc, d_cand, dtype)))
    return ROCS_ERR_ALIGNMENT;
  if (d_req > 0 && (!aligned16(XR) || !aligned16(W_CR) || !row_stride_ok(ld_xr, d_req, dtype) ||
                    !row_stride_ok(ld_wcr, d_req, dtype)))
    return ROCS_ERR_ALIGNMENT;
  cudaStream_t stream = (cudaStream_t)stream_;
  const float* Z = nullptr;
  const size_t z_bytes = d_req > 0 ? rocs_ikbo_linear_workspace(plan, d_out) : 0;
  if (row_stats != nullptr) {
    if (!aligned16(row_stats) || d_cand <= 0) return row_stats && d_cand <= 0 ? ROCS_ERR_INVALID_ARG : ROCS_ERR_ALIGNMENT;
    const size_t need = rocs_ikbo_linear_stats_workspace(plan, d_out);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
      return ROCS_ERR_WORKSPACE;
  }
  if (d_req > 0) {
    const size_t need = z_bytes;
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
      return ROCS_ERR_WORKSPACE;
    // Request half, once per request (Section 4.1): Z = X^R W_CR^T + bias, fp32.
    rocs_status_t st = linear_dispatch(dtype, plan->R, d_req, d_out, XR, ld_xr, W_CR, ld_wcr, bias,
                                       nullptr, 0, nullptr, ROCS_ACT_NONE, workspace, d_out,
                                       /*out_f32=*/true, stream);
    if (st != ROCS_OK) return st;
    Z = (const float*)workspace;
    bias = nullptr;
  }
  // Candidate half with the request term gathered in the epilogue (Eq. 14, Section 4.2.1).
  // The request half was enqueued directly in front: the candidate kernel may overlap its set-up
  // with it (it waits for it before reading Z).  Only meaningful when both went to tensor cores.
  const bool request_half_on_umma = Z != nullptr && dtype == ROCS_BF16 && g_path.load() == ROCS_PATH_AUTO &&
                                    umma_linear_supported(plan->R, d_req, d_out, ld_xr, ld_wcr, d_out, true);
  // Row sums for a following normalisation: left as partials by the candidate kernel's epilogue where
  // the CTA-pair kernel runs (and added up by a small kernel), otherwise taken from the stored output.
  float2* partials = nullptr;
  if (row_stats != nullptr && dtype == ROCS_BF16 && g_path.load() == ROCS_PATH_AUTO &&
      umma_linear_supported(plan->N, d_cand, d_out, ld_xc, ld_wcc, ld_y, false) &&
      umma_linear_ws2_supported(plan->N, d_cand, d_out, false))
    partials = reinterpret_cast<float2*>(static_cast<uint8_t*>(workspace) + z_bytes);
  rocs_status_t st = linear_dispatch(dtype, plan->N, d_cand, d_out, XC, ld_xc, W_CC, ld_wcc, bias, Z, d_out,
                                     Z ? plan->row2req : nullptr, act, Y, ld_y, /*out_f32=*/false, stream,
                                     request_half_on_umma, partials, plan->R);
  if (st != ROCS_OK || row_stats == nullptr) return st;
  if (partials != nullptr)
    return row_stats_from_partials(plan->N, umma_linear_ws2_stat_partials(d_out), partials,
                                   reinterpret_cast<float2*>(row_stats), stream);
  return row_stats_direct(dtype, plan->N, d_out, Y, ld_y, reinterpret_cast<float2*>(row_stats), stream);
}

rocs_status_t rocs_ikbo_linear(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t d_req,
                               int32_t d_cand, int32_t d_out, const void* XR, int64_t ld_xr,
                               const void* XC, int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                               const void* W_CC, int64_t ld_wcc, const float* bias, rocs_act_t act,
                               void* Y, int64_t ld_y, void* workspace, size_t workspace_bytes,
                               void* stream_) {
  return ikbo_linear_impl(plan, dtype, d_req, d_cand, d_out, XR, ld_xr, XC, ld_xc, W_CR, ld_wcr, W_CC, ld_wcc, bias,
                          act, Y, ld_y, nullptr, workspace, workspace_bytes, stream_);
}

size_t rocs_ikbo_linear_stats_workspace(const rocs_plan_t* plan, int32_t d_out) {
  if (!plan || d_out <= 0) return 0;
  return rocs_ikbo_linear_workspace(plan, d_out) +
         round_up((size_t)plan->N * (size_t)umma_linear_ws2_stat_partials(d_out) * sizeof(float2), 256);
}

rocs_status_t rocs_ikbo_linear_stats(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t d_req,
                                     int32_t d_cand, int32_t d_out, const void* XR, int64_t ld_xr,
                                     const void* XC, int64_t ld_xc, const void* W_CR, int64_t ld_wcr,
                                     const void* W_CC, int64_t ld_wcc, const float* bias, rocs_act_t act,
                                     void* Y, int64_t ld_y, float* row_stats, void* workspace,
                                     size_t workspace_bytes, void* stream_) {
  if (!row_stats && plan && plan->N > 0) return ROCS_ERR_INVALID_ARG;
  return ikbo_linear_impl(plan, dtype, d_req, d_cand, d_out, XR, ld_xr, XC, ld_xc, W_CR, ld_wcr, W_CC, ld_wcc, bias,
                          act, Y, ld_y, row_stats, workspace, workspace_bytes, stream_);
}

rocs_status_t rocs_weight_row_sums(rocs_dtype_t dtype, int32_t d_out, int32_t d_in, const void* W, int64_t ld_w,
                                   float* wbar, void* stream_) {
  if ((dtype != ROCS_BF16 && dtype != ROCS_F32) || d_out <= 0 || d_in <= 0 || !W || !wbar) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(wbar) || !row_stride_ok(ld_w, d_in, dtype)) return ROCS_ERR_ALIGNMENT;
  return weight_row_sums(dtype, d_out, d_in, W, ld_w, wbar, (cudaStream_t)stream_);
}

rocs_status_t rocs_linear_normed(rocs_dtype_t dtype, rocs_norm_t kind, int64_t M, int32_t d_in, int32_t d_out,
                                 const void* X, int64_t ld_x, const float* row_stats, float eps, const void* W,
                                 int64_t ld_w, const float* wbar, const float* bias, rocs_act_t act, void* Y,
                                 int64_t ld_y, void* stream_) {
  if ((dtype != ROCS_BF16 && dtype != ROCS_F32) || (kind != ROCS_NORM_LAYER && kind != ROCS_NORM_RMS))
    return ROCS_ERR_INVALID_ARG;
  if (M < 0 || d_in <= 0 || d_out <= 0 || !X || !W || !Y || !row_stats || !(eps >= 0.f)) return ROCS_ERR_INVALID_ARG;
  if (kind == ROCS_NORM_LAYER && !wbar) return ROCS_ERR_INVALID_ARG;
  if (act != ROCS_ACT_NONE && act != ROCS_ACT_RELU) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || !aligned16(bias) || !aligned16(wbar) || !aligned16(row_stats) ||
      !row_stride_ok(ld_x, d_in, dtype) || !row_stride_ok(ld_w, d_in, dtype) || !row_stride_ok(ld_y, d_out, dtype))
    return ROCS_ERR_ALIGNMENT;
  // The folded form lives in the epilogue of the wide-layer kernel; other shapes normalise with
  // rocs_group_norm and call rocs_linear.
  if (dtype != ROCS_BF16 || g_path.load() != ROCS_PATH_AUTO || d_out % 4 != 0 ||
      !umma_linear_pair_supported(M, d_in, d_out, false, false))
    return ROCS_ERR_UNSUPPORTED;
  RowNorm norm;
  norm.row_stats = reinterpret_cast<const float2*>(row_stats);
  norm.kind = (int)kind;
  norm.eps = eps;
  norm.wbar = wbar;
  return umma_linear_pair(M, d_in, d_out, X, ld_x, W, ld_w, bias, (int)act, Y, ld_y, (cudaStream_t)stream_, &norm);
}

rocs_status_t rocs_linear(rocs_dtype_t dtype, int64_t M, int32_t d_in, int32_t d_out, const void* X,
                          int64_t ld_x, const void* W, int64_t ld_w, const float* bias,
                          rocs_act_t act, void* Y, int64_t ld_y, void* stream_) {
  if (dtype != ROCS_BF16 && dtype != ROCS_F32) return ROCS_ERR_INVALID_ARG;
  if (M < 0 || d_in <= 0 || d_out <= 0 || !X || !W || !Y) return ROCS_ERR_INVALID_ARG;
  if (act != ROCS_ACT_NONE && act != ROCS_ACT_RELU) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || !aligned16(bias) || !row_stride_ok(ld_x, d_in, dtype) ||
      !row_stride_ok(ld_w, d_in, dtype) || !row_stride_ok(ld_y, d_out, dtype))
    return ROCS_ERR_ALIGNMENT;
  return linear_dispatch(dtype, M, d_in, d_out, X, ld_x, W, ld_w, bias, nullptr, 0, nullptr, act, Y,
                         ld_y, false, (cudaStream_t)stream_);
}

size_t rocs_dca_attention_workspace(const rocs_plan_t*, int32_t, int32_t, int32_t) { return 0; }

rocs_status_t rocs_dca_attention(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_q, int32_t H,
                                 int32_t dh, float scale, const void* Q, const void* K,
                                 const void* V, int64_t T, const int32_t* seq_offsets, void* O,
                                 void* workspace, size_t workspace_bytes, void* stream_) {
  (void)workspace;
  (void)workspace_bytes;
  if (!plan || (dtype != ROCS_BF16 && dtype != ROCS_F32)) return ROCS_ERR_INVALID_ARG;
  if (n_q <= 0 || H <= 0 || dh <= 0 || T < 0 || T > 0x7fffffffLL || !seq_offsets) return ROCS_ERR_INVALID_ARG;
  if (plan->N > 0 && (!Q || !O)) return ROCS_ERR_INVALID_ARG;
  if (T > 0 && (!K || !V)) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) ||
      ((int64_t)dh * (int64_t)elem_size(dtype)) % 16 != 0)
    return ROCS_ERR_ALIGNMENT;
  if (dh > 256) return ROCS_ERR_UNSUPPORTED;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)dh);
  cudaStream_t stream = (cudaStream_t)stream_;
  if (dtype == ROCS_BF16 && g_path.load() == ROCS_PATH_AUTO && umma_dca_supported(n_q, H, dh))
    return umma_dca(plan, n_q, H, dh, scale, Q, K, V, seq_offsets, T, O, stream);
  return simt_dca(dtype, plan, n_q, H, dh, scale, Q, K, V, seq_offsets, O, stream);
}

size_t rocs_glm_interaction_workspace(const rocs_plan_t* plan, int32_t n_r, int32_t n_c, int32_t n_co) {
  if (!plan || n_r < 0 || n_c < 0 || n_co <= 0) return 0;
  return round_up((size_t)plan->R * (size_t)n_co * (size_t)(n_r + n_c) * sizeof(float), 256);
}

rocs_status_t rocs_glm_interaction(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_r,
                                   int32_t n_c, int32_t d, const void* XR, const void* XC,
                                   const void* W, int32_t n_ro, int32_t n_co, void* YR, void* YC,
                                   void* OR_, void* OC, void* workspace, size_t workspace_bytes,
                                   void* stream_) {
  if (!plan || (dtype != ROCS_BF16 && dtype != ROCS_F32)) return ROCS_ERR_INVALID_ARG;
  if (n_r < 0 || n_c < 0 || n_r + n_c <= 0 || d <= 0 || n_ro < 0 || n_co < 0) return ROCS_ERR_INVALID_ARG;
  if ((n_r > 0 && plan->R > 0 && !XR) || (n_c > 0 && plan->N > 0 && !XC)) return ROCS_ERR_INVALID_ARG;
  if (!W && (n_ro != 0 || n_co != 0 || OR_ || OC)) return ROCS_ERR_INVALID_ARG;
  if (W && n_ro + n_co <= 0) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(XR) || !aligned16(XC) || !aligned16(W) || !aligned16(YR) || !aligned16(YC) ||
      !aligned16(OR_) || !aligned16(OC) || ((int64_t)d * (int64_t)elem_size(dtype)) % 16 != 0)
    return ROCS_ERR_ALIGNMENT;
  cudaStream_t stream = (cudaStream_t)stream_;
  float* zr = nullptr;
  if (W && n_co > 0) {
    const size_t need = rocs_glm_interaction_workspace(plan, n_r, n_c, n_co);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
      return ROCS_ERR_WORKSPACE;
    zr = (float*)workspace;
  }
  if (dtype == ROCS_BF16 && g_path.load() == ROCS_PATH_AUTO && umma_glm_supported(n_r, n_c, d, n_ro, n_co)) {
    // Request side once per request (tiny), candidate side on tensor cores.
    rocs_status_t st = glm_request_mma_supported(n_r, d, n_ro, n_co)
                           ? glm_request_mma(plan, n_r, n_c, d, XR, W, n_ro, n_co, YR, OR_, zr, stream)
                           : simt_glm(dtype, plan, n_r, n_c, d, XR, nullptr, W, n_ro, n_co, YR, nullptr, OR_,
                                      nullptr, zr, stream);
    if (st != ROCS_OK) return st;
    if (!YC && !OC) return ROCS_OK;
    return umma_glm(plan, n_r, n_c, d, XR, XC, W, n_ro, n_co, YC, OC, zr, stream);
  }
  return simt_glm(dtype, plan, n_r, n_c, d, XR, XC, W, n_ro, n_co, YR, YC, OR_, OC, zr, stream);
}

size_t rocs_glm_fm_projection_workspace(const rocs_plan_t* plan, int32_t d, int32_t k) {
  if (!plan || d <= 0 || k <= 0) return 0;
  return round_up((size_t)std::max(plan->R, 1) * (size_t)k * (size_t)d * sizeof(float), 256);
}

rocs_status_t rocs_glm_fm_projection(const rocs_plan_t* plan, rocs_dtype_t dtype, int32_t n_r, int32_t n_c,
                                     int32_t d, int32_t k, const void* XR, const void* XC, const void* P,
                                     void* FR, void* FC, void* workspace, size_t workspace_bytes, void* stream_) {
  if (!plan || (dtype != ROCS_BF16 && dtype != ROCS_F32)) return ROCS_ERR_INVALID_ARG;
  if (n_r <= 0 || n_c <= 0 || d <= 0 || k <= 0 || !P) return ROCS_ERR_INVALID_ARG;
  if ((plan->R > 0 && !XR) || (plan->N > 0 && FC && !XC)) return ROCS_ERR_INVALID_ARG;
  if (!aligned16(XR) || !aligned16(XC) || !aligned16(P) || !aligned16(FR) || !aligned16(FC) ||
      ((int64_t)d * (int64_t)elem_size(dtype)) % 16 != 0)
    return ROCS_ERR_ALIGNMENT;
  const size_t need = rocs_glm_fm_projection_workspace(plan, d, k);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return ROCS_ERR_WORKSPACE;
  return fm_projection(dtype, plan, n_r, n_c, d, k, XR, XC, P, FR, FC, (float*)workspace,
                       g_path.load() == ROCS_PATH_AUTO, (cudaStream_t)stream_);
}

rocs_status_t rocs_group_norm(rocs_dtype_t dtype, rocs_norm_t kind, int64_t M, int32_t d, const void* X,
                              int64_t ld_x, const void* gamma, const void* beta, float eps, void* Y, int64_t ld_y,
                              void* stream_) {
  if ((dtype != ROCS_BF16 && dtype != ROCS_F32) || (kind != ROCS_NORM_LAYER && kind != ROCS_NORM_RMS))
    return ROCS_ERR_INVALID_ARG;
  if (M < 0 || d <= 0 || ld_x < d || ld_y < d || !(eps >= 0.f)) return ROCS_ERR_INVALID_ARG;
  if (M > 0 && (!X || !Y)) return ROCS_ERR_INVALID_ARG;
  const int64_t es = (int64_t)elem_size(dtype);
  if (!aligned16(X) || !aligned16(Y) || !aligned16(gamma) || !aligned16(beta) || (ld_x * es) % 16 != 0 ||
      (ld_y * es) % 16 != 0)
    return ROCS_ERR_ALIGNMENT;
  return group_norm(dtype, (int)kind, M, d, X, ld_x, gamma, beta, eps, Y, ld_y, (cudaStream_t)stream_);
}

rocs_status_t rocs_last_device_status(uint32_t* detail_host) {
  uint32_t* word = device_status_word();
  if (!word) return ROCS_ERR_CUDA;
  uint32_t v = 0;
  ROCS_CUDA_TRY(cudaDeviceSynchronize());
  ROCS_CUDA_TRY(cudaMemcpy(&v, word, sizeof v, cudaMemcpyDeviceToHost));
  if (v != 0) {
    const uint32_t zero = 0;
    ROCS_CUDA_TRY(cudaMemcpy(word, &zero, sizeof zero, cudaMemcpyHostToDevice));
  }
  if (detail_host) *detail_host = v;
  return v == 0 ? ROCS_OK : ROCS_ERR_TIMEOUT;
}

}  // extern "C"
