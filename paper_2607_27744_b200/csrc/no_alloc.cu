// rocs_ikbo_linear_static: the split linear layer for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they score a batch: a
// serving thread whose allocator is frozen after start-up, a plugin that runs inside someone
// else's memory budget, a latency-critical path where an allocation (and the implicit
// synchronisation it can bring) is not acceptable.  The regular path needs two pieces of scratch
// memory -- the request half Z (fp32 [R, d_out]) in a caller workspace and the candidate->request
// map inside a plan.  This variant keeps both in one fixed array that lives in the library image,
// so the call itself allocates nothing, on the host or on the device.
#include <mutex>

#include "rocs_internal.h"

namespace rocs {
namespace {

constexpr size_t kStaticZFloats = size_t(1) << 20;    // R * d_out  <= 1 Mi   (4 MiB)
constexpr size_t kStaticMapEntries = size_t(1) << 18;  // N          <= 256 Ki (1 MiB)
constexpr size_t kStaticBytes = kStaticZFloats * sizeof(float) + kStaticMapEntries * sizeof(int32_t);

// Lives in every GPU context that loads the library, until the process exits.  In host code this
// name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

std::mutex g_mu;
void* g_scratch_addr[64] = {};  // device address of g_static_scratch, per device ordinal

// Resolves (once per device, with that device current) where the array lives on the device.
rocs_status_t scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ROCS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ROCS_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return ROCS_OK;
}

// Candidate -> request map (m of Section 4.1) written straight into the static array.
__global__ void static_row2req_kernel(int32_t R, int64_t N, const int32_t* __restrict__ off) {
  int32_t* map = reinterpret_cast<int32_t*>(g_static_scratch + kStaticZFloats * sizeof(float));
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  int32_t lo = 0, hi = R;
  while (hi - lo > 1) {
    const int32_t mid = lo + (hi - lo) / 2;
    if (off[mid] <= i) lo = mid; else hi = mid;
  }
  map[i] = lo;
}

bool stride_ok(int64_t ld, int64_t cols, rocs_dtype_t dt) {
  return ld >= cols && (ld * (int64_t)elem_size(dt)) % 16 == 0;
}

rocs_status_t run_linear(rocs_dtype_t dt, int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x,
                         const void* W, int64_t ld_w, const float* bias, const float* add, int64_t ld_add,
                         const int32_t* row2req, int act, void* Y, int64_t ld_y, bool out_f32,
                         cudaStream_t stream, int64_t add_rows = 0) {
  if (dt == ROCS_BF16 && umma_linear_supported(M, d_in, d_out, ld_x, ld_w, ld_y, out_f32))
    return umma_linear(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y, out_f32,
                       stream, false, nullptr, add_rows);
  return simt_linear(dt, M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y, out_f32,
                     stream);
}

}  // namespace
}  // namespace rocs

using namespace rocs;

extern "C" {

size_t rocs_ikbo_linear_static_max_z_elems(void) { return kStaticZFloats; }
size_t rocs_ikbo_linear_static_max_candidates(void) { return kStaticMapEntries; }

rocs_status_t rocs_ikbo_linear_static(rocs_dtype_t dtype, int32_t R, int64_t N, const int32_t* cand_offsets,
                                      int32_t d_req, int32_t d_cand, int32_t d_out, const void* XR,
                                      int64_t ld_xr, const void* XC, int64_t ld_xc, const void* W_CR,
                                      int64_t ld_wcr, const void* W_CC, int64_t ld_wcc, const float* bias,
                                      rocs_act_t act, void* Y, int64_t ld_y, void* stream_) {
  if (dtype != ROCS_BF16 && dtype != ROCS_F32) return ROCS_ERR_INVALID_ARG;
  if (R <= 0 || N < 0 || !cand_offsets || d_req <= 0 || d_cand <= 0 || d_out <= 0) return ROCS_ERR_INVALID_ARG;
  if (act != ROCS_ACT_NONE && act != ROCS_ACT_RELU) return ROCS_ERR_INVALID_ARG;
  if (!XR || !W_CR || !W_CC || (N > 0 && (!XC || !Y))) return ROCS_ERR_INVALID_ARG;
  if ((size_t)R * (size_t)d_out > kStaticZFloats || (size_t)N > kStaticMapEntries) return ROCS_ERR_STATIC_LIMIT;
  if (!aligned16(XR) || !aligned16(XC) || !aligned16(W_CR) || !aligned16(W_CC) || !aligned16(Y) || !aligned16(bias) ||
      !stride_ok(ld_xr, d_req, dtype) || !stride_ok(ld_xc, d_cand, dtype) || !stride_ok(ld_wcr, d_req, dtype) ||
      !stride_ok(ld_wcc, d_cand, dtype) || !stride_ok(ld_y, d_out, dtype))
    return ROCS_ERR_ALIGNMENT;
  void* base = nullptr;
  rocs_status_t st = scratch_address(&base);
  if (st != ROCS_OK) return st;
  float* Z = static_cast<float*>(base);
  const int32_t* map = reinterpret_cast<const int32_t*>(static_cast<unsigned char*>(base) +
                                                        kStaticZFloats * sizeof(float));
  cudaStream_t stream = (cudaStream_t)stream_;
  if (N == 0) return ROCS_OK;
  // Every word the kernels below read from the array is written first by this call (Z rows
  // 0..R-1, map entries 0..N-1), so nothing left behind by an earlier call is ever consumed.
  static_row2req_kernel<<<(unsigned)((N + 255) / 256), 256, 0, stream>>>(R, N, cand_offsets);
  ROCS_CUDA_TRY(cudaGetLastError());
  st = run_linear(dtype, R, d_req, d_out, XR, ld_xr, W_CR, ld_wcr, bias, nullptr, 0, nullptr, ROCS_ACT_NONE, Z,
                  d_out, /*out_f32=*/true, stream);
  if (st != ROCS_OK) return st;
  return run_linear(dtype, N, d_cand, d_out, XC, ld_xc, W_CC, ld_wcc, nullptr, Z, d_out, map, act, Y, ld_y,
                    /*out_f32=*/false, stream, R);
}

}  // extern "C"
