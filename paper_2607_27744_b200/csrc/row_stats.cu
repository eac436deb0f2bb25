// Per-row sums for a group-local normalisation (Eq. 7) that is folded into the layer AFTER the one
// that writes the rows:  norm(y) W^T = sc (y W^T) + sh (W 1),  so the rows are never normalised in
// memory.  The producing layer's epilogue leaves a few (sum, sum of squares) partials per row; they
// are added up here in a fixed order.  Also: the same sums straight from a stored tensor (for layers
// whose kernel does not emit partials) and the row sums of a weight matrix (W 1, LayerNorm's shift).
#include "rocs_internal.h"

namespace rocs {
namespace {

__global__ void stats_from_partials_kernel(int64_t M, int32_t P, const float2* __restrict__ partials,
                                           float2* __restrict__ row_stats) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  float s = 0.f, q = 0.f;
  for (int32_t k = 0; k < P; ++k) {
    const float2 v = partials[i * P + k];
    s += v.x;
    q += v.y;
  }
  row_stats[i] = make_float2(s, q);
}

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// one warp per row; lanes stride over the columns, partial sums combined by a fixed shuffle tree
template <typename T>
__global__ void stats_direct_kernel(int64_t M, int32_t d, const T* __restrict__ Y, int64_t ld, float2* __restrict__ out,
                                    int32_t as_weight_sums, float* __restrict__ wbar) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  if (row >= M) return;
  const int lane = threadIdx.x % 32;
  float s = 0.f, q = 0.f;
  for (int32_t c = lane; c < d; c += 32) {
    const float v = to_f32<T>(Y[row * ld + c]);
    s += v;
    q = fmaf(v, v, q);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    q += __shfl_xor_sync(0xffffffffu, q, o);
  }
  if (lane == 0) {
    if (as_weight_sums) wbar[row] = s; else out[row] = make_float2(s, q);
  }
}

}  // namespace

rocs_status_t row_stats_from_partials(int64_t M, int32_t P, const float2* partials, float2* row_stats,
                                      cudaStream_t stream) {
  if (M == 0) return ROCS_OK;
  stats_from_partials_kernel<<<(unsigned)((M + 255) / 256), 256, 0, stream>>>(M, P, partials, row_stats);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

static rocs_status_t launch_direct(rocs_dtype_t dt, int64_t M, int32_t d, const void* Y, int64_t ld, float2* out,
                                   int32_t as_weight_sums, float* wbar, cudaStream_t stream) {
  if (M == 0) return ROCS_OK;
  const unsigned blocks = (unsigned)((M + 7) / 8);
  if (dt == ROCS_BF16)
    stats_direct_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(M, d, (const __nv_bfloat16*)Y, ld, out, as_weight_sums, wbar);
  else
    stats_direct_kernel<float><<<blocks, 256, 0, stream>>>(M, d, (const float*)Y, ld, out, as_weight_sums, wbar);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

rocs_status_t row_stats_direct(rocs_dtype_t dt, int64_t M, int32_t d, const void* Y, int64_t ld_y, float2* row_stats,
                               cudaStream_t stream) {
  return launch_direct(dt, M, d, Y, ld_y, row_stats, 0, nullptr, stream);
}

rocs_status_t weight_row_sums(rocs_dtype_t dt, int32_t d_out, int32_t d_in, const void* W, int64_t ld_w, float* wbar,
                              cudaStream_t stream) {
  return launch_direct(dt, d_out, d_in, W, ld_w, nullptr, 1, wbar, stream);
}

}  // namespace rocs
