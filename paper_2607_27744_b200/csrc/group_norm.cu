// Group-local normalisation (Eq. 7): every row of ONE group's tensor X [M, d] is normalised over
// its own d coordinates, so no statistic spans two groups (request rows and candidate rows are
// separate tensors and separate calls).
//   LayerNorm:  y = (x - mean) / sqrt(var + eps) * gamma + beta     (biased variance)
//   RMSNorm:    y = x / sqrt(mean(x^2) + eps) * gamma
// Pure streaming work (read once, write once): one warp per row, the row held in registers as
// 16-byte vectors (coalesced 512-byte warp accesses), statistics in fp32 by warp shuffles, the
// variance taken around the mean from the registers (no E[x^2] - E[x]^2 cancellation).  Rows
// wider than the register variant allows, or with a width that is no multiple of one warp's
// 16-byte vectors, run on a two-pass variant that re-reads the row (from L1/L2).
#include <algorithm>

#include "rocs_internal.h"

namespace rocs {
namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
struct Vec;  // 16 bytes of T
template <>
struct Vec<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ void load(const float* p, float (&f)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&f)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// d == NV * 32 * Vec<T>::kElems: lane l owns vectors l, l + 32, ...
template <typename T, int NV>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
group_norm_rows_kernel(int kind, int64_t M, const T* __restrict__ X, int64_t ld_x, const T* __restrict__ gamma,
                       const T* __restrict__ beta, float eps, T* __restrict__ Y, int64_t ld_y) {
  constexpr int E = Vec<T>::kElems;
  constexpr int d = NV * 32 * E;
  const int lane = threadIdx.x % 32;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerBlock + threadIdx.x / 32;
  const int64_t n_warps = (int64_t)gridDim.x * kWarpsPerBlock;
  for (int64_t row = warp; row < M; row += n_warps) {
    float x[NV][E];
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      Vec<T>::load(X + row * ld_x + (v * 32 + lane) * E, x[v]);
#pragma unroll
      for (int e = 0; e < E; ++e) s += x[v][e];
    }
    float mean = 0.f;
    if (kind == ROCS_NORM_LAYER) mean = warp_sum(s) * (1.f / d);
    float sq = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
      for (int e = 0; e < E; ++e) {
        x[v][e] -= mean;
        sq = fmaf(x[v][e], x[v][e], sq);
      }
    const float inv = rsqrtf(warp_sum(sq) * (1.f / d) + eps);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int col = (v * 32 + lane) * E;
      float g[E], b[E];
#pragma unroll
      for (int e = 0; e < E; ++e) {
        g[e] = 1.f;
        b[e] = 0.f;
      }
      if (gamma) Vec<T>::load(gamma + col, g);
      if (beta && kind == ROCS_NORM_LAYER) Vec<T>::load(beta + col, b);
#pragma unroll
      for (int e = 0; e < E; ++e) x[v][e] = fmaf(x[v][e] * inv, g[e], b[e]);
      Vec<T>::store(Y + row * ld_y + col, x[v]);
    }
  }
}

__device__ __forceinline__ float ld_f(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16* p, int64_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_f(float* p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_f(__nv_bfloat16* p, int64_t i, float v) { p[i] = __float2bfloat16_rn(v); }

// any d: the row is read three times (sum, centred squares, output), scalar accesses
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
group_norm_general_kernel(int kind, int64_t M, int32_t d, const T* __restrict__ X, int64_t ld_x,
                          const T* __restrict__ gamma, const T* __restrict__ beta, float eps, T* __restrict__ Y,
                          int64_t ld_y) {
  const int lane = threadIdx.x % 32;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerBlock + threadIdx.x / 32;
  const int64_t n_warps = (int64_t)gridDim.x * kWarpsPerBlock;
  for (int64_t row = warp; row < M; row += n_warps) {
    const T* x = X + row * ld_x;
    float mean = 0.f;
    if (kind == ROCS_NORM_LAYER) {
      float s = 0.f;
      for (int e = lane; e < d; e += 32) s += ld_f(x, e);
      mean = warp_sum(s) / d;
    }
    float sq = 0.f;
    for (int e = lane; e < d; e += 32) {
      const float c = ld_f(x, e) - mean;
      sq = fmaf(c, c, sq);
    }
    const float inv = rsqrtf(warp_sum(sq) / d + eps);
    for (int e = lane; e < d; e += 32) {
      const float g = gamma ? ld_f(gamma, e) : 1.f;
      const float b = (beta && kind == ROCS_NORM_LAYER) ? ld_f(beta, e) : 0.f;
      st_f(Y, row * ld_y + e, fmaf((ld_f(x, e) - mean) * inv, g, b));
    }
  }
}

int sm_count_norm() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

template <typename T>
rocs_status_t launch_norm(int kind, int64_t M, int32_t d, const void* X, int64_t ld_x, const void* gamma,
                          const void* beta, float eps, void* Y, int64_t ld_y, cudaStream_t stream) {
  if (M == 0) return ROCS_OK;
  constexpr int E = Vec<T>::kElems;
  const int64_t want = (M + kWarpsPerBlock - 1) / kWarpsPerBlock;
  const int grid = (int)std::min<int64_t>(want, (int64_t)sm_count_norm() * 8);  // 64 resident warps per SM
  const int threads = kWarpsPerBlock * 32;
  const bool vec_ok = d % (32 * E) == 0 && ld_x % E == 0 && ld_y % E == 0;
  const int nv = vec_ok ? d / (32 * E) : 0;
#define ROCS_NORM_LAUNCH(NV_)                                                                                      \
  group_norm_rows_kernel<T, NV_><<<grid, threads, 0, stream>>>(kind, M, (const T*)X, ld_x, (const T*)gamma,        \
                                                               (const T*)beta, eps, (T*)Y, ld_y)
  switch (nv) {
    case 1: ROCS_NORM_LAUNCH(1); break;
    case 2: ROCS_NORM_LAUNCH(2); break;
    case 3: ROCS_NORM_LAUNCH(3); break;
    case 4: ROCS_NORM_LAUNCH(4); break;
    case 6: ROCS_NORM_LAUNCH(6); break;
    case 8: ROCS_NORM_LAUNCH(8); break;
    default:
      group_norm_general_kernel<T><<<grid, threads, 0, stream>>>(kind, M, d, (const T*)X, ld_x, (const T*)gamma,
                                                                 (const T*)beta, eps, (T*)Y, ld_y);
  }
#undef ROCS_NORM_LAUNCH
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace

rocs_status_t group_norm(rocs_dtype_t dt, int kind, int64_t M, int32_t d, const void* X, int64_t ld_x,
                         const void* gamma, const void* beta, float eps, void* Y, int64_t ld_y, cudaStream_t stream) {
  if (dt == ROCS_F32) return launch_norm<float>(kind, M, d, X, ld_x, gamma, beta, eps, Y, ld_y, stream);
  return launch_norm<__nv_bfloat16>(kind, M, d, X, ld_x, gamma, beta, eps, Y, ld_y, stream);
}

}  // namespace rocs
