// Helpers of the plain (non tensor-core) kernels.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

namespace rocs {

// Copies `rows` dense rows of `d` elements (fp32 or bf16, global memory) into shared memory as fp32
// with row stride `ds`.  Where rows are whole 16-byte vectors the block issues four vector loads per
// thread before it touches shared memory, so a request's operand arrives after about one memory
// latency instead of one per element (measured on the request-side kernels of the interaction
// operators: 16 dependent scalar loads per thread cost more than all of their arithmetic).
template <typename T>
__device__ __forceinline__ void rows_to_shared(const T* __restrict__ src, float* __restrict__ dst, int rows, int d,
                                               int ds) {
  constexpr int kVec = 16 / (int)sizeof(T);
  const int total = rows * d;
  if (d % kVec == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const int n_vec = total / kVec;
    constexpr int kBatch = 4;
    for (int base = threadIdx.x; base < n_vec; base += kBatch * blockDim.x) {
      uint4 raw[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int v = base + u * blockDim.x;
        if (v < n_vec) raw[u] = __ldg(reinterpret_cast<const uint4*>(src) + v);
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int v = base + u * blockDim.x;
        if (v >= n_vec) continue;
        const int e = v * kVec;
        float* out = dst + (e / d) * ds + e % d;
        if constexpr (sizeof(T) == 4) {
          out[0] = __uint_as_float(raw[u].x);
          out[1] = __uint_as_float(raw[u].y);
          out[2] = __uint_as_float(raw[u].z);
          out[3] = __uint_as_float(raw[u].w);
        } else {
          const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {  // bf16 -> fp32 is a shift into the high half
            out[2 * j] = __uint_as_float(w[j] << 16);
            out[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
          }
        }
      }
    }
  } else {
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
      if constexpr (sizeof(T) == 4)
        dst[(e / d) * ds + e % d] = reinterpret_cast<const float*>(src)[e];
      else
        dst[(e / d) * ds + e % d] = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(src)[e]);
    }
  }
}

}  // namespace rocs
