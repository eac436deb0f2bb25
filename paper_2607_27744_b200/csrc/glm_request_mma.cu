// Request side of the GLM interaction (Eq. 9-10, top rows of the masked matrix) and of its row-axis
// compression (Eq. 5-6), bf16, once per request:
//     YR[r] = [ X^R_r X^R_r^T , 0 ]        OR[r] = W_RR YR[r]        ZR[r] = W_CR YR[r]  (fp32)
// ZR is the request term the candidate kernel adds to every candidate of the request.
//
// One block of 8 warps per request.  The n_r x n_r Gram block comes from warp-level tensor-core
// products (mma.sync m16n8k16) straight out of a bf16 copy of X^R_r in shared memory: both operands
// of X^R X^R^T are rows of that copy with the d index contiguous, which is the layout ldmatrix hands
// to the row-major A and the column-major B fragment alike.  A plain FMA version of the same block
// spent its time waiting on shared-memory reads with two warps per scheduler (10 us for 128 requests
// of 32 x 128); the rest of the kernel (the small products with W) stays on plain FMAs.
#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Shared memory: xb bf16 [n_rp][d + 8] (n_rp = n_r rounded up to 16, padding rows zero; a row stride
// of 16 mod 32 bytes keeps ldmatrix free of bank conflicts), g fp32 [n_r][n_r], w fp32 [n_ro + n_co][n_r].
__global__ void __launch_bounds__(kThreads) glm_request_mma_kernel(
    int32_t n_r, int32_t n_c, int32_t d, const __nv_bfloat16* __restrict__ XR, const __nv_bfloat16* __restrict__ W,
    int32_t n_ro, int32_t n_co, __nv_bfloat16* __restrict__ YR, __nv_bfloat16* __restrict__ OR_,
    float* __restrict__ ZR) {
  extern __shared__ __align__(16) uint8_t smem_req[];
  const int32_t n = n_r + n_c;
  const int32_t n_rp = (n_r + 15) / 16 * 16;
  const int32_t row_bytes = (d + 8) * 2;
  uint8_t* xb = smem_req;
  float* g = reinterpret_cast<float*>(xb + (size_t)n_rp * row_bytes);
  float* w = g + (size_t)n_r * n_r;
  const int32_t r = blockIdx.x;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  // the candidate kernel launched behind this one may start: it waits for this grid before it reads ZR
  ptx::griddep_launch_dependents();

  // X^R_r as it is (bf16), 16 bytes per load, four loads in flight per thread
  const int32_t vec_per_row = d / 8;
  const int32_t n_vec = n_r * vec_per_row;
  const uint4* src = reinterpret_cast<const uint4*>(XR + (int64_t)r * n_r * d);
  for (int32_t base = threadIdx.x; base < n_vec; base += 4 * kThreads) {
    uint4 raw[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (base + u * kThreads < n_vec) raw[u] = __ldg(src + base + u * kThreads);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int32_t v = base + u * kThreads;
      if (v < n_vec) *reinterpret_cast<uint4*>(xb + (v / vec_per_row) * row_bytes + (v % vec_per_row) * 16) = raw[u];
    }
  }
  for (int32_t v = n_vec + threadIdx.x; v < n_rp * vec_per_row; v += kThreads)
    *reinterpret_cast<uint4*>(xb + (v / vec_per_row) * row_bytes + (v % vec_per_row) * 16) = make_uint4(0u, 0u, 0u, 0u);
  if (W)
    for (int32_t e = threadIdx.x; e < (n_ro + n_co) * n_r; e += kThreads)
      w[e] = __bfloat162float(W[(int64_t)(e / n_r) * n + e % n_r]);
  __syncthreads();

  // Gram block: 16 x 8 output tiles dealt round the warps
  const int32_t n_nt = n_rp / 8, n_tiles = (n_rp / 16) * n_nt;
  const uint32_t xb_addr = ptx::smem_u32(xb);
  const int g8 = lane / 4, t4 = lane % 4;
  for (int32_t t = warp; t < n_tiles; t += kThreads / 32) {
    const int32_t m0 = (t / n_nt) * 16, n0 = (t % n_nt) * 8;
    // ldmatrix row addresses: A = four 8x8 blocks (rows m0.., m0+8.. x columns k0.., k0+8..), B = two
    // (rows n0.. x columns k0.., k0+8..)
    const uint32_t a_addr = xb_addr + (m0 + (lane & 7) + ((lane >> 3) & 1) * 8) * row_bytes + ((lane >> 4) & 1) * 16;
    const uint32_t b_addr = xb_addr + (n0 + (lane & 7)) * row_bytes + ((lane >> 3) & 1) * 16;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    for (int32_t k0 = 0; k0 < d; k0 += 16) {
      uint32_t a[4], b[2];
      ldsm_x4(a_addr + k0 * 2, a);
      ldsm_x2(b_addr + k0 * 2, b);
      mma_bf16(c, a, b);
    }
    const int32_t col = n0 + 2 * t4;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int32_t row = m0 + g8 + h * 8;
      if (row < n_r) {
        if (col < n_r) g[row * n_r + col] = c[2 * h];
        if (col + 1 < n_r) g[row * n_r + col + 1] = c[2 * h + 1];
      }
    }
  }
  __syncthreads();

  if (YR)
    for (int32_t idx = threadIdx.x; idx < n_r * n; idx += kThreads) {
      const int32_t a = idx / n, b = idx % n;
      YR[(int64_t)r * n_r * n + idx] = __float2bfloat16_rn(b < n_r ? g[a * n_r + b] : 0.f);
    }
  if (W) {
    for (int32_t idx = threadIdx.x; idx < (n_ro + n_co) * n; idx += kThreads) {
      const int32_t o = idx / n, b = idx % n;
      float acc = 0.f;
      if (b < n_r) {
        float acc1 = 0.f;
        int32_t a = 0;
        for (; a + 1 < n_r; a += 2) {
          acc = fmaf(w[o * n_r + a], g[a * n_r + b], acc);
          acc1 = fmaf(w[o * n_r + a + 1], g[(a + 1) * n_r + b], acc1);
        }
        if (a < n_r) acc = fmaf(w[o * n_r + a], g[a * n_r + b], acc);
        acc += acc1;
      }
      if (o < n_ro) {
        if (OR_) OR_[((int64_t)r * n_ro + o) * n + b] = __float2bfloat16_rn(acc);
      } else if (ZR) {
        ZR[((int64_t)r * n_co + (o - n_ro)) * n + b] = acc;
      }
    }
  }
}

size_t request_smem(int32_t n_r, int32_t d, int32_t n_ro, int32_t n_co) {
  const size_t n_rp = (size_t)(n_r + 15) / 16 * 16;
  return n_rp * (size_t)(d + 8) * 2 + ((size_t)n_r * n_r + (size_t)(n_ro + n_co) * n_r) * sizeof(float);
}

}  // namespace

bool glm_request_mma_supported(int32_t n_r, int32_t d, int32_t n_ro, int32_t n_co) {
  return n_r >= 1 && d >= 16 && d % 16 == 0 && request_smem(n_r, d, n_ro, n_co) <= 200 * 1024;
}

rocs_status_t glm_request_mma(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, const void* XR,
                              const void* W, int32_t n_ro, int32_t n_co, void* YR, void* OR_, float* zr,
                              cudaStream_t stream) {
  if (plan->R == 0) return ROCS_OK;
  const size_t smem = request_smem(n_r, d, n_ro, n_co);
  ROCS_CUDA_TRY(cudaFuncSetAttribute(glm_request_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  glm_request_mma_kernel<<<plan->R, kThreads, smem, stream>>>(n_r, n_c, d, (const __nv_bfloat16*)XR,
                                                             (const __nv_bfloat16*)W, n_ro, n_co,
                                                             (__nv_bfloat16*)YR, (__nv_bfloat16*)OR_, zr);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
