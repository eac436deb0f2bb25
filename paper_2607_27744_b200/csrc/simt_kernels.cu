// General CUDA-core kernels: fp32 FMA arithmetic on fp32 or bf16 storage.  They accept every
// legal shape, carry the fp32 path, and serve bf16 shapes the tensor-core kernels do not take.
// Every output row is produced by a fixed instruction sequence over that row's own inputs, so
// results are bitwise deterministic and independent of neighbouring candidates (Eq. 1).
#include "rocs_internal.h"
#include "simt_util.cuh"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

__device__ __forceinline__ float ld_f(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16* p, int64_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_f(float* p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_f(__nv_bfloat16* p, int64_t i, float v) { p[i] = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Linear: Y[i, n] = act(sum_k X[i, k] W[n, k] + bias[n] + add[row2req[i], n])      (Eq. 4 / Eq. 14)
// 64x64 output tile per block, 16-wide k slices through shared memory, 4x4 outputs per thread.
// ---------------------------------------------------------------------------------------------
constexpr int LBM = 64, LBN = 64, LBK = 16;

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256) linear_simt_kernel(
    int64_t M, int32_t d_in, int32_t d_out, const TIn* __restrict__ X, int64_t ld_x,
    const TIn* __restrict__ W, int64_t ld_w, const float* __restrict__ bias,
    const float* __restrict__ add, int64_t ld_add, const int32_t* __restrict__ row2req, int act,
    TOut* __restrict__ Y, int64_t ld_y) {
  __shared__ float As[LBK][LBM + 4];
  __shared__ float Bs[LBK][LBN + 4];
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  const int64_t m0 = (int64_t)blockIdx.x * LBM;
  const int32_t n0 = blockIdx.y * LBN;
  float acc[4][4] = {};
  for (int32_t k0 = 0; k0 < d_in; k0 += LBK) {
    for (int e = tid; e < LBM * LBK; e += 256) {
      const int r = e / LBK, k = e % LBK;
      const int64_t gm = m0 + r;
      As[k][r] = (gm < M && k0 + k < d_in) ? ld_f(X, gm * ld_x + k0 + k) : 0.f;
      const int32_t gn = n0 + r;
      Bs[k][r] = (gn < d_out && k0 + k < d_in) ? ld_f(W, (int64_t)gn * ld_w + k0 + k) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < LBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
    const float* add_row = add ? add + (int64_t)(row2req ? row2req[gm] : gm) * ld_add : nullptr;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int32_t gn = n0 + tx * 4 + j;
      if (gn >= d_out) continue;
      float v = acc[i][j];
      if (bias) v += bias[gn];
      if (add_row) v += add_row[gn];
      if (act == ROCS_ACT_RELU) v = fmaxf(v, 0.f);
      st_f(Y, gm * ld_y + gn, v);
    }
  }
}

template <typename TIn, typename TOut>
rocs_status_t launch_linear(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x,
                            const void* W, int64_t ld_w, const float* bias, const float* add,
                            int64_t ld_add, const int32_t* row2req, int act, void* Y, int64_t ld_y,
                            cudaStream_t stream) {
  if (M == 0 || d_out == 0) return ROCS_OK;
  dim3 grid((unsigned)((M + LBM - 1) / LBM), (unsigned)((d_out + LBN - 1) / LBN));
  linear_simt_kernel<TIn, TOut><<<grid, 256, 0, stream>>>(
      M, d_in, d_out, (const TIn*)X, ld_x, (const TIn*)W, ld_w, bias, add, ld_add, row2req, act,
      (TOut*)Y, ld_y);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

// ---------------------------------------------------------------------------------------------
// Cross attention (Eq. 13): one warp per (query row, head).  Keys are visited 32 at a time (one
// per lane) with a running maximum and normaliser; values are accumulated with lanes spread
// over the head dimension.  The request of the row comes from row2req, its keys from
// seq_offsets: K/V are read in place, never copied per candidate.
// ---------------------------------------------------------------------------------------------
constexpr int DCA_WARPS = 4;
constexpr int DCA_MAX_DH = 256;

template <typename T>
__global__ void __launch_bounds__(DCA_WARPS * 32) dca_simt_kernel(
    int64_t n_rows, int32_t n_q, int32_t H, int32_t dh, float scale, const T* __restrict__ Q,
    const T* __restrict__ K, const T* __restrict__ V, const int32_t* __restrict__ row2req,
    const int32_t* __restrict__ seq_offsets, T* __restrict__ O) {
  __shared__ float qs[DCA_WARPS][DCA_MAX_DH];
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int64_t item = (int64_t)blockIdx.x * DCA_WARPS + warp;
  if (item >= n_rows * H) return;
  const int64_t qrow = item / H;
  const int32_t h = (int32_t)(item % H);
  const int32_t r = row2req[qrow / n_q];
  const int64_t s0 = seq_offsets[r];
  const int32_t L = seq_offsets[r + 1] - seq_offsets[r];
  const int64_t hd = (int64_t)H * dh;
  const int64_t qbase = qrow * hd + (int64_t)h * dh;
  for (int e = lane; e < dh; e += 32) qs[warp][e] = ld_f(Q, qbase + e);
  __syncwarp();
  float m = -INFINITY, l = 0.f;
  float acc[DCA_MAX_DH / 32];
#pragma unroll
  for (int u = 0; u < DCA_MAX_DH / 32; ++u) acc[u] = 0.f;
  for (int32_t j0 = 0; j0 < L; j0 += 32) {
    const int32_t j = j0 + lane;
    float s = -INFINITY;
    if (j < L) {
      const int64_t kb = (s0 + j) * hd + (int64_t)h * dh;
      float dot = 0.f;
      for (int e = 0; e < dh; ++e) dot = fmaf(qs[warp][e], ld_f(K, kb + e), dot);
      s = dot * scale;
    }
    float cmax = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
    const float m_new = fmaxf(m, cmax);
    const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
    const float p = (j < L) ? expf(s - m_new) : 0.f;
    float psum = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
    l = l * corr + psum;
#pragma unroll
    for (int u = 0; u < DCA_MAX_DH / 32; ++u) acc[u] *= corr;
    const int32_t cnt = min(32, L - j0);
    for (int jj = 0; jj < cnt; ++jj) {
      const float pj = __shfl_sync(0xffffffffu, p, jj);
      const int64_t vb = (s0 + j0 + jj) * hd + (int64_t)h * dh;
#pragma unroll
      for (int u = 0; u < DCA_MAX_DH / 32; ++u) {
        const int e = lane + 32 * u;
        if (e < dh) acc[u] = fmaf(pj, ld_f(V, vb + e), acc[u]);
      }
    }
    m = m_new;
  }
  const float inv = (L > 0) ? 1.f / l : 0.f;
#pragma unroll
  for (int u = 0; u < DCA_MAX_DH / 32; ++u) {
    const int e = lane + 32 * u;
    if (e < dh) st_f(O, qbase + e, acc[u] * inv);
  }
}

// ---------------------------------------------------------------------------------------------
// GLM factorization machine (Eq. 9-10) and row-axis compression (Eq. 5-6).
// Request kernel (one block per request): YR = [X^R X^R^T, 0], OR = W_RR YR, and the request
// term ZR = W_CR YR that the candidate kernel adds to every candidate of the request.
// Candidate kernel (one block per candidate): YC = [X^C X^R^T, X^C X^C^T], OC = ZR + W_CC YC.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) glm_request_simt_kernel(
    int32_t n_r, int32_t n_c, int32_t d, const T* __restrict__ XR, const T* __restrict__ W,
    int32_t n_ro, int32_t n_co, T* __restrict__ YR, T* __restrict__ OR_, float* __restrict__ ZR) {
  extern __shared__ float sm[];
  const int32_t n = n_r + n_c;
  const int32_t ds = d + 1;                    // padded row stride: rows land in different banks
  float* xr = sm;                              // [n_r, d + 1]
  float* g = xr + (size_t)n_r * ds;            // [n_r, n_r]
  float* w = g + (size_t)n_r * n_r;            // [n_ro + n_co, n_r]: the request columns of W
  const int32_t r = blockIdx.x;
  // a candidate kernel launched behind this one as a programmatic dependent may start now: it streams
  // its own operands and waits for this grid only before it reads ZR
  ptx::griddep_launch_dependents();
  rows_to_shared(XR + (int64_t)r * n_r * d, xr, n_r, d, ds);
  if (W)
    for (int e = threadIdx.x; e < (n_ro + n_co) * n_r; e += blockDim.x)
      w[e] = ld_f(W, (int64_t)(e / n_r) * n + e % n_r);
  __syncthreads();
  // four neighbouring columns of one row per thread: four independent accumulation chains
  const int n_r4 = (n_r + 3) / 4;
  for (int idx = threadIdx.x; idx < n_r * n_r4; idx += blockDim.x) {
    const int a = idx / n_r4, b0 = (idx % n_r4) * 4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const float* xa = xr + a * ds;
    const float* xb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) xb[u] = xr + min(b0 + u, n_r - 1) * ds;
#pragma unroll 4
    for (int e = 0; e < d; ++e) {
      const float va = xa[e];
#pragma unroll
      for (int u = 0; u < 4; ++u) acc[u] = fmaf(va, xb[u][e], acc[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (b0 + u < n_r) g[a * n_r + b0 + u] = acc[u];
  }
  __syncthreads();
  if (YR)
    for (int idx = threadIdx.x; idx < n_r * n; idx += blockDim.x) {
      const int a = idx / n, b = idx % n;
      st_f(YR, (int64_t)r * n_r * n + idx, b < n_r ? g[a * n_r + b] : 0.f);
    }
  if (W) {
    for (int idx = threadIdx.x; idx < (n_ro + n_co) * n; idx += blockDim.x) {
      const int o = idx / n, b = idx % n;
      float acc = 0.f;
      if (b < n_r) {
        float acc1 = 0.f;  // two chains: the sum is short but each step waits for two shared-memory reads
        int a = 0;
        for (; a + 1 < n_r; a += 2) {
          acc = fmaf(w[o * n_r + a], g[a * n_r + b], acc);
          acc1 = fmaf(w[o * n_r + a + 1], g[(a + 1) * n_r + b], acc1);
        }
        if (a < n_r) acc = fmaf(w[o * n_r + a], g[a * n_r + b], acc);
        acc += acc1;
      }
      if (o < n_ro) {
        if (OR_) st_f(OR_, ((int64_t)r * n_ro + o) * n + b, acc);
      } else if (ZR) {
        ZR[((int64_t)r * n_co + (o - n_ro)) * n + b] = acc;
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(128) glm_candidate_simt_kernel(
    int32_t n_r, int32_t n_c, int32_t d, const T* __restrict__ XR, const T* __restrict__ XC,
    const T* __restrict__ W, int32_t n_ro, int32_t n_co, const int32_t* __restrict__ row2req,
    const float* __restrict__ ZR, T* __restrict__ YC, T* __restrict__ OC) {
  extern __shared__ float sm[];
  const int32_t n = n_r + n_c;
  const int32_t ds = d + 1;          // padded row stride: rows land in different banks
  float* x = sm;                     // [n, d + 1]: request rows then candidate rows
  float* yc = sm + (size_t)n * ds;   // [n_c, n]
  const int64_t i = blockIdx.x;
  const int32_t r = row2req[i];
  for (int e = threadIdx.x; e < n_r * d; e += blockDim.x) x[(e / d) * ds + e % d] = ld_f(XR, (int64_t)r * n_r * d + e);
  for (int e = threadIdx.x; e < n_c * d; e += blockDim.x)
    x[(n_r + e / d) * ds + e % d] = ld_f(XC, i * n_c * d + e);
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_c * n; idx += blockDim.x) {
    const int a = idx / n, b = idx % n;
    const float* xa = x + (size_t)(n_r + a) * ds;
    const float* xb = x + (size_t)b * ds;
    float acc = 0.f;
    for (int e = 0; e < d; ++e) acc = fmaf(xa[e], xb[e], acc);
    yc[idx] = acc;
    if (YC) st_f(YC, i * n_c * n + idx, acc);
  }
  if (!W || !OC) return;
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_co * n; idx += blockDim.x) {
    const int o = idx / n, b = idx % n;
    float acc = 0.f;
    for (int a = 0; a < n_c; ++a) acc = fmaf(ld_f(W, (int64_t)(n_ro + o) * n + n_r + a), yc[a * n + b], acc);
    acc += ZR[((int64_t)r * n_co + o) * n + b];
    st_f(OC, (i * n_co + o) * n + b, acc);
  }
}

}  // namespace

rocs_status_t simt_linear(rocs_dtype_t dt, int64_t M, int32_t d_in, int32_t d_out, const void* X,
                          int64_t ld_x, const void* W, int64_t ld_w, const float* bias,
                          const float* add, int64_t ld_add, const int32_t* row2req, int act,
                          void* Y, int64_t ld_y, bool out_f32, cudaStream_t stream) {
  if (dt == ROCS_F32)
    return launch_linear<float, float>(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req,
                                       act, Y, ld_y, stream);
  if (out_f32)
    return launch_linear<__nv_bfloat16, float>(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add,
                                               row2req, act, Y, ld_y, stream);
  return launch_linear<__nv_bfloat16, __nv_bfloat16>(M, d_in, d_out, X, ld_x, W, ld_w, bias, add,
                                                     ld_add, row2req, act, Y, ld_y, stream);
}

rocs_status_t simt_dca(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_q, int32_t H, int32_t dh,
                       float scale, const void* Q, const void* K, const void* V,
                       const int32_t* seq_offsets, void* O, cudaStream_t stream) {
  if (dh > DCA_MAX_DH) return ROCS_ERR_UNSUPPORTED;
  const int64_t n_rows = plan->N * n_q;
  const int64_t items = n_rows * H;
  if (items == 0) return ROCS_OK;
  const int64_t blocks = (items + DCA_WARPS - 1) / DCA_WARPS;
  if (blocks > 0x7fffffffLL) return ROCS_ERR_UNSUPPORTED;
  if (dt == ROCS_F32)
    dca_simt_kernel<float><<<(unsigned)blocks, DCA_WARPS * 32, 0, stream>>>(
        n_rows, n_q, H, dh, scale, (const float*)Q, (const float*)K, (const float*)V, plan->row2req,
        seq_offsets, (float*)O);
  else
    dca_simt_kernel<__nv_bfloat16><<<(unsigned)blocks, DCA_WARPS * 32, 0, stream>>>(
        n_rows, n_q, H, dh, scale, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K,
        (const __nv_bfloat16*)V, plan->row2req, seq_offsets, (__nv_bfloat16*)O);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

template <typename T>
static rocs_status_t launch_glm(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d,
                                const void* XR, const void* XC, const void* W, int32_t n_ro,
                                int32_t n_co, void* YR, void* YC, void* OR_, void* OC, float* zr,
                                bool request_side, bool candidate_side, cudaStream_t stream) {
  const int32_t n = n_r + n_c;
  const size_t smem_r = ((size_t)n_r * (d + 1) + (size_t)n_r * n_r + (size_t)(n_ro + n_co) * n_r) * sizeof(float);
  const size_t smem_c = ((size_t)n * (d + 1) + (size_t)n_c * n) * sizeof(float);
  constexpr size_t kMaxSmem = 200 * 1024;
  if (smem_r > kMaxSmem || smem_c > kMaxSmem) return ROCS_ERR_UNSUPPORTED;
  if (request_side && plan->R > 0) {
    ROCS_CUDA_TRY(cudaFuncSetAttribute(glm_request_simt_kernel<T>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
    glm_request_simt_kernel<T><<<plan->R, 256, smem_r, stream>>>(
        n_r, n_c, d, (const T*)XR, (const T*)W, n_ro, n_co, (T*)YR, (T*)OR_, zr);
    ROCS_CUDA_TRY(cudaGetLastError());
  }
  if (candidate_side && plan->N > 0 && (YC || OC)) {
    ROCS_CUDA_TRY(cudaFuncSetAttribute(glm_candidate_simt_kernel<T>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
    glm_candidate_simt_kernel<T><<<(unsigned)plan->N, 128, smem_c, stream>>>(
        n_r, n_c, d, (const T*)XR, (const T*)XC, (const T*)W, n_ro, n_co, plan->row2req, zr, (T*)YC,
        (T*)OC);
    ROCS_CUDA_TRY(cudaGetLastError());
  }
  return ROCS_OK;
}

// YC == OC == nullptr runs only the request side (used in front of the tensor-core candidate
// kernel); XC == nullptr is then allowed.
rocs_status_t simt_glm(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d,
                       const void* XR, const void* XC, const void* W, int32_t n_ro, int32_t n_co,
                       void* YR, void* YC, void* OR_, void* OC, float* zr_workspace,
                       cudaStream_t stream) {
  if (dt == ROCS_F32)
    return launch_glm<float>(plan, n_r, n_c, d, XR, XC, W, n_ro, n_co, YR, YC, OR_, OC, zr_workspace,
                             true, true, stream);
  return launch_glm<__nv_bfloat16>(plan, n_r, n_c, d, XR, XC, W, n_ro, n_co, YR, YC, OR_, OC,
                                   zr_workspace, true, true, stream);
}

}  // namespace rocs
