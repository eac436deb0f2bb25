// Projected factorization machine for two groups: F = G P, G the masked interaction matrix of
// Eq. 9-10 and P [n_r + n_c, k] a projection of its column axis (the compression dimension k of an
// FM block).  With P = [P_R; P_C] the in-kernel-broadcast form (Section 4.1) is
//     T[r]  = X^R_r^T P_R                       [d, k]   once per request, fp32, in the workspace
//     FR[r] = X^R_r T[r]                        [n_r, k] once per request
//     FC[i] = X^C_i (T[m_i] + X^C_i^T P_C)      [n_c, k] per candidate
// so a candidate reads its own 2 n_c d bytes and nothing of the request but the d x k block T,
// which stays in registers while consecutive candidates belong to the same request.
//
// The candidate side is bound by HBM (about 30 flop per byte): the bf16 kernel streams candidate
// tiles through a TMA ring and gives every warp one candidate at a time, whose two small products
// (16 x d x 16 each) run on mma.sync m16n8k16 straight out of the swizzled tile:
//   step 1   H^T = T^T + P_C^T X^C_i    accumulators start at T^T (fp32); X^C_i is the K x N
//                                       operand, read with ldmatrix.trans
//   step 2   FC_i = X^C_i H             H rounded to bf16 once: the accumulator layout of step 1
//                                       is the B-operand layout of step 2, so it never leaves
//                                       registers; X^C_i is the M x K operand, read with ldmatrix
// A general kernel (any shape, fp32 or bf16 storage, fp32 FMA) covers everything else.
#include <algorithm>

#include "rocs_internal.h"
#include "simt_util.cuh"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

__device__ __forceinline__ float ld_f(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16* p, int64_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_f(float* p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_f(__nv_bfloat16* p, int64_t i, float v) { p[i] = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Request side, one block per request:  TT[r] = P_R^T X^R_r  ([k, d] fp32, the transpose of T)
// and FR[r] = X^R_r T[r].
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) fm_request_kernel(int32_t n_r, int32_t d, int32_t k, const T* __restrict__ XR,
                                                         const T* __restrict__ P, float* __restrict__ TT,
                                                         T* __restrict__ FR) {
  extern __shared__ float sm[];
  const int32_t ds = d + 1;           // padded row stride: rows land in different banks
  float* xr = sm;                     // [n_r, d + 1]
  float* tt = xr + (size_t)n_r * ds;  // [k, d + 1]
  float* pr = tt + (size_t)k * ds;    // [n_r, k]
  const int32_t r = blockIdx.x;
  // the candidate kernel may start now: it streams X^C on its own and waits for this grid only
  // before it reads TT
  ptx::griddep_launch_dependents();
  rows_to_shared(XR + (int64_t)r * n_r * d, xr, n_r, d, ds);
  for (int e = threadIdx.x; e < n_r * k; e += blockDim.x) pr[e] = ld_f(P, e);
  __syncthreads();
  // TT: one column e and up to eight projection columns c per work item, i.e. eight independent sums
  // per thread fed by one read of X^R per step
  constexpr int kCg = 8;
  const int n_cg = (k + kCg - 1) / kCg;
  for (int idx = threadIdx.x; idx < n_cg * d; idx += blockDim.x) {
    const int c0 = (idx / d) * kCg, e = idx % d;
    float acc[kCg];
#pragma unroll
    for (int u = 0; u < kCg; ++u) acc[u] = 0.f;
    for (int a = 0; a < n_r; ++a) {
      const float x = xr[a * ds + e];
#pragma unroll
      for (int u = 0; u < kCg; ++u) acc[u] = fmaf(pr[a * k + min(c0 + u, k - 1)], x, acc[u]);
    }
#pragma unroll
    for (int u = 0; u < kCg; ++u)
      if (c0 + u < k) {
        tt[(c0 + u) * ds + e] = acc[u];
        TT[((int64_t)r * k + c0 + u) * d + e] = acc[u];
      }
  }
  if (!FR) return;
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_r * k; idx += blockDim.x) {
    const int a = idx / k, c = idx % k;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};  // four chains over d, added in a fixed order
    int e = 0;
    for (; e + 3 < d; e += 4) {
#pragma unroll
      for (int u = 0; u < 4; ++u) acc[u] = fmaf(xr[a * ds + e + u], tt[c * ds + e + u], acc[u]);
    }
    for (; e < d; ++e) acc[0] = fmaf(xr[a * ds + e], tt[c * ds + e], acc[0]);
    st_f(FR, ((int64_t)r * n_r + a) * k + c, (acc[0] + acc[1]) + (acc[2] + acc[3]));
  }
}

// ---------------------------------------------------------------------------------------------
// Candidate side, general kernel: one block per candidate.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) fm_candidate_simt_kernel(int32_t n_r, int32_t n_c, int32_t d, int32_t k,
                                                                const T* __restrict__ XC, const T* __restrict__ P,
                                                                const int32_t* __restrict__ row2req,
                                                                const float* __restrict__ TT, T* __restrict__ FC) {
  extern __shared__ float sm[];
  const int32_t ds = d + 1;
  float* xc = sm;                     // [n_c, d + 1]
  float* ht = xc + (size_t)n_c * ds;  // [k, d + 1]
  float* pc = ht + (size_t)k * ds;    // [n_c, k]
  const int64_t i = blockIdx.x;
  const int32_t r = row2req[i];
  for (int e = threadIdx.x; e < n_c * d; e += blockDim.x) xc[(e / d) * ds + e % d] = ld_f(XC, i * n_c * d + e);
  for (int e = threadIdx.x; e < n_c * k; e += blockDim.x) pc[e] = ld_f(P, (int64_t)n_r * k + e);
  __syncthreads();
  for (int idx = threadIdx.x; idx < k * d; idx += blockDim.x) {
    const int c = idx / d, e = idx % d;
    float acc = TT[((int64_t)r * k + c) * d + e];
    for (int a = 0; a < n_c; ++a) acc = fmaf(pc[a * k + c], xc[a * ds + e], acc);
    ht[c * ds + e] = acc;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_c * k; idx += blockDim.x) {
    const int a = idx / k, c = idx % k;
    float acc = 0.f;
    for (int e = 0; e < d; ++e) acc = fmaf(xc[a * ds + e], ht[c * ds + e], acc);
    st_f(FC, (i * n_c + a) * k + c, acc);
  }
}

// ---------------------------------------------------------------------------------------------
// Candidate side, bf16 streaming kernel: n_c = 16, k in {8, 16}, d a multiple of 64 up to 256.
// ---------------------------------------------------------------------------------------------
constexpr int kNc = 16;            // rows per candidate
constexpr int kTileCands = 8;      // candidates per tile = compute warps per CTA
constexpr int kTileRows = kNc * kTileCands;  // 128
constexpr int kFmThreads = (kTileCands + 1) * 32;
constexpr int kSlabBytes = kTileRows * 128;  // 64 columns of the tile, 128-byte swizzled rows
constexpr uint32_t kStatusFm = 0x600;

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// ---------------------------------------------------------------------------------------------
// Request side on warp-level tensor cores (bf16; k and d multiples of 8 and 16): the same two products
// as fm_request_kernel out of bf16 copies of X^R_r and P_R in shared memory.
//   TT[c][e] = sum_a P_R[a][c] X^R[a][e]   A = P_R^T and B = X^R, both read with ldmatrix.trans
//   FR[a][c] = sum_e X^R[a][e] TT[c][e]    A = X^R rows, B = rows of TT: TT enters as a bf16 pair
//                                          (value rounded to bf16 + the rounded remainder), two products,
//                                          so FR keeps fp32-level accuracy (relative error 2^-17)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}

__global__ void __launch_bounds__(256) fm_request_mma_kernel(int32_t n_r, int32_t d, int32_t k,
                                                             const __nv_bfloat16* __restrict__ XR,
                                                             const __nv_bfloat16* __restrict__ P, float* __restrict__ TT,
                                                             __nv_bfloat16* __restrict__ FR) {
  extern __shared__ __align__(16) uint8_t smem_fmr[];
  const int32_t n_rp = (n_r + 15) / 16 * 16, kp = (k + 15) / 16 * 16;
  const int32_t x_row = (d + 8) * 2, p_row = (kp + 8) * 2;  // bytes; 16 mod 32: ldmatrix without bank conflicts
  uint8_t* xb = smem_fmr;                    // [n_rp][d + 8] bf16, padding rows zero
  uint8_t* pb = xb + (size_t)n_rp * x_row;   // [n_rp][kp + 8] bf16, padding rows and columns zero
  uint8_t* th = pb + (size_t)n_rp * p_row;   // [kp][d + 8] bf16: TT rounded
  uint8_t* tl = th + (size_t)kp * x_row;     // [kp][d + 8] bf16: what the rounding left
  const int32_t r = blockIdx.x;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  ptx::griddep_launch_dependents();

  const int32_t vpr = d / 8, n_vec = n_r * vpr;
  const uint4* src = reinterpret_cast<const uint4*>(XR + (int64_t)r * n_r * d);
  for (int32_t base = threadIdx.x; base < n_vec; base += 4 * 256) {
    uint4 raw[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (base + u * 256 < n_vec) raw[u] = __ldg(src + base + u * 256);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int32_t v = base + u * 256;
      if (v < n_vec) *reinterpret_cast<uint4*>(xb + (v / vpr) * x_row + (v % vpr) * 16) = raw[u];
    }
  }
  for (int32_t v = n_vec + threadIdx.x; v < n_rp * vpr; v += 256)
    *reinterpret_cast<uint4*>(xb + (v / vpr) * x_row + (v % vpr) * 16) = make_uint4(0u, 0u, 0u, 0u);
  for (int32_t e = threadIdx.x; e < n_rp * kp; e += 256) {
    const int32_t a = e / kp, c = e % kp;
    reinterpret_cast<__nv_bfloat16*>(pb + a * p_row)[c] = (a < n_r && c < k) ? P[a * k + c] : __float2bfloat16_rn(0.f);
  }
  __syncthreads();

  const uint32_t xb_a = smem_u32(xb), pb_a = smem_u32(pb), th_a = smem_u32(th), tl_a = smem_u32(tl);
  const int g8 = lane / 4, t4 = lane % 4;
  const int lr = lane & 7, lq = lane >> 3;  // row inside an 8x8 block, which of the four blocks
  // ---- TT: 16 projection columns (one M tile per 16 of kp) x pairs of 8-wide column tiles of d
  const int32_t n_pairs = d / 16;
  for (int32_t t = warp; t < (kp / 16) * n_pairs; t += 8) {
    const int32_t c0 = (t / n_pairs) * 16, e0 = (t % n_pairs) * 16;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    for (int32_t a0 = 0; a0 < n_rp; a0 += 16) {
      uint32_t fa[4], fb[4];
      // A = P_R^T: blocks (c lo, a lo), (c hi, a lo), (c lo, a hi), (c hi, a hi) of the transposed tile
      ldmatrix_x4_trans(pb_a + (a0 + lr + (lq >> 1) * 8) * p_row + (c0 + (lq & 1) * 8) * 2, fa);
      // B = X^R: blocks (a lo, e lo), (a hi, e lo), (a lo, e hi), (a hi, e hi)
      ldmatrix_x4_trans(xb_a + (a0 + lr + (lq & 1) * 8) * x_row + (e0 + (lq >> 1) * 8) * 2, fb);
      mma_bf16(acc[0], fa, fb[0], fb[1]);
      mma_bf16(acc[1], fa, fb[2], fb[3]);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int32_t c = c0 + g8 + j * 8, e = e0 + h * 8 + 2 * t4;
        const float v0 = acc[h][2 * j], v1 = acc[h][2 * j + 1];
        if (c < k) *reinterpret_cast<float2*>(TT + ((int64_t)r * k + c) * d + e) = make_float2(v0, v1);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(v0, v1);
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v0 - __low2float(hi), v1 - __high2float(hi));
        *reinterpret_cast<__nv_bfloat162*>(th + c * x_row + e * 2) = hi;
        *reinterpret_cast<__nv_bfloat162*>(tl + c * x_row + e * 2) = lo;
      }
  }
  if (!FR) return;
  __syncthreads();
  // ---- FR: 16 x 8 tiles over (a, c)
  const int32_t n_ct = kp / 8;
  for (int32_t t = warp; t < (n_rp / 16) * n_ct; t += 8) {
    const int32_t a0 = (t / n_ct) * 16, c0 = (t % n_ct) * 8;
    const uint32_t a_addr = xb_a + (a0 + lr + (lq & 1) * 8) * x_row + (lq >> 1) * 16;
    const uint32_t b_off = (c0 + lr) * x_row + (lq & 1) * 16;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int32_t e0 = 0; e0 < d; e0 += 16) {
      uint32_t fa[4], bh[2], bl[2];
      ldmatrix_x4(a_addr + e0 * 2, fa);
      ldmatrix_x2(th_a + b_off + e0 * 2, bh);
      ldmatrix_x2(tl_a + b_off + e0 * 2, bl);
      mma_bf16(acc, fa, bh[0], bh[1]);
      mma_bf16(acc, fa, bl[0], bl[1]);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int32_t a = a0 + g8 + h * 8, c = c0 + 2 * t4;
      if (a < n_r) {
        if (c < k) FR[((int64_t)r * n_r + a) * k + c] = __float2bfloat16_rn(acc[2 * h]);
        if (c + 1 < k) FR[((int64_t)r * n_r + a) * k + c + 1] = __float2bfloat16_rn(acc[2 * h + 1]);
      }
    }
  }
}

struct FmParams {
  int64_t N;
  int32_t n_r, k, num_tiles;
  const __nv_bfloat16* P;        // [n_r + 16, k]
  const int32_t* row2req;        // [N]
  const float* TT;               // [R, k, d]
  __nv_bfloat16* FC;             // [N, 16, k]
  uint32_t* status;
};

template <int D, int STAGES>
__global__ void __launch_bounds__(kFmThreads, 1)
fm_candidate_mma_kernel(const __grid_constant__ CUtensorMap map_xc, const FmParams p) {
  constexpr int kSlabs = D / 64;
  constexpr int kStageBytes = kSlabs * kSlabBytes;
  constexpr int kPairs = D / 16;  // pairs of 8-column groups = k-steps of step 2
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * kStageBytes);
  uint64_t* empty = full + STAGES;
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(empty + STAGES);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles assume a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.status, 0u, kStatusFm | 15);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kTileCands);
    }
    abort_flag->v = 0;
    fence_mbar_init();
  }
  __syncthreads();
  // a contiguous run of tiles per CTA: consecutive candidates mostly share their request, so the
  // request's T block is reloaded only where a segment ends
  const int32_t tiles_per_cta = (p.num_tiles + (int32_t)gridDim.x - 1) / (int32_t)gridDim.x;
  const int32_t tile_begin = min((int32_t)blockIdx.x * tiles_per_cta, p.num_tiles);
  const int32_t tile_end = min(tile_begin + tiles_per_cta, p.num_tiles);

  if (warp == kTileCands) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_xc);
      uint32_t it = 0;
      for (int32_t t = tile_begin; t < tile_end; ++t, ++it) {
        const int s = it % STAGES;
        if (!mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1, abort_flag, p.status, kStatusFm | 1)) break;
        mbar_expect_tx(&full[s], kStageBytes);
#pragma unroll
        for (int sl = 0; sl < kSlabs; ++sl)
          tma_load_2d(smem + s * kStageBytes + sl * kSlabBytes, &map_xc, &full[s], sl * 64, t * kTileRows);
      }
      // loads in flight land in this CTA's shared memory: wait for them before the CTA may exit
      for (int s = 0; s < STAGES; ++s) {
        const uint32_t n_issued = it / STAGES + (((int)(it % STAGES) > s) ? 1 : 0);
        if (n_issued == 0) continue;
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(&full[s], (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else {
    // ------------------------------ one candidate per warp ---------------------------------
    const int g = lane / 4, tq = lane % 4;  // fragment row group and column pair
    // P_C^T as the M x K operand of step 1: A[m = projection column][kk = candidate row]
    uint32_t pa[4];
    {
      const __nv_bfloat16* pc = p.P + (int64_t)p.n_r * p.k;
      auto at = [&](int row, int col) -> float {  // P_C[row][col], zero beyond k columns
        return col < p.k ? __bfloat162float(pc[row * p.k + col]) : 0.f;
      };
      pa[0] = pack_bf16(at(2 * tq, g), at(2 * tq + 1, g));
      pa[1] = pack_bf16(at(2 * tq, g + 8), at(2 * tq + 1, g + 8));
      pa[2] = pack_bf16(at(2 * tq + 8, g), at(2 * tq + 9, g));
      pa[3] = pack_bf16(at(2 * tq + 8, g + 8), at(2 * tq + 9, g + 8));
    }
    // this lane's address pattern inside a candidate's 16 rows: row, and which of the two
    // 8-column groups of a pair
    const int lrow = (lane % 8) + ((lane / 8) % 2) * 8;
    const int lsel = lane / 16;
    float tfrag[kPairs][2][4];  // T^T of the cached request in step-1 accumulator layout
    int32_t cached_req = -1;
    uint32_t it = 0;
    // the request of this warp's candidate, fetched one tile ahead of its use (the load would
    // otherwise sit on every candidate's critical path)
    int32_t r_next = 0;
    if (tile_begin < tile_end && (int64_t)tile_begin * kTileCands + warp < p.N)
      r_next = p.row2req[(int64_t)tile_begin * kTileCands + warp];
    for (int32_t t = tile_begin; t < tile_end; ++t, ++it) {
      const int s = it % STAGES;
      const int32_t r = r_next;
      {
        const int64_t cand_next = (int64_t)(t + 1) * kTileCands + warp;
        if (t + 1 < tile_end && cand_next < p.N) r_next = p.row2req[cand_next];
      }
      if (!mbar_wait(&full[s], (it / STAGES) & 1, abort_flag, p.status, kStatusFm | 2)) break;
      const int64_t cand = (int64_t)t * kTileCands + warp;
      if (cand < p.N) {
        if (r != cached_req) {
          if (cached_req < 0) griddep_wait();  // TT comes from the request kernel launched just before
          cached_req = r;
          const float* tt = p.TT + (int64_t)r * p.k * D;
#pragma unroll
          for (int cp = 0; cp < kPairs; ++cp)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int col = (2 * cp + h) * 8 + 2 * tq;
              const float2 lo = g < p.k ? *reinterpret_cast<const float2*>(tt + g * D + col) : make_float2(0.f, 0.f);
              const float2 hi = g + 8 < p.k ? *reinterpret_cast<const float2*>(tt + (g + 8) * D + col) : make_float2(0.f, 0.f);
              tfrag[cp][h][0] = lo.x;
              tfrag[cp][h][1] = lo.y;
              tfrag[cp][h][2] = hi.x;
              tfrag[cp][h][3] = hi.y;
            }
        }
        const uint32_t tile = smem_u32(smem + s * kStageBytes);
        const int trow = warp * kNc + lrow;
        // step 1: H^T (16 x D) = T^T + P_C^T X^C, rounded to bf16 as the K x N operand of step 2
        uint32_t hb[kPairs][2][2];  // [k-step][projection columns 0-7 | 8-15][b0, b1]
#pragma unroll
        for (int cp = 0; cp < kPairs; ++cp) {
          const int chunk = 2 * cp + lsel;  // 16-byte chunk along d
          uint32_t xb[4];
          ldmatrix_x4_trans(tile + (chunk / 8) * kSlabBytes + trow * 128 + (((chunk % 8) ^ (trow & 7)) << 4), xb);
          float acc0[4], acc1[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            acc0[e] = tfrag[cp][0][e];
            acc1[e] = tfrag[cp][1][e];
          }
          mma_bf16(acc0, pa, xb[0], xb[1]);
          mma_bf16(acc1, pa, xb[2], xb[3]);
          hb[cp][0][0] = pack_bf16(acc0[0], acc0[1]);
          hb[cp][0][1] = pack_bf16(acc1[0], acc1[1]);
          hb[cp][1][0] = pack_bf16(acc0[2], acc0[3]);
          hb[cp][1][1] = pack_bf16(acc1[2], acc1[3]);
        }
        // step 2: FC (16 x 16) = X^C H
        float out0[4] = {0.f, 0.f, 0.f, 0.f}, out1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int cp = 0; cp < kPairs; ++cp) {
          const int chunk = 2 * cp + lsel;
          uint32_t xa[4];
          ldmatrix_x4(tile + (chunk / 8) * kSlabBytes + trow * 128 + (((chunk % 8) ^ (trow & 7)) << 4), xa);
          mma_bf16(out0, xa, hb[cp][0][0], hb[cp][0][1]);
          mma_bf16(out1, xa, hb[cp][1][0], hb[cp][1][1]);
        }
        __nv_bfloat16* fc = p.FC + cand * kNc * p.k;
        *reinterpret_cast<uint32_t*>(fc + g * p.k + 2 * tq) = pack_bf16(out0[0], out0[1]);
        *reinterpret_cast<uint32_t*>(fc + (g + 8) * p.k + 2 * tq) = pack_bf16(out0[2], out0[3]);
        if (p.k > 8) {
          *reinterpret_cast<uint32_t*>(fc + g * p.k + 8 + 2 * tq) = pack_bf16(out1[0], out1[1]);
          *reinterpret_cast<uint32_t*>(fc + (g + 8) * p.k + 8 + 2 * tq) = pack_bf16(out1[2], out1[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
  }
}

int sm_count_fm() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

template <int D>
rocs_status_t launch_fm_mma(const rocs_plan* plan, int32_t n_r, int32_t k, const void* XC, const void* P,
                            const float* TT, void* FC, cudaStream_t stream) {
  constexpr int kStages = D <= 64 ? 8 : D <= 128 ? 6 : 3;
  constexpr int kSmem = kStages * (D / 64) * kSlabBytes + 512;
  CUtensorMap map_xc;
  if (!make_tensor_map_2d(&map_xc, XC, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)plan->N * kNc, D, D, kTileRows, 64,
                          true))
    return ROCS_ERR_CUDA;
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  FmParams p{};
  p.N = plan->N;
  p.n_r = n_r;
  p.k = k;
  p.num_tiles = (int32_t)((plan->N + kTileCands - 1) / kTileCands);
  p.P = (const __nv_bfloat16*)P;
  p.row2req = plan->row2req;
  p.TT = TT;
  p.FC = (__nv_bfloat16*)FC;
  p.status = status;
  auto kern = fm_candidate_mma_kernel<D, kStages>;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
  // Launched so that it may overlap the request kernel in front of it on the stream (that kernel
  // releases its dependents at once); nothing else this kernel reads is written by that launch.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::min(p.num_tiles, sm_count_fm()));
  cfg.blockDim = dim3(kFmThreads);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, map_xc, p));
  return ROCS_OK;
}

template <typename T>
rocs_status_t launch_fm(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, int32_t k, const void* XR,
                        const void* XC, const void* P, void* FR, void* FC, float* TT, bool fast_candidates,
                        bool tensor_core_request, cudaStream_t stream) {
  constexpr size_t kMaxSmem = 200 * 1024;
  const size_t smem_r = ((size_t)(n_r + k) * (d + 1) + (size_t)n_r * k) * sizeof(float);
  const size_t smem_c = ((size_t)(n_c + k) * (d + 1) + (size_t)n_c * k) * sizeof(float);
  if (smem_r > kMaxSmem || smem_c > kMaxSmem) return ROCS_ERR_UNSUPPORTED;
  const size_t n_rp = (size_t)(n_r + 15) / 16 * 16, kp = (size_t)(k + 15) / 16 * 16;
  const size_t smem_mma = n_rp * ((size_t)(d + 8) * 2 + (kp + 8) * 2) + 2 * kp * (size_t)(d + 8) * 2;
  if (plan->R > 0 && tensor_core_request && sizeof(T) == 2 && d % 16 == 0 && k % 8 == 0 && smem_mma <= kMaxSmem) {
    ROCS_CUDA_TRY(cudaFuncSetAttribute(fm_request_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_mma));
    fm_request_mma_kernel<<<plan->R, 256, smem_mma, stream>>>(n_r, d, k, (const __nv_bfloat16*)XR,
                                                              (const __nv_bfloat16*)P, TT, (__nv_bfloat16*)FR);
    ROCS_CUDA_TRY(cudaGetLastError());
  } else if (plan->R > 0) {
    ROCS_CUDA_TRY(cudaFuncSetAttribute(fm_request_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
    fm_request_kernel<T><<<plan->R, 256, smem_r, stream>>>(n_r, d, k, (const T*)XR, (const T*)P, TT, (T*)FR);
    ROCS_CUDA_TRY(cudaGetLastError());
  }
  if (plan->N == 0 || !FC) return ROCS_OK;
  if (fast_candidates) {
    switch (d) {
      case 64: return launch_fm_mma<64>(plan, n_r, k, XC, P, TT, FC, stream);
      case 128: return launch_fm_mma<128>(plan, n_r, k, XC, P, TT, FC, stream);
      case 192: return launch_fm_mma<192>(plan, n_r, k, XC, P, TT, FC, stream);
      case 256: return launch_fm_mma<256>(plan, n_r, k, XC, P, TT, FC, stream);
      default: break;
    }
  }
  ROCS_CUDA_TRY(cudaFuncSetAttribute(fm_candidate_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
  fm_candidate_simt_kernel<T><<<(unsigned)plan->N, 128, smem_c, stream>>>(n_r, n_c, d, k, (const T*)XC, (const T*)P,
                                                                         plan->row2req, TT, (T*)FC);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace

bool fm_projection_fast_supported(int32_t n_c, int32_t d, int32_t k) {
  return n_c == kNc && (k == 8 || k == 16) && d % 64 == 0 && d >= 64 && d <= 256;
}

rocs_status_t fm_projection(rocs_dtype_t dt, const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, int32_t k,
                            const void* XR, const void* XC, const void* P, void* FR, void* FC, float* tt_workspace,
                            bool allow_fast, cudaStream_t stream) {
  if (dt == ROCS_F32)
    return launch_fm<float>(plan, n_r, n_c, d, k, XR, XC, P, FR, FC, tt_workspace, false, false, stream);
  return launch_fm<__nv_bfloat16>(plan, n_r, n_c, d, k, XR, XC, P, FR, FC, tt_workspace,
                                  allow_fast && fm_projection_fast_supported(n_c, d, k), allow_fast, stream);
}

}  // namespace rocs
