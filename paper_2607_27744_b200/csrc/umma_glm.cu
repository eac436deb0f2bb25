// GLM factorization machine, candidate rows (Eq. 10, bottom row), with the optional row-axis
// compression (Eq. 6) fused in:
//     YC[i] = [ X^C_i X^R_r^T , X^C_i X^C_i^T ]        r = request of candidate i
//     OC[i] = ZR[r] + W_CC YC[i]                       ZR[r] = W_CR YR[r], once per request (fp32)
// The request operand X^R_r is loaded on demand next to the candidate tile; it is never
// replicated per candidate (the in-kernel broadcast of Section 4 applied to Eq. 9-10).
//
// Tile = 128 / n_c consecutive candidates of ONE request = 128 rows of X^C (tiles never cross a
// request).  Shared memory holds, per 64-wide slice of d, the rows [X^R_r (padded to 16) ; X^C tile]
// back to back, so a single tcgen05.mma per 16-deep K step computes
//     D[128, n_r_pad + 128] = X^C_tile * [X^R_r ; X^C_tile]^T
// whose first n_r columns are the request-candidate block and whose 128 x 128 tail holds each
// candidate's own n_c x n_c block on the diagonal (the off-diagonal products are discarded: the
// kernel is bound by reading X^C from HBM, the tensor pipe has slack).
//
// Persistent CTA, 10 warps: warp 0 TMA producer, warp 1 MMA issuer, two epilogue groups of four
// warps that alternate tiles (each owns one TMEM accumulator and one staging area), so one group
// drains and compresses a tile while the tensor pipe fills the other accumulator.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr int kGroupThreads = 128;
constexpr uint32_t kStatusGlm = 0x200;
constexpr int kAccStride = 256;  // TMEM columns per accumulator

struct GlmParams {
  const Tile* tiles;
  int32_t num_tiles;
  int32_t n_r, n_r_pad, n_c, d, n_ro, n_co;
  int32_t stages, stage_bytes, group_staging_bytes, yc_stride;
  const __nv_bfloat16* W;  // [n_ro + n_co, n] or null
  const float* ZR;         // [R, n_co, n] or null
  __nv_bfloat16* YC;       // [N, n_c, n] or null
  __nv_bfloat16* OC;       // [N, n_co, n] or null
  uint32_t* status;
};

__device__ __forceinline__ void group_sync(int g) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(kGroupThreads) : "memory");
}

template <int NC>
__global__ void __launch_bounds__(kThreads, 1)
glm_umma_kernel(const __grid_constant__ CUtensorMap map_xr, const __grid_constant__ CUtensorMap map_xc,
                const GlmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + p.stages * p.stage_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(staging + 2 * p.group_staging_bytes);
  uint64_t* empty = full + 8;
  uint64_t* tmem_full = empty + 8;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* drain = tmem_empty + 2;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int32_t n = p.n_r + p.n_c;
  const int32_t k_slices = p.d / 64;
  const int32_t slice_bytes = (p.n_r_pad + 128) * 128;
  const int32_t xr_bytes = p.n_r_pad * 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], 4);
    }
    mbar_init(drain, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_ptr, 2 * kAccStride);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_xr);
      prefetch_tensormap(&map_xc);
      uint32_t it = 0;
      bool ok = true;
      for (int32_t t = blockIdx.x; t < p.num_tiles; t += gridDim.x, ++it) {
        const Tile tile = p.tiles[t];
        const int s = it % p.stages;
        if (!mbar_wait(&empty[s], ((it / p.stages) & 1) ^ 1, abort_flag, p.status, kStatusGlm | 1)) { ok = false; break; }
        uint8_t* st = smem + s * p.stage_bytes;
        mbar_expect_tx(&full[s], p.stage_bytes);
        for (int32_t ks = 0; ks < k_slices; ++ks) {
          tma_load_2d(st + ks * slice_bytes, &map_xr, &full[s], ks * 64, tile.req * p.n_r);
          tma_load_2d(st + ks * slice_bytes + xr_bytes, &map_xc, &full[s], ks * 64, tile.cand0 * NC);
        }
      }
      if (!ok) {
        for (int s = 0; s < p.stages; ++s) {
          const uint32_t n_issued = it / p.stages + (((int)(it % p.stages) > s) ? 1 : 0);
          if (n_issued == 0) continue;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ---------------------------------------------
    const uint32_t idesc = umma_idesc_bf16(128, (uint32_t)(p.n_r_pad + 128), false, false);
    uint32_t it = 0;
    bool ok = true;
    for (int32_t t = blockIdx.x; t < p.num_tiles; t += gridDim.x, ++it) {
      const uint32_t acc = it & 1;
      const int s = it % p.stages;
      if (!mbar_wait(&tmem_empty[acc], ((it >> 1) & 1) ^ 1, abort_flag, p.status, kStatusGlm | 2)) { ok = false; break; }
      if (!mbar_wait(&full[s], (it / p.stages) & 1, abort_flag, p.status, kStatusGlm | 3)) { ok = false; break; }
      tc_fence_after_sync();
      if (lane == 0) {
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        const uint32_t st = smem_u32(smem + s * p.stage_bytes);
        for (int32_t ks = 0; ks < k_slices; ++ks) {
          const uint64_t b_desc = smem_desc_sw128(st + ks * slice_bytes, 1024, 16);             // [X^R ; X^C]
          const uint64_t a_desc = smem_desc_sw128(st + ks * slice_bytes + xr_bytes, 1024, 16);  // X^C
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (ks | k) != 0 ? 1u : 0u);
        }
        umma_commit(&empty[s]);
        umma_commit(&tmem_full[acc]);
      }
      __syncwarp();
    }
    if (!ok && lane == 0) {
      umma_commit(drain);
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(drain, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ------------------------------ epilogue groups ----------------------------------------
    const int g = (warp - 2) / 4;         // group 0: warps 2-5, group 1: warps 6-9
    const int q = warp % 4;               // TMEM lane quadrant
    const int gt = (warp - 2) % 4 * 32 + lane;  // thread index inside the group, 0..127
    const int row = q * 32 + lane;        // tile row = TMEM lane
    float* yc = reinterpret_cast<float*>(staging + g * p.group_staging_bytes);  // [128][yc_stride]
    float* wcc = yc + 128 * p.yc_stride;                                         // [n_c][n_co]
    __nv_bfloat16* oc_s = reinterpret_cast<__nv_bfloat16*>(wcc + ((NC * p.n_co + 3) & ~3));  // [cands][n_co][n]
    const bool compress = p.W != nullptr && p.OC != nullptr;
    if (compress) {
      // W_CC, transposed to [a][o] so that one broadcast 16-byte load fetches four outputs.
      for (int e = gt; e < NC * p.n_co; e += kGroupThreads) {
        const int a = e / p.n_co, o = e % p.n_co;
        wcc[e] = __bfloat162float(p.W[(int64_t)(p.n_ro + o) * n + p.n_r + a]);
      }
    }
    group_sync(g);
    uint32_t it = 0;
    for (int32_t t = blockIdx.x; t < p.num_tiles; t += gridDim.x, ++it) {
      if ((int)(it & 1) != g) continue;
      const Tile tile = p.tiles[t];
      if (!mbar_wait(&tmem_full[g], (it >> 1) & 1, abort_flag, p.status, kStatusGlm | 4)) break;
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + g * kAccStride + ((uint32_t)(q * 32) << 16);
      float* my = yc + row * p.yc_stride;
      // request-candidate block: columns 0 .. n_r-1
      for (int32_t c0 = 0; c0 < p.n_r; c0 += 16) {
        uint32_t v[16];
        tmem_ld_32x32b_x16(t_row + c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < p.n_r) my[c0 + j] = __uint_as_float(v[j]);
      }
      // candidate-candidate block: the 32 x 32 diagonal block of this warp's rows, of which each
      // thread keeps the NC columns of its own candidate
      {
        uint32_t v[32];
        tmem_ld_32x32b_x32(t_row + p.n_r_pad + q * 32, v);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty[g]);
        const int sub = lane / NC;  // which candidate of the warp's 32 / NC this row belongs to
#pragma unroll
        for (int j = 0; j < NC; ++j) {
          uint32_t x = v[j];
#pragma unroll
          for (int s2 = 1; s2 < 32 / NC; ++s2) x = (sub == s2) ? v[s2 * NC + j] : x;
          my[p.n_r + j] = __uint_as_float(x);
        }
      }
      group_sync(g);
      const int32_t rows_valid = tile.count * NC;
      if (p.YC != nullptr) {
        // raw block, bf16, 8 values (16 bytes) per store; rows of the tile are contiguous in YC
        __nv_bfloat16* dst = p.YC + (int64_t)tile.cand0 * NC * n;
        const int32_t vecs = rows_valid * n / 8;
        for (int32_t e = gt; e < vecs; e += kGroupThreads) {
          const int32_t r0 = (e * 8) / n, c0 = (e * 8) % n;
          const float* src = yc + r0 * p.yc_stride + c0;
          uint4 w;
          __nv_bfloat162 h;
          h = __floats2bfloat162_rn(src[0], src[1]); w.x = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(src[2], src[3]); w.y = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(src[4], src[5]); w.z = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(src[6], src[7]); w.w = *reinterpret_cast<uint32_t*>(&h);
          *reinterpret_cast<uint4*>(dst + (int64_t)e * 8) = w;
        }
      }
      if (compress) {
        // OC[c][o][b] = ZR[r][o][b] + sum_a W_CC[o][a] YC[c][a][b]; a thread owns up to four (c, b)
        // pairs at a time and all outputs o of them, four outputs per pass.
        const float* zr = p.ZR + (int64_t)tile.req * p.n_co * n;
        const int32_t pairs = tile.count * n;
        for (int32_t e0 = 0; e0 < pairs; e0 += 4 * kGroupThreads) {
          int32_t c[4], b[4];
          bool on[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int32_t e = e0 + u * kGroupThreads + gt;
            on[u] = e < pairs;
            c[u] = on[u] ? e / n : 0;
            b[u] = on[u] ? e % n : 0;
          }
          for (int32_t o0 = 0; o0 < p.n_co; o0 += 4) {
            float acc[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
              for (int oo = 0; oo < 4; ++oo)
                acc[u][oo] = (on[u] && o0 + oo < p.n_co) ? __ldg(zr + (o0 + oo) * n + b[u]) : 0.f;
#pragma unroll
            for (int a = 0; a < NC; ++a) {
              float w[4];
#pragma unroll
              for (int oo = 0; oo < 4; ++oo) w[oo] = (o0 + oo < p.n_co) ? wcc[a * p.n_co + o0 + oo] : 0.f;
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                const float y = yc[(c[u] * NC + a) * p.yc_stride + b[u]];
#pragma unroll
                for (int oo = 0; oo < 4; ++oo) acc[u][oo] = fmaf(w[oo], y, acc[u][oo]);
              }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
              for (int oo = 0; oo < 4; ++oo)
                if (on[u] && o0 + oo < p.n_co)
                  oc_s[(c[u] * p.n_co + o0 + oo) * n + b[u]] = __float2bfloat16_rn(acc[u][oo]);
          }
        }
        group_sync(g);
        const uint4* src = reinterpret_cast<const uint4*>(oc_s);
        uint4* dst = reinterpret_cast<uint4*>(p.OC + (int64_t)tile.cand0 * p.n_co * n);
        const int32_t vecs = tile.count * p.n_co * n / 8;
        for (int32_t e = gt; e < vecs; e += kGroupThreads) dst[e] = src[e];
      }
      group_sync(g);  // staging is reused by this group's next tile
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * kAccStride);
  }
}

int sm_count_glm() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

constexpr int kMaxSmem = 227 * 1024;

struct GlmLayout {
  int32_t n_r_pad, stage_bytes, group_staging_bytes, yc_stride, stages, smem_bytes;
  bool ok;
};

GlmLayout glm_layout(int32_t n_r, int32_t n_c, int32_t d, int32_t n_co) {
  GlmLayout L{};
  const int32_t n = n_r + n_c;
  L.n_r_pad = (n_r + 15) / 16 * 16;
  L.stage_bytes = (L.n_r_pad + 128) * d * 2;
  L.yc_stride = n | 1;  // odd stride: row-per-thread writes hit distinct banks
  const int32_t cands = 128 / n_c;
  int32_t gs = 128 * L.yc_stride * 4 + ((n_c * n_co + 3) & ~3) * 4 + cands * n_co * n * 2;
  L.group_staging_bytes = (gs + 127) & ~127;
  const int32_t fixed = 2 * L.group_staging_bytes + 512 + 1024;
  L.stages = std::min(6, (kMaxSmem - fixed) / L.stage_bytes);
  L.smem_bytes = L.stages * L.stage_bytes + fixed;
  L.ok = L.stages >= 2;
  return L;
}

}  // namespace

bool umma_glm_supported(int32_t n_r, int32_t n_c, int32_t d, int32_t n_ro, int32_t n_co) {
  (void)n_ro;
  if (n_c != 8 && n_c != 16 && n_c != 32) return false;
  if (n_r < 1 || n_r > 128) return false;
  if (d % 64 != 0 || d < 64 || d > 256) return false;
  if ((n_r + n_c) % 8 != 0) return false;
  return glm_layout(n_r, n_c, d, n_co).ok;
}

rocs_status_t umma_glm(const rocs_plan* plan, int32_t n_r, int32_t n_c, int32_t d, const void* XR,
                       const void* XC, const void* W, int32_t n_ro, int32_t n_co, void* YC, void* OC,
                       const float* zr_workspace, cudaStream_t stream) {
  if (plan->N == 0) return ROCS_OK;
  TileList tl;
  rocs_status_t st = plan_tiles(plan, 128 / n_c, stream, &tl);
  if (st != ROCS_OK) return st;
  if (tl.num == 0) return ROCS_OK;
  const GlmLayout L = glm_layout(n_r, n_c, d, n_co);
  CUtensorMap map_xr, map_xc;
  if (!make_tensor_map_2d(&map_xr, XR, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)plan->R * n_r, (uint64_t)d,
                          (uint64_t)d, (uint32_t)L.n_r_pad, 64, true) ||
      !make_tensor_map_2d(&map_xc, XC, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)plan->N * n_c, (uint64_t)d,
                          (uint64_t)d, 128, 64, true))
    return ROCS_ERR_CUDA;
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  GlmParams p{};
  p.tiles = tl.dev;
  p.num_tiles = tl.num;
  p.n_r = n_r; p.n_r_pad = L.n_r_pad; p.n_c = n_c; p.d = d; p.n_ro = n_ro; p.n_co = n_co;
  p.stages = L.stages; p.stage_bytes = L.stage_bytes; p.group_staging_bytes = L.group_staging_bytes;
  p.yc_stride = L.yc_stride;
  p.W = (const __nv_bfloat16*)W; p.ZR = zr_workspace;
  p.YC = (__nv_bfloat16*)YC; p.OC = (__nv_bfloat16*)OC;
  p.status = status;
  const int grid = std::min(tl.num, sm_count_glm());
#define ROCS_GLM_LAUNCH(NC_)                                                                                  \
  do {                                                                                                        \
    ROCS_CUDA_TRY(cudaFuncSetAttribute(glm_umma_kernel<NC_>, cudaFuncAttributeMaxDynamicSharedMemorySize,     \
                                       L.smem_bytes));                                                        \
    glm_umma_kernel<NC_><<<grid, kThreads, L.smem_bytes, stream>>>(map_xr, map_xc, p);                        \
  } while (0)
  if (n_c == 8) ROCS_GLM_LAUNCH(8);
  else if (n_c == 16) ROCS_GLM_LAUNCH(16);
  else ROCS_GLM_LAUNCH(32);
#undef ROCS_GLM_LAUNCH
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
