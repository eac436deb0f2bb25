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
// warps that alternate tiles (each owns one TMEM accumulator), so one group drains a tile while the
// tensor pipe fills the other accumulator.  An epilogue warp owns 32 rows = 32 / n_c whole
// candidates: it rounds their YC rows to bf16 into a private shared-memory buffer, copies them out
// if the raw block is wanted, and forms OC = ZR + W_CC YC per candidate with warp-level
// mma.sync m16n8k16 (W_CC fragments live in registers, YC fragments come through ldmatrix), so the
// compression sees the same bf16 YC values a caller would read back.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr uint32_t kStatusGlm = 0x200;
constexpr int kAccStride = 256;  // TMEM columns per accumulator

struct GlmParams {
  const Tile* tiles;
  int32_t num_tiles;
  int32_t n_r, n_r_pad, n_c, d, n_ro, n_co;
  int32_t stages, stage_bytes, group_staging_bytes, yc_stride;
  const __nv_bfloat16* W;  // [n_ro + n_co, n] or null
  const float* ZR;         // [R, n_co, n] or null
  int32_t zr_from_previous_launch;  // launched as a programmatic dependent of the kernel that writes ZR
  __nv_bfloat16* YC;       // [N, n_c, n] or null
  __nv_bfloat16* OC;       // [N, n_co, n] or null
  uint32_t* status;
};

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
  // Each CTA takes a contiguous run of tiles: consecutive tiles mostly share a request, so its
  // X^R rows and ZR block stay hot in L1/L2, and the X^C stream of a CTA is sequential in HBM.
  const int32_t t_begin = (int32_t)((int64_t)blockIdx.x * p.num_tiles / gridDim.x);
  const int32_t t_end = (int32_t)((int64_t)(blockIdx.x + 1) * p.num_tiles / gridDim.x);

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
      for (int32_t t = t_begin; t < t_end; ++t, ++it) {
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
    for (int32_t t = t_begin; t < t_end; ++t, ++it) {
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
    // Everything below is local to one warp: a warp owns 32 tile rows = 32 / NC whole candidates.
    const int g = (warp - 2) / 4;  // group 0: warps 2-5, group 1: warps 6-9
    const int q = warp % 4;        // TMEM lane quadrant = rows 32q .. 32q+31 of the tile
    const int n8 = n / 8;
    // bf16 copy of this warp's 32 rows of YC, row stride yc_stride bytes (16 mod 32: no conflicts)
    uint8_t* yc_w = staging + g * p.group_staging_bytes + q * 32 * p.yc_stride;
    uint8_t* my = yc_w + lane * p.yc_stride;
    const bool compress = p.W != nullptr && p.OC != nullptr;
    bool zr_ready = !p.zr_from_previous_launch;
    // A fragments of W_CC for mma.m16n8k16 (rows = outputs o, padded to 16; cols = a, padded to
    // 16 per K step): a0 = (g8, 2t..), a1 = (g8+8, 2t..), a2 = (g8, 2t+8..), a3 = (g8+8, 2t+8..)
    constexpr int KS = (NC + 15) / 16;
    uint32_t wa[KS][4];
    const int g8 = lane / 4, t4 = lane % 4;
    if (compress) {
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int o = g8 + (i & 1) * 8, a0 = ks * 16 + 2 * t4 + (i >> 1) * 8;
          __nv_bfloat16 lo = __float2bfloat16_rn(0.f), hi = lo;
          if (o < p.n_co) {
            const __nv_bfloat16* wrow = p.W + (int64_t)(p.n_ro + o) * n + p.n_r;
            if (a0 < NC) lo = wrow[a0];
            if (a0 + 1 < NC) hi = wrow[a0 + 1];
          }
          __nv_bfloat162 h2(lo, hi);
          wa[ks][i] = *reinterpret_cast<uint32_t*>(&h2);
        }
    }
    uint32_t it = 0;
    for (int32_t t = t_begin; t < t_end; ++t, ++it) {
      if ((int)(it & 1) != g) continue;
      const Tile tile = p.tiles[t];
      if (!mbar_wait(&tmem_full[g], (it >> 1) & 1, abort_flag, p.status, kStatusGlm | 4)) break;
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + g * kAccStride + ((uint32_t)(q * 32) << 16);
      // All TMEM reads of the tile are issued before the first wait: the first 32 columns of the
      // request-candidate block and the 32 x 32 diagonal block of this warp's rows.
      uint32_t vcr[32], vcc[32];
      tmem_ld_32x32b_x32(t_row, vcr);
      tmem_ld_32x32b_x32(t_row + p.n_r_pad + q * 32, vcc);
      tmem_ld_wait();
      auto store8 = [&](const uint32_t* v, int32_t col) {
        uint4 w;
        __nv_bfloat162 b2;
        b2 = __floats2bfloat162_rn(__uint_as_float(v[0]), __uint_as_float(v[1])); w.x = *reinterpret_cast<uint32_t*>(&b2);
        b2 = __floats2bfloat162_rn(__uint_as_float(v[2]), __uint_as_float(v[3])); w.y = *reinterpret_cast<uint32_t*>(&b2);
        b2 = __floats2bfloat162_rn(__uint_as_float(v[4]), __uint_as_float(v[5])); w.z = *reinterpret_cast<uint32_t*>(&b2);
        b2 = __floats2bfloat162_rn(__uint_as_float(v[6]), __uint_as_float(v[7])); w.w = *reinterpret_cast<uint32_t*>(&b2);
        *reinterpret_cast<uint4*>(my + col * 2) = w;
      };
#pragma unroll
      for (int h = 0; h < 4; ++h)
        if (8 * h < p.n_r) store8(vcr + 8 * h, 8 * h);
      for (int32_t c0 = 32; c0 < p.n_r; c0 += 32) {  // wider request blocks: 32 more columns per pass
        tmem_ld_32x32b_x32(t_row + c0, vcr);
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < 4; ++h)
          if (c0 + 8 * h < p.n_r) store8(vcr + 8 * h, c0 + 8 * h);
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[g]);
      {
        // of the diagonal block each thread keeps the NC columns of its own candidate
        const int sub = lane / NC;
        uint32_t x[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) {
          uint32_t xv = vcc[j];
#pragma unroll
          for (int s2 = 1; s2 < 32 / NC; ++s2) xv = (sub == s2) ? vcc[s2 * NC + j] : xv;
          x[j] = xv;
        }
#pragma unroll
        for (int j = 0; j < NC; j += 8) store8(x + j, p.n_r + j);
      }
      __syncwarp();
      const int32_t rows_valid = min(32, tile.count * NC - q * 32);  // this warp's rows that are real
      if (rows_valid <= 0) continue;
      if (p.YC != nullptr) {
        // raw block: the warp's rows are contiguous in YC; 16-byte vectors
        uint4* dst = reinterpret_cast<uint4*>(p.YC + ((int64_t)tile.cand0 * NC + q * 32) * n);
        const int32_t vecs = rows_valid * n8;
        for (int32_t e = lane; e < vecs; e += 32) {
          const int32_t r0 = e / n8, c8 = e % n8;
          dst[e] = *reinterpret_cast<const uint4*>(yc_w + r0 * p.yc_stride + c8 * 16);
        }
      }
      if (compress) {
        // OC[c] (n_co x n) = ZR[r] + W_CC (n_co x NC) * YC[c] (NC x n) per candidate, on the warp-level
        // tensor-core path (mma.sync m16n8k16): the product is tiny and needs no TMEM round trip.
        const float* zr = p.ZR + (int64_t)tile.req * p.n_co * n;
        if (!zr_ready) {  // the request kernel must have finished before its result is read
          griddep_wait();
          zr_ready = true;
        }
        const int32_t cands = rows_valid / NC;
        for (int32_t cl = 0; cl < cands; ++cl) {
          __nv_bfloat16* oc = p.OC + ((int64_t)tile.cand0 + q * (32 / NC) + cl) * p.n_co * n;
          // six 8-column blocks at a time, all loads first, so the tensor-core ops overlap
          for (int32_t j0 = 0; j0 < n8; j0 += 6) {
            float dd[6][4];
            uint32_t bb[6][KS][2];
#pragma unroll
            for (int u = 0; u < 6; ++u) {
              const int32_t j = min(j0 + u, n8 - 1);
              const int32_t col = 8 * j + 2 * t4;
              dd[u][0] = dd[u][1] = dd[u][2] = dd[u][3] = 0.f;
              if (g8 < p.n_co) {
                const float2 z = __ldg(reinterpret_cast<const float2*>(zr + g8 * n + col));
                dd[u][0] = z.x; dd[u][1] = z.y;
              }
              if (g8 + 8 < p.n_co) {
                const float2 z = __ldg(reinterpret_cast<const float2*>(zr + (g8 + 8) * n + col));
                dd[u][2] = z.x; dd[u][3] = z.y;
              }
#pragma unroll
              for (int ks = 0; ks < KS; ++ks) {
                bb[u][ks][1] = 0u;
                if constexpr (NC >= 16) {
                  const uint32_t addr = smem_u32(yc_w + (cl * NC + ks * 16 + (lane & 15)) * p.yc_stride + j * 16);
                  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
                               : "=r"(bb[u][ks][0]), "=r"(bb[u][ks][1]) : "r"(addr));
                } else {
                  const uint32_t addr8 = smem_u32(yc_w + (cl * NC + (lane & 7)) * p.yc_stride + j * 16);
                  asm volatile("ldmatrix.sync.aligned.m8n8.x1.trans.shared.b16 {%0}, [%1];" : "=r"(bb[u][ks][0]) : "r"(addr8));
                }
              }
            }
#pragma unroll
            for (int u = 0; u < 6; ++u)
#pragma unroll
              for (int ks = 0; ks < KS; ++ks)
                asm volatile(
                    "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                    "{%0, %1, %2, %3};"
                    : "+f"(dd[u][0]), "+f"(dd[u][1]), "+f"(dd[u][2]), "+f"(dd[u][3])
                    : "r"(wa[ks][0]), "r"(wa[ks][1]), "r"(wa[ks][2]), "r"(wa[ks][3]), "r"(bb[u][ks][0]), "r"(bb[u][ks][1]));
#pragma unroll
            for (int u = 0; u < 6; ++u) {
              if (j0 + u >= n8) continue;
              const int32_t col = 8 * (j0 + u) + 2 * t4;
              if (g8 < p.n_co) *reinterpret_cast<__nv_bfloat162*>(oc + g8 * n + col) = __floats2bfloat162_rn(dd[u][0], dd[u][1]);
              if (g8 + 8 < p.n_co)
                *reinterpret_cast<__nv_bfloat162*>(oc + (g8 + 8) * n + col) = __floats2bfloat162_rn(dd[u][2], dd[u][3]);
            }
          }
        }
      }
      __syncwarp();  // the row buffer is rewritten by this warp's next tile
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
  // bf16 rows; a stride of 16 mod 32 bytes keeps 16-byte row writes and ldmatrix reads conflict free
  L.yc_stride = (n * 2) % 32 == 0 ? n * 2 + 16 : n * 2;
  (void)n_co;
  L.group_staging_bytes = (128 * L.yc_stride + 127) & ~127;
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
  if (n_r % 8 != 0 || n_co > 16) return false;
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
  // The request kernel runs directly in front on the same stream and releases its dependents at once:
  // this kernel sets itself up and streams X^C beside it and waits for it only before it reads ZR.
  p.zr_from_previous_launch = (zr_workspace != nullptr && W != nullptr && OC != nullptr) ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = L.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.zr_from_previous_launch ? 1 : 0;
#define ROCS_GLM_LAUNCH(NC_)                                                                                  \
  do {                                                                                                        \
    ROCS_CUDA_TRY(cudaFuncSetAttribute(glm_umma_kernel<NC_>, cudaFuncAttributeMaxDynamicSharedMemorySize,     \
                                       L.smem_bytes));                                                        \
    ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, glm_umma_kernel<NC_>, map_xr, map_xc, p));                         \
  } while (0)
  if (n_c == 8) ROCS_GLM_LAUNCH(8);
  else if (n_c == 16) ROCS_GLM_LAUNCH(16);
  else ROCS_GLM_LAUNCH(32);
#undef ROCS_GLM_LAUNCH
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
