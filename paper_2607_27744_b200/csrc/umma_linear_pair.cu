// K-ring GEMM on CTA pairs (tcgen05 cta_group::2) for wide plain layers (Eq. 4, one group):
//     Y[i, n] = act( sum_k X[i, k] W[n, k] + bias[n] )
// Two CTAs of a cluster drive one 256 x 256 x 16 MMA per K step: each CTA streams its own 128 rows of
// X and HALF of the 256-row weight tile through its shared-memory ring, so a CTA moves 32 KB per
// 64-deep K block instead of the 48 KB a single-CTA 128 x 256 tile needs, and the pair shares every
// weight byte it loads.  Two TMEM accumulators let the epilogue of a tile overlap the next main loop.
//   warp 0 (both CTAs)  TMA producer; completion of both CTAs' tiles is counted on the LEADER's barrier
//   warp 1 (leader)     tcgen05.mma.cta_group::2; commits are multicast to both CTAs' barriers
//   warps 2-9 (both)    epilogue, two warps per TMEM lane quadrant: TMEM -> registers, + bias,
//                       ReLU, bf16, swizzled staging, TMA store
// Tiles are ordered with the column index fastest, so pairs running at the same time share X in L2.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kABytes = BM * BK * 2;         // 16 KB: this CTA's rows of X
constexpr int kBBytes = (BN / 2) * BK * 2;   // 16 KB: this CTA's half of the weight tile
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 6;
constexpr int kStagingBytes = kEpiWarps * 4096;  // one 32-row x 128-byte box per warp, used by both column chunks
constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 512 + 1024;
constexpr uint32_t kStatusPair = 0x300;

struct PairParams {
  int64_t M;
  int32_t d_in, d_out;
  const float* bias;
  int32_t act;
  uint32_t* status;
  // optional normalisation of the input rows, folded into the epilogue:
  //   norm(x) W^T = sc (x W^T) + sh wbar,  sc = 1 / sqrt(var + eps), sh = -mean sc   (LayerNorm)
  //                                        sc = 1 / sqrt(mean(x^2) + eps), sh = 0    (RMSNorm)
  const float2* in_stats;   // [M] (sum, sum of squares) of each input row, or NULL
  const float* wbar;        // [d_out] row sums of W (LayerNorm)
  int32_t norm_kind;
  float eps, inv_d;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   const __grid_constant__ CUtensorMap map_y, const PairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + kStages * kStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(staging + kStagingBytes);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* drain = tmem_empty + 2;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = cluster_ctarank();
  const int32_t pair = blockIdx.x / 2, pairs = gridDim.x / 2;
  const int32_t super_tiles = (int32_t)((p.M + 2 * BM - 1) / (2 * BM));
  const int32_t n_tiles = (p.d_out + BN - 1) / BN;
  const int32_t k_blocks = (p.d_in + BK - 1) / BK;
  const int64_t num_tiles = (int64_t)super_tiles * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], 2 * kEpiWarps);
    }
    mbar_init(drain, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_ptr, 2 * BN);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  // Launched as a programmatic dependent: everything above (barriers, tensor memory) may run while the
  // kernel in front of this one on the stream finishes; nothing below touches global memory before that
  // kernel is complete.  The next kernel on the stream is released only after this wait, so whatever
  // it may assume about its predecessors holds transitively.
  griddep_wait();
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      uint32_t it = 0;
      bool ok = true;
      for (int64_t t = pair; t < num_tiles && ok; t += pairs) {
        const int32_t m0 = (int32_t)(t / n_tiles) * 2 * BM + (int32_t)rank * BM;
        const int32_t n0 = (int32_t)(t % n_tiles) * BN + (int32_t)rank * (BN / 2);
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % kStages;
          if (!mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, abort_flag, p.status, kStatusPair | 1)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(&full[s], 2 * kStageBytes);  // both CTAs' bytes land on the leader's barrier
          const uint32_t full_leader = map_to_cta(smem_u32(&full[s]), 0);
          uint8_t* st = smem + s * kStageBytes;
          tma_load_2d_pair(st, &map_x, full_leader, kb * BK, m0);
          tma_load_2d_pair(st + kABytes, &map_w, full_leader, kb * BK, n0);
        }
      }
      if (!ok) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000) {}  // let copies in flight land before the CTA leaves
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only) ---------------------------
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN, false, false);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int64_t t = pair; t < num_tiles && ok; t += pairs, ++lt) {
        const uint32_t acc = lt & 1;
        if (!mbar_wait(&tmem_empty[acc], ((lt >> 1) & 1) ^ 1, abort_flag, p.status, kStatusPair | 2)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % kStages;
          if (!mbar_wait(&full[s], (it / kStages) & 1, abort_flag, p.status, kStatusPair | 3)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t st = smem_u32(smem + s * kStageBytes);
          const uint64_t a_desc = smem_desc_sw128(st, 1024, 16);
          const uint64_t b_desc = smem_desc_sw128(st + kABytes, 1024, 16);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_ss_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&empty[s], 3);
        }
        if (ok) umma_commit_pair(&tmem_full[acc], 3);
      }
      if (!ok) {
        umma_commit_pair(drain, 1);
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(drain, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs) ------------------------------------
    const int q = warp % 4;
    const int half = (warp - 2) / 4;
    uint8_t* my_stage = staging + (warp - 2) * 4096;
    const uint32_t tmem_empty_leader[2] = {map_to_cta(smem_u32(&tmem_empty[0]), 0),
                                           map_to_cta(smem_u32(&tmem_empty[1]), 0)};
    uint32_t lt = 0;
    for (int64_t t = pair; t < num_tiles; t += pairs, ++lt) {
      const uint32_t acc = lt & 1;
      const int32_t m0 = (int32_t)(t / n_tiles) * 2 * BM + (int32_t)rank * BM;
      const int32_t n0 = (int32_t)(t % n_tiles) * BN;
      if (!mbar_wait(&tmem_full[acc], (lt >> 1) & 1, abort_flag, p.status, kStatusPair | 4)) break;
      tc_fence_after_sync();
      if (lane == 0) tma_store_wait_read<0>();  // the previous tile's stores have read this warp's boxes
      __syncwarp();
      const uint32_t t_row = tmem_base + acc * BN + half * 128 + ((uint32_t)(q * 32) << 16);
      float sc = 1.f, sh = 0.f;
      if (p.in_stats != nullptr) {
        const int64_t row = (int64_t)m0 + q * 32 + lane;
        const float2 st = row < p.M ? __ldg(&p.in_stats[row]) : make_float2(0.f, 0.f);
        const float mean = st.x * p.inv_d, ms = st.y * p.inv_d;
        if (p.norm_kind == ROCS_NORM_RMS) {
          sc = rsqrtf(ms + p.eps);
        } else {
          sc = rsqrtf(fmaxf(ms - mean * mean, 0.f) + p.eps);
          sh = -mean * sc;
        }
      }
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int32_t col0 = n0 + half * 128 + c * 64;
        uint32_t v[64];
        tmem_ld_32x32b_x32(t_row + c * 64, v);
        tmem_ld_32x32b_x32(t_row + c * 64 + 32, v + 32);
        tmem_ld_wait();
        if (c == 1) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_relaxed(tmem_empty_leader[acc]);
        }
        float f[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) f[i] = __uint_as_float(v[i]);
        if (p.in_stats != nullptr) {
#pragma unroll
          for (int i = 0; i < 64; ++i) f[i] *= sc;
          if (p.norm_kind != ROCS_NORM_RMS) {
#pragma unroll
            for (int i = 0; i < 64; i += 4) {
              if (col0 + i < p.d_out) {
                const float4 w = __ldg(reinterpret_cast<const float4*>(p.wbar + col0 + i));
                f[i] = fmaf(sh, w.x, f[i]); f[i + 1] = fmaf(sh, w.y, f[i + 1]);
                f[i + 2] = fmaf(sh, w.z, f[i + 2]); f[i + 3] = fmaf(sh, w.w, f[i + 3]);
              }
            }
          }
        }
        if (p.bias != nullptr) {
#pragma unroll
          for (int i = 0; i < 64; i += 4) {
            if (col0 + i < p.d_out) {
              const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col0 + i));
              f[i] += b.x; f[i + 1] += b.y; f[i + 2] += b.z; f[i + 3] += b.w;
            }
          }
        }
        if (p.act == ROCS_ACT_RELU) {
#pragma unroll
          for (int i = 0; i < 64; ++i) f[i] = fmaxf(f[i], 0.f);
        }
        if (c == 1) {  // the store of the first chunk has finished reading the box
          if (lane == 0) tma_store_wait_read<0>();
          __syncwarp();
        }
        uint8_t* row_ptr = my_stage + lane * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint4 w;
          __nv_bfloat162 h0 = __floats2bfloat162_rn(f[8 * j + 0], f[8 * j + 1]);
          __nv_bfloat162 h1 = __floats2bfloat162_rn(f[8 * j + 2], f[8 * j + 3]);
          __nv_bfloat162 h2 = __floats2bfloat162_rn(f[8 * j + 4], f[8 * j + 5]);
          __nv_bfloat162 h3 = __floats2bfloat162_rn(f[8 * j + 6], f[8 * j + 7]);
          w.x = *reinterpret_cast<uint32_t*>(&h0);
          w.y = *reinterpret_cast<uint32_t*>(&h1);
          w.z = *reinterpret_cast<uint32_t*>(&h2);
          w.w = *reinterpret_cast<uint32_t*>(&h3);
          *reinterpret_cast<uint4*>(row_ptr + ((j ^ (lane & 7)) << 4)) = w;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (col0 < p.d_out && (int64_t)m0 + q * 32 < p.M) tma_store_2d(&map_y, my_stage, col0, m0 + q * 32);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_all<0>();
  }

  tc_fence_before_sync();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 2 * BN);
  }
}

int sm_count_pair() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

}  // namespace

bool umma_linear_pair_supported(int64_t M, int32_t d_in, int32_t d_out, bool out_f32, bool has_add) {
  if (out_f32 || has_add || d_in < 8 || d_out < 256 || d_out % 8 != 0) return false;
  if (M < 2048 || M > 0x7fffff00LL) return false;  // enough 256-row tiles to fill the pairs
  return true;
}

rocs_status_t umma_linear_pair(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x, const void* W,
                               int64_t ld_w, const float* bias, int act, void* Y, int64_t ld_y, cudaStream_t stream,
                               const RowNorm* norm) {
  CUtensorMap map_x, map_w, map_y;
  if (!make_tensor_map_2d(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_in, (uint64_t)ld_x,
                          BM, BK, true) ||
      !make_tensor_map_2d(&map_w, W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_out, (uint64_t)d_in,
                          (uint64_t)ld_w, BN / 2, BK, true) ||
      !make_tensor_map_2d(&map_y, Y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_out, (uint64_t)ld_y,
                          32, 64, true))
    return ROCS_ERR_CUDA;
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  PairParams p{M, d_in, d_out, bias, act, status, nullptr, nullptr, 0, 0.f, 0.f};
  if (norm != nullptr) {
    p.in_stats = norm->row_stats;
    p.wbar = norm->wbar;
    p.norm_kind = norm->kind;
    p.eps = norm->eps;
    p.inv_d = 1.f / (float)d_in;
  }
  const int64_t tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((d_out + BN - 1) / BN);
  const int pairs = (int)std::min<int64_t>(tiles, sm_count_pair() / 2);
  ROCS_CUDA_TRY(cudaFuncSetAttribute(linear_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_pair_kernel, map_x, map_w, map_y, p));
  return ROCS_OK;
}

}  // namespace rocs
