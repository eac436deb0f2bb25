// Linear layer on the 5th-generation tensor cores (Eq. 4 / Eq. 14):
//     Y[i, n] = act( sum_k X[i, k] W[n, k] + bias[n] + add[row2req[i], n] )
// `add` is the request half Z of the split layer; it is gathered per output row in the epilogue
// through the candidate->request map (the in-kernel broadcast of Section 4.2.1), so the broadcast
// tensor never exists.
//
// One persistent CTA per SM, 6 warps:
//   warp 0   TMA producer: 128 x 64 tiles of X and BN x 64 tiles of W into a shared-memory ring
//   warp 1   issues tcgen05.mma (128 x BN x 16, bf16 -> fp32) into one of two TMEM accumulators
//   warps 2-5 epilogue: TMEM -> registers, + Z[m_i] (+ bias), ReLU, round to the output type,
//            128-byte-swizzled staging in shared memory, TMA store (clipped at the edges)
// The two accumulators let the epilogue of tile t overlap the main loop of tile t + 1.
// Tiles are ordered with the output-column index fastest, so CTAs working at the same time share
// the same rows of X in L2.  M tiles may span several requests: each row looks up its own request.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int BM = 128;           // rows per tile = TMEM lanes
constexpr int BK = 64;            // 64 bf16 = one 128-byte swizzle row
constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
constexpr uint32_t kStatusLinear = 0x100;

template <int BN>
struct LinearCfg {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStagingBytes = kEpiWarps * 2 * 4096;  // per warp: two 32-row x 128-byte buffers
  static constexpr int kTmemCols = 2 * BN >= 32 ? 2 * BN : 32;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 256 /*barriers*/ + 1024 /*align*/;
};

struct LinearParams {
  int64_t M;
  int32_t d_in, d_out;
  const float* bias;
  const float* add;
  int64_t ld_add;
  const int32_t* row2req;
  int32_t act;
  uint32_t* status;
};

template <int BN, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
linear_umma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   const __grid_constant__ CUtensorMap map_y, const LinearParams p) {
  using Cfg = LinearCfg<BN>;
  constexpr int kStages = Cfg::kStages;
  constexpr int CH = 128 / (int)sizeof(OutT);  // output columns per 128-byte staging row

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + kStages * Cfg::kStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(staging + Cfg::kStagingBytes);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* drain = tmem_empty + 2;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int32_t m_tiles = (int32_t)((p.M + BM - 1) / BM);
  const int32_t n_tiles = (p.d_out + BN - 1) / BN;
  const int32_t k_blocks = (p.d_in + BK - 1) / BK;
  const int64_t num_tiles = (int64_t)m_tiles * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], kEpiWarps);
    }
    mbar_init(drain, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_ptr, Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  // Launched as a programmatic dependent: the set-up above may overlap the end of the kernel in front;
  // nothing below touches global memory before that kernel is complete.  Then the kernel behind this one
  // (the candidate half behind the request half) may begin its own set-up; it waits for this grid before
  // it reads our output, and since it is released only after the wait above, everything in front of this
  // kernel is complete by the time it starts.
  griddep_wait();
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      uint32_t it = 0;
      bool ok = true;
      for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const int32_t m0 = (int32_t)(t / n_tiles) * BM, n0 = (int32_t)(t % n_tiles) * BN;
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag, p.status, kStatusLinear | 1)) { ok = false; break; }
          uint8_t* a = smem + s * Cfg::kStageBytes;
          mbar_expect_tx(&full[s], Cfg::kStageBytes);
          tma_load_2d(a, &map_x, &full[s], kb * BK, m0);
          tma_load_2d(a + Cfg::kABytes, &map_w, &full[s], kb * BK, n0);
        }
      }
      if (!ok) {
        // Aborting: let the copies already in flight land before the CTA gives up its shared memory.
        for (int s = 0; s < kStages; ++s) {
          const uint32_t n_issued = it / kStages + (((int)(it % kStages) > s) ? 1 : 0);  // loads issued to stage s
          if (n_issued == 0) continue;
          const uint32_t ph = (n_issued - 1) & 1;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&full[s], ph) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ---------------------------------------------
    constexpr uint32_t idesc = umma_idesc_bf16(BM, BN, false, false);
    uint32_t it = 0, lt = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++lt) {
      const uint32_t acc = lt & 1;
      if (!mbar_wait(&tmem_empty[acc], ((lt >> 1) & 1) ^ 1, abort_flag, p.status, kStatusLinear | 2)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
        const int s = it % kStages;
        if (!mbar_wait(&full[s], (it / kStages) & 1, abort_flag, p.status, kStatusLinear | 3)) { ok = false; break; }
        tc_fence_after_sync();
        if (lane == 0) {
          const uint32_t a_addr = smem_u32(smem + s * Cfg::kStageBytes);
          const uint64_t a_desc = smem_desc_sw128(a_addr, 1024, 16);
          const uint64_t b_desc = smem_desc_sw128(a_addr + Cfg::kABytes, 1024, 16);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)  // +32 bytes = 16 bf16 along K, in 16-byte units
            umma_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(&empty[s]);  // frees the stage once these MMAs have read it
        }
        __syncwarp();
      }
      if (ok && lane == 0) umma_commit(&tmem_full[acc]);
      __syncwarp();
    }
    if (!ok && lane == 0) {
      umma_commit(drain);
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(drain, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ------------------------------ epilogue -----------------------------------------------
    const int q = warp % 4;  // TMEM lane quadrant this warp may read
    uint8_t* my_stage = staging + (warp - 2) * 8192;
    uint32_t lt = 0, stores = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++lt) {
      const uint32_t acc = lt & 1;
      const int32_t m0 = (int32_t)(t / n_tiles) * BM, n0 = (int32_t)(t % n_tiles) * BN;
      const int64_t row = (int64_t)m0 + q * 32 + lane;
      const float* add_row = nullptr;
      if (p.add != nullptr && row < p.M)
        add_row = p.add + (int64_t)(p.row2req ? p.row2req[row] : row) * p.ld_add;
      if (!mbar_wait(&tmem_full[acc], (lt >> 1) & 1, abort_flag, p.status, kStatusLinear | 4)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
      constexpr int kChunks = BN / CH;
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        const int32_t col0 = n0 + c * CH;
        if (col0 >= p.d_out) break;
        uint32_t v[CH];
        tmem_ld_32x32b_x32(t_row + c * CH, v);
        if constexpr (CH == 64) tmem_ld_32x32b_x32(t_row + c * CH + 32, v + 32);
        tmem_ld_wait();
        if (c == kChunks - 1 || col0 + CH >= p.d_out) {
          // last read of this accumulator: hand it back to the MMA warp before finishing the math
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        float f[CH];
#pragma unroll
        for (int i = 0; i < CH; ++i) f[i] = __uint_as_float(v[i]);
        if (add_row != nullptr) {
#pragma unroll
          for (int i = 0; i < CH; i += 4) {
            if (col0 + i < p.d_out) {
              const float4 z = __ldg(reinterpret_cast<const float4*>(add_row + col0 + i));
              f[i] += z.x; f[i + 1] += z.y; f[i + 2] += z.z; f[i + 3] += z.w;
            }
          }
        }
        if (p.bias != nullptr) {
#pragma unroll
          for (int i = 0; i < CH; i += 4) {
            if (col0 + i < p.d_out) {
              const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col0 + i));
              f[i] += b.x; f[i + 1] += b.y; f[i + 2] += b.z; f[i + 3] += b.w;
            }
          }
        }
        if (p.act == ROCS_ACT_RELU) {
#pragma unroll
          for (int i = 0; i < CH; ++i) f[i] = fmaxf(f[i], 0.f);
        }
        // staging buffer (two per warp): make sure the TMA store that last read it has finished
        uint8_t* buf = my_stage + (stores & 1) * 4096;
        if (lane == 0) tma_store_wait_read<1>();
        __syncwarp();
        uint8_t* row_ptr = buf + lane * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {  // eight 16-byte chunks per 128-byte row, XOR-swizzled by row
          uint4 w;
          if constexpr (sizeof(OutT) == 2) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(f[8 * j + 0], f[8 * j + 1]);
            __nv_bfloat162 h1 = __floats2bfloat162_rn(f[8 * j + 2], f[8 * j + 3]);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(f[8 * j + 4], f[8 * j + 5]);
            __nv_bfloat162 h3 = __floats2bfloat162_rn(f[8 * j + 6], f[8 * j + 7]);
            w.x = *reinterpret_cast<uint32_t*>(&h0);
            w.y = *reinterpret_cast<uint32_t*>(&h1);
            w.z = *reinterpret_cast<uint32_t*>(&h2);
            w.w = *reinterpret_cast<uint32_t*>(&h3);
          } else {
            w.x = __float_as_uint(f[4 * j + 0]);
            w.y = __float_as_uint(f[4 * j + 1]);
            w.z = __float_as_uint(f[4 * j + 2]);
            w.w = __float_as_uint(f[4 * j + 3]);
          }
          *reinterpret_cast<uint4*>(row_ptr + ((j ^ (lane & 7)) << 4)) = w;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&map_y, buf, col0, m0 + q * 32);
          tma_store_commit();
        }
        ++stores;
      }
    }
    if (lane == 0) tma_store_wait_all<0>();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

template <int BN, typename OutT>
rocs_status_t launch(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x, const void* W,
                     int64_t ld_w, const float* bias, const float* add, int64_t ld_add, const int32_t* row2req,
                     int act, void* Y, int64_t ld_y, cudaStream_t stream) {
  using Cfg = LinearCfg<BN>;
  constexpr int CH = 128 / (int)sizeof(OutT);
  CUtensorMap map_x, map_w, map_y;
  if (!make_tensor_map_2d(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_in, (uint64_t)ld_x,
                          BM, BK, true) ||
      !make_tensor_map_2d(&map_w, W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_out, (uint64_t)d_in,
                          (uint64_t)ld_w, BN, BK, true) ||
      !make_tensor_map_2d(&map_y, Y, sizeof(OutT) == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                          sizeof(OutT), (uint64_t)M, (uint64_t)d_out, (uint64_t)ld_y, 32, CH, true))
    return ROCS_ERR_CUDA;
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  auto kernel = linear_umma_kernel<BN, OutT>;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
  const int64_t tiles = ((M + BM - 1) / BM) * ((d_out + BN - 1) / BN);
  const int grid = (int)std::min<int64_t>(tiles, sm_count());
  LinearParams p{M, d_in, d_out, bias, add, ld_add, row2req, act, status};
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_x, map_w, map_y, p));
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace

bool umma_linear_supported(int64_t M, int32_t d_in, int32_t d_out, int64_t ld_x, int64_t ld_w, int64_t ld_y,
                           bool out_f32) {
  (void)ld_x; (void)ld_w; (void)ld_y;  // row strides are already multiples of 16 bytes at the ABI
  if (M < 1 || M > 0x7fffff00LL || d_in < 8 || d_out < 8) return false;
  if (d_out % 4 != 0) return false;  // fp32 request rows are read as float4
  (void)out_f32;
  return true;
}

rocs_status_t umma_linear(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x, const void* W,
                          int64_t ld_w, const float* bias, const float* add, int64_t ld_add,
                          const int32_t* row2req, int act, void* Y, int64_t ld_y, bool out_f32,
                          cudaStream_t stream, bool add_from_previous_launch, float2* stat_partials,
                          int64_t add_rows) {
  if (umma_linear_ws2_supported(M, d_in, d_out, out_f32))
    return umma_linear_ws2(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y, stream,
                           add_from_previous_launch, stat_partials, add_rows);
  if (stat_partials != nullptr) return ROCS_ERR_UNSUPPORTED;  // the caller asks for them only where the kernel above applies
  if (umma_linear_pair_supported(M, d_in, d_out, out_f32, add != nullptr))
    return umma_linear_pair(M, d_in, d_out, X, ld_x, W, ld_w, bias, act, Y, ld_y, stream);
#define ROCS_LAUNCH(BN_)                                                                                   \
  (out_f32 ? launch<BN_, float>(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, ld_y, \
                                stream)                                                                    \
           : launch<BN_, __nv_bfloat16>(M, d_in, d_out, X, ld_x, W, ld_w, bias, add, ld_add, row2req, act, Y, \
                                        ld_y, stream))
  // Widest tile that still gives every SM something to do: a small batch (the request half at
  // batch size R) is spread over more, narrower tiles instead of leaving most SMs idle.
  const int64_t m_tiles = (M + BM - 1) / BM;
  const int sms = sm_count();
  int bn = d_out > 128 ? 256 : (d_out > 64 ? 128 : 64);
  while (bn > 64 && m_tiles * ((d_out + bn - 1) / bn) < sms) bn /= 2;
  if (bn == 256) return ROCS_LAUNCH(256);
  if (bn == 128) return ROCS_LAUNCH(128);
  return ROCS_LAUNCH(64);
#undef ROCS_LAUNCH
}

}  // namespace rocs
