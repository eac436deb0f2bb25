// Weight-stationary variant of the tensor-core linear layer for narrow inputs (d_in <= 256), the
// shape of the candidate half of a split layer (Eq. 14): Y_i = act(Z[m_i] + X^C_i W_CC^T).
//
// With a short K loop the output dominates: per 128 x 256 tile the kernel reads 64 KB of X and
// writes 64 KB of Y, so re-streaming a 128 KB weight slice per tile from L2 (as a K-ring GEMM
// does) costs more than everything else.  Here every CTA keeps ONE 256-column slice of W in
// shared memory for its whole life and only streams X tiles:
//   CTA b: column slice n = b % n_slices, row-tile group g = b / n_slices; tiles g, g + G, ...
//   warp 0    TMA producer: W slice once; per tile the X tile (k_blocks x 16 KB) and, per 32-row
//             slab, the fp32 request row Z[r, slice] of the slab's first request
//   warp 1    tcgen05.mma 128 x 256 x 16 into one of two TMEM accumulators
//   warps 2-9 epilogue, two warps per TMEM lane quadrant (128 columns each): TMEM -> registers,
//             + Z, ReLU, bf16, 32-byte vector stores straight to global memory
// The request row comes from shared memory when the thread's request is the slab's first request
// (always, when segments are long) and from global memory otherwise (short segments), selected
// per thread through one generic pointer: the in-kernel broadcast of Section 4.2.1 without an
// exposed gather latency.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kAStageBytes = BM * BK * 2;   // 16 KB
constexpr int kWBlockBytes = BN * BK * 2;   // 32 KB per 64-wide K block
constexpr int kZBufBytes = 4 * BN * 4;      // four slabs x 256 fp32
constexpr int kZBufs = 4;                   // request-row buffers: the producer may run this many tiles ahead
constexpr uint32_t kStatusWs = 0x300;

struct WsParams {
  int64_t M;
  int32_t d_in, d_out;
  int32_t n_slices, groups, a_stages;
  const float* bias;
  const float* add;
  int64_t ld_add;
  const int32_t* row2req;
  int32_t act;
  __nv_bfloat16* Y;
  int64_t ld_y;
  uint32_t* status;
};

__global__ void __launch_bounds__(kThreads, 1)
linear_ws_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_z, const WsParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int32_t k_blocks = (p.d_in + BK - 1) / BK;
  uint8_t* w_smem = smem;
  uint8_t* a_smem = w_smem + k_blocks * kWBlockBytes;
  float* z_smem = reinterpret_cast<float*>(a_smem + p.a_stages * kAStageBytes);  // [kZBufs][4][256]
  uint64_t* a_full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(z_smem) + kZBufs * kZBufBytes);
  uint64_t* a_empty = a_full + 8;
  uint64_t* tmem_full = a_empty + 8;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* z_full = tmem_empty + 2;
  uint64_t* z_empty = z_full + kZBufs;
  uint64_t* w_full = z_empty + kZBufs;
  uint64_t* drain = w_full + 1;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int32_t slice = blockIdx.x % p.n_slices, group = blockIdx.x / p.n_slices;
  const int32_t n0 = slice * BN;
  const int32_t m_tiles = (int32_t)((p.M + BM - 1) / BM);
  const bool has_add = p.add != nullptr;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.a_stages; ++s) {
      mbar_init(&a_full[s], 1);
      mbar_init(&a_empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], kEpiWarps);
    }
    for (int a = 0; a < kZBufs; ++a) {
      mbar_init(&z_full[a], 1);
      mbar_init(&z_empty[a], kEpiWarps);
    }
    mbar_init(w_full, 1);
    mbar_init(drain, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_ptr, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      mbar_expect_tx(w_full, k_blocks * kWBlockBytes);
      for (int32_t kb = 0; kb < k_blocks; ++kb) tma_load_2d(w_smem + kb * kWBlockBytes, &map_w, w_full, kb * BK, n0);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      // request ids of the four slabs of a tile, fetched one tile ahead of their use
      int32_t req_next[4] = {0, 0, 0, 0};
      auto fetch_req = [&](int32_t mt_) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int64_t r0 = min((int64_t)mt_ * BM + q * 32, p.M - 1);
          req_next[q] = p.row2req ? p.row2req[r0] : (int32_t)r0;
        }
      };
      if (has_add && group < m_tiles) fetch_req(group);
      for (int32_t mt = group; mt < m_tiles && ok; mt += p.groups, ++lt) {
        const int32_t m0 = mt * BM;
        // X first: the MMA needs it now; the request rows are only needed by this tile's epilogue
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % p.a_stages;
          if (!mbar_wait(&a_empty[s], ((it / p.a_stages) & 1) ^ 1, abort_flag, p.status, kStatusWs | 1)) { ok = false; break; }
          mbar_expect_tx(&a_full[s], kAStageBytes);
          tma_load_2d(a_smem + s * kAStageBytes, &map_x, &a_full[s], kb * BK, m0);
        }
        if (!ok) break;
        if (has_add) {
          const uint32_t zb = lt % kZBufs;
          if (!mbar_wait(&z_empty[zb], ((lt / kZBufs) & 1) ^ 1, abort_flag, p.status, kStatusWs | 5)) { ok = false; break; }
          mbar_expect_tx(&z_full[zb], kZBufBytes);
#pragma unroll
          for (int q = 0; q < 4; ++q) tma_load_2d(z_smem + (zb * 4 + q) * BN, &map_z, &z_full[zb], n0, req_next[q]);
          if (mt + p.groups < m_tiles) fetch_req(mt + p.groups);
        }
      }
      if (!ok) {
        for (int s = 0; s < p.a_stages; ++s) {
          const uint32_t n_issued = it / p.a_stages + (((int)(it % p.a_stages) > s) ? 1 : 0);
          if (n_issued == 0) continue;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&a_full[s], (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(w_full, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ---------------------------------------------
    constexpr uint32_t idesc = umma_idesc_bf16(BM, BN, false, false);
    uint32_t it = 0, lt = 0;
    bool ok = mbar_wait(w_full, 0, abort_flag, p.status, kStatusWs | 6);
    for (int32_t mt = group; mt < m_tiles && ok; mt += p.groups, ++lt) {
      const uint32_t acc = lt & 1;
      if (!mbar_wait(&tmem_empty[acc], ((lt >> 1) & 1) ^ 1, abort_flag, p.status, kStatusWs | 2)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
        const int s = it % p.a_stages;
        if (!mbar_wait(&a_full[s], (it / p.a_stages) & 1, abort_flag, p.status, kStatusWs | 3)) { ok = false; break; }
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t a_desc = smem_desc_sw128(smem_u32(a_smem + s * kAStageBytes), 1024, 16);
          const uint64_t b_desc = smem_desc_sw128(smem_u32(w_smem + kb * kWBlockBytes), 1024, 16);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) umma_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(&a_empty[s]);
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
    const int q = warp % 4;             // TMEM lane quadrant = 32-row slab of the tile
    const int half = (warp - 2) / 4;    // which 128 of the slice's 256 columns
    uint32_t lt = 0;
    for (int32_t mt = group; mt < m_tiles; mt += p.groups, ++lt) {
      const uint32_t acc = lt & 1;
      const int32_t m0 = mt * BM;
      const int64_t row = (int64_t)m0 + q * 32 + lane;
      const float* zrow = nullptr;
      if (has_add) {
        const int64_t rc = min(row, p.M - 1);
        const int32_t my_req = p.row2req ? p.row2req[rc] : (int32_t)rc;
        const int32_t slab_req = __shfl_sync(0xffffffffu, my_req, 0);
        // shared-memory copy when this row belongs to the slab's first request, global otherwise
        zrow = (my_req == slab_req) ? (z_smem + ((lt % kZBufs) * 4 + q) * BN) : (p.add + (int64_t)my_req * p.ld_add + n0);
        if (!mbar_wait(&z_full[lt % kZBufs], (lt / kZBufs) & 1, abort_flag, p.status, kStatusWs | 7)) break;
      }
      if (!mbar_wait(&tmem_full[acc], (lt >> 1) & 1, abort_flag, p.status, kStatusWs | 4)) break;
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + acc * BN + half * 128 + ((uint32_t)(q * 32) << 16);
      __nv_bfloat16* yrow = p.Y + row * p.ld_y + n0 + half * 128;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int32_t colL = half * 128 + c * 64;   // column inside the slice
        uint32_t v[64];
        tmem_ld_32x32b_x32(t_row + c * 64, v);
        tmem_ld_32x32b_x32(t_row + c * 64 + 32, v + 32);
        tmem_ld_wait();
        if (c == 1) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        float f[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) f[i] = __uint_as_float(v[i]);
        if (has_add) {
#pragma unroll
          for (int i = 0; i < 64; i += 4) {
            if (n0 + colL + i < p.d_out) {
              const float4 z = *reinterpret_cast<const float4*>(zrow + colL + i);
              f[i] += z.x; f[i + 1] += z.y; f[i + 2] += z.z; f[i + 3] += z.w;
            }
          }
        }
        if (p.bias != nullptr) {
#pragma unroll
          for (int i = 0; i < 64; i += 4) {
            if (n0 + colL + i < p.d_out) {
              const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + n0 + colL + i));
              f[i] += b.x; f[i + 1] += b.y; f[i + 2] += b.z; f[i + 3] += b.w;
            }
          }
        }
        if (p.act == ROCS_ACT_RELU) {
#pragma unroll
          for (int i = 0; i < 64; ++i) f[i] = fmaxf(f[i], 0.f);
        }
        if (row < p.M) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              __nv_bfloat162 h = __floats2bfloat162_rn(f[16 * j + 2 * u], f[16 * j + 2 * u + 1]);
              w[u] = *reinterpret_cast<uint32_t*>(&h);
            }
            const int32_t col = n0 + colL + 16 * j;
            __nv_bfloat16* dst = yrow + c * 64 + 16 * j;
            if (col + 16 <= p.d_out && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
              asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]),
                           "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                           : "memory");
            } else {
#pragma unroll
              for (int u = 0; u < 2; ++u)   // two 16-byte halves, each either fully inside or outside
                if (col + 8 * u < p.d_out)
                  *reinterpret_cast<uint4*>(dst + 8 * u) = make_uint4(w[4 * u], w[4 * u + 1], w[4 * u + 2], w[4 * u + 3]);
            }
          }
        }
      }
      if (has_add) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&z_empty[lt % kZBufs]);
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

int sm_count_ws() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

}  // namespace

bool umma_linear_ws_supported(int64_t M, int32_t d_in, int32_t d_out, bool out_f32) {
  if (out_f32 || d_in < 8 || d_in > 256 || d_out < 64 || d_out % 8 != 0) return false;
  if (M < 512) return false;  // not worth parking a weight slice per CTA
  return (d_out + BN - 1) / BN <= sm_count_ws();
}

rocs_status_t umma_linear_ws(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x, const void* W,
                             int64_t ld_w, const float* bias, const float* add, int64_t ld_add,
                             const int32_t* row2req, int act, void* Y, int64_t ld_y, cudaStream_t stream) {
  const int32_t k_blocks = (d_in + BK - 1) / BK;
  CUtensorMap map_x, map_w, map_z;
  if (!make_tensor_map_2d(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_in, (uint64_t)ld_x,
                          BM, BK, true) ||
      !make_tensor_map_2d(&map_w, W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_out, (uint64_t)d_in,
                          (uint64_t)ld_w, BN, BK, true))
    return ROCS_ERR_CUDA;
  if (add != nullptr) {
    // Z is [rows, d_out] fp32 with row stride ld_add; the row count only bounds the map, and the
    // kernel addresses rows through row2req, so a generous bound is safe.
    if (!make_tensor_map_2d(&map_z, add, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, (uint64_t)0x7fffffff, (uint64_t)d_out,
                            (uint64_t)ld_add, 1, BN, false))
      return ROCS_ERR_CUDA;
  } else {
    map_z = map_x;
  }
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  WsParams p{};
  p.M = M; p.d_in = d_in; p.d_out = d_out;
  p.n_slices = (d_out + BN - 1) / BN;
  const int32_t m_tiles = (int32_t)((M + BM - 1) / BM);
  p.groups = std::max(1, std::min(m_tiles, sm_count_ws() / p.n_slices));
  const int fixed = k_blocks * kWBlockBytes + kZBufs * kZBufBytes + 512 + 1024;
  p.a_stages = std::min(8, (227 * 1024 - fixed) / kAStageBytes);
  p.bias = bias; p.add = add; p.ld_add = ld_add; p.row2req = row2req; p.act = act;
  p.Y = (__nv_bfloat16*)Y; p.ld_y = ld_y; p.status = status;
  const int smem_bytes = fixed + p.a_stages * kAStageBytes;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(linear_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
  linear_ws_kernel<<<p.n_slices * p.groups, kThreads, smem_bytes, stream>>>(map_x, map_w, map_z, p);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
