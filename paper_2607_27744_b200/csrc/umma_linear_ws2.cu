// Weight-stationary linear layer on CTA PAIRS (tcgen05 cta_group::2) for narrow inputs (d_in <= 256),
// the candidate half of a split layer (Eq. 14):  Y_i = act(Z[m_i] + X^C_i W_CC^T).
//
// Two CTAs of a cluster (two SMs) drive one 256 x 256 x 16 MMA: each CTA supplies its own 128 rows of
// X and HALF of the 256-column weight slice, and receives its own 128 rows of the accumulator in
// its own TMEM.  Parking only half a slice per SM (64 KB at d_in = 256) leaves shared memory for a
// deep X ring AND a swizzled staging area, so the output leaves through TMA stores: the epilogue
// spends shared-memory wavefronts on 16-byte row pieces instead of one global-memory wavefront per
// 32-byte piece, which is what bounds the single-CTA variant (measured here as well: the same
// epilogue with 32-byte register stores runs in 107 us instead of 84 on configuration 2).  The X ring
// is what the time is most sensitive to (2 / 3 / 4 / 5 / 7 stages: 127 / 107 / 93 / 86 / 84 us), so
// each epilogue warp stages through ONE 4 KB box, used for both of its 64-column chunks, and the
// shared memory saved goes to the ring.
//
//   pair P: column slice P % n_slices, row group P / n_slices; super-tiles (256 rows) g, g + G, ...
//   warp 0 (both CTAs)  TMA producer: its half of W once; per tile its X tile (k_blocks x 16 KB,
//                       completion counted on the LEADER's barrier) and the request rows Z[r, slice]
//                       of its four 32-row slabs
//   warp 1 (leader)     tcgen05.mma.cta_group::2 into one of two TMEM accumulators; commits are
//                       multicast to both CTAs' barriers
//   warps 2-9 (both)    epilogue, two warps per TMEM lane quadrant (128 columns each): TMEM ->
//                       registers, + Z (shared-memory broadcast when the slab has one request,
//                       global gather otherwise), ReLU, bf16, swizzled staging, TMA store
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kAStageBytes = BM * BK * 2;        // 16 KB
constexpr int kWBlockBytes = (BN / 2) * BK * 2;  // this CTA's half of a 64-wide K block: 16 KB
constexpr int kZBufBytes = 4 * BN * 4;           // four slabs x 256 fp32
constexpr int kZBufs = 4;                        // request-row buffers: the producer may run this many tiles ahead
constexpr int kStagingBytes = kEpiWarps * 4096;  // per warp: one 32-row x 128-byte box, reused by both column chunks
constexpr uint32_t kStatusWs2 = 0x500;

struct Ws2Params {
  int64_t M;
  int32_t d_in, d_out;
  int32_t n_slices, groups, a_stages;
  const float* bias;
  const float* add;
  int64_t ld_add;
  const int32_t* row2req;
  int32_t act;
  int32_t wait_for_previous;  // launched with programmatic serialization behind the kernel that writes `add`
  float2* stat_partials;      // [M][2 n_slices] (sum, sum of squares) of each row's 128 columns per epilogue warp, or NULL
  uint32_t* status;
};

__device__ __forceinline__ float4 lds128(const float* p) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(smem_u32(p)));
  return v;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_ws2_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                  const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_y,
                  const Ws2Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int32_t k_blocks = (p.d_in + BK - 1) / BK;
  uint8_t* w_smem = smem;
  uint8_t* a_smem = w_smem + k_blocks * kWBlockBytes;
  uint8_t* staging = a_smem + p.a_stages * kAStageBytes;
  float* z_smem = reinterpret_cast<float*>(staging + kStagingBytes);  // [kZBufs][4][256]
  uint64_t* a_full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(z_smem) + kZBufs * kZBufBytes);
  uint64_t* a_empty = a_full + 10;
  uint64_t* tmem_full = a_empty + 10;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* z_full = tmem_empty + 2;
  uint64_t* z_empty = z_full + kZBufs;
  uint64_t* w_full = z_empty + kZBufs;
  uint64_t* drain = w_full + 1;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const int32_t pair = blockIdx.x / 2;
  const int32_t slice = pair % p.n_slices, group = pair / p.n_slices;
  const int32_t n0 = slice * BN;
  const int32_t super_tiles = (int32_t)((p.M + 2 * BM - 1) / (2 * BM));
  const bool has_add = p.add != nullptr;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.a_stages; ++s) {
      mbar_init(&a_full[s], 1);
      mbar_init(&a_empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], 2 * kEpiWarps);  // the epilogue warps of both CTAs
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
    tmem_alloc_pair(tmem_ptr, 2 * BN);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  cluster_sync_all();  // barriers of both CTAs are initialised before anything signals across the pair
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  // A kernel launched behind this one as a programmatic dependent (the next layer) may set itself up as
  // SMs become free; it waits for this whole grid before it touches global memory.
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      const uint32_t w_full_leader = map_to_cta(smem_u32(w_full), 0);
      if (rank == 0) mbar_expect_tx(w_full, 2 * k_blocks * kWBlockBytes);
      for (int32_t kb = 0; kb < k_blocks; ++kb)
        tma_load_2d_pair(w_smem + kb * kWBlockBytes, &map_w, w_full_leader, kb * BK, n0 + (int32_t)rank * (BN / 2));
      uint32_t it = 0, lt = 0;
      bool ok = true;
      // request ids of the four slabs of a tile, fetched one tile ahead of their use
      int32_t req_next[4] = {0, 0, 0, 0};
      auto fetch_req = [&](int32_t st_) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int64_t r0 = min((int64_t)st_ * 2 * BM + (int64_t)rank * BM + q * 32, p.M - 1);
          req_next[q] = p.row2req ? p.row2req[r0] : (int32_t)r0;
        }
      };
      if (has_add && group < super_tiles) fetch_req(group);
      bool previous_done = !p.wait_for_previous;
      for (int32_t st = group; st < super_tiles && ok; st += p.groups, ++lt) {
        const int32_t m0 = st * 2 * BM + (int32_t)rank * BM;
        // X first: the MMA needs it now; the request rows are only needed by this tile's epilogue
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % p.a_stages;
          if (!mbar_wait(&a_empty[s], ((it / p.a_stages) & 1) ^ 1, abort_flag, p.status, kStatusWs2 | 1)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(&a_full[s], 2 * kAStageBytes);  // both CTAs' tiles land on the leader's barrier
          tma_load_2d_pair(a_smem + s * kAStageBytes, &map_x, map_to_cta(smem_u32(&a_full[s]), 0), kb * BK, m0);
        }
        if (!ok) break;
        if (has_add) {
          const uint32_t zb = lt % kZBufs;
          if (!mbar_wait(&z_empty[zb], ((lt / kZBufs) & 1) ^ 1, abort_flag, p.status, kStatusWs2 | 5)) { ok = false; break; }
          if (!previous_done) {  // the request half must have finished before its rows are read
            griddep_wait();
            previous_done = true;
          }
          mbar_expect_tx(&z_full[zb], kZBufBytes);
#pragma unroll
          for (int q = 0; q < 4; ++q) tma_load_2d(z_smem + (zb * 4 + q) * BN, &map_z, &z_full[zb], n0, req_next[q]);
          if (st + p.groups < super_tiles) fetch_req(st + p.groups);
        }
      }
      if (!ok) {
        // Aborting: give the copies already in flight time to land before the CTA gives up its memory.
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only): a single thread -----------
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN, false, false);
      uint32_t it = 0, lt = 0;
      bool ok = mbar_wait(w_full, 0, abort_flag, p.status, kStatusWs2 | 6);
      const uint64_t b_desc0 = smem_desc_sw128(smem_u32(w_smem), 1024, 16);
      for (int32_t st = group; st < super_tiles && ok; st += p.groups, ++lt) {
        const uint32_t acc = lt & 1;
        if (!mbar_wait(&tmem_empty[acc], ((lt >> 1) & 1) ^ 1, abort_flag, p.status, kStatusWs2 | 2)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % p.a_stages;
          if (!mbar_wait(&a_full[s], (it / p.a_stages) & 1, abort_flag, p.status, kStatusWs2 | 3)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t a_desc = smem_desc_sw128(smem_u32(a_smem + s * kAStageBytes), 1024, 16);
          const uint64_t b_desc = b_desc0 + kb * (kWBlockBytes >> 4);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_ss_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&a_empty[s], 3);  // frees the stage in both CTAs
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
    const int q = warp % 4;             // TMEM lane quadrant = 32-row slab of this CTA's 128 rows
    const int half = (warp - 2) / 4;    // which 128 of the slice's 256 columns
    uint8_t* my_stage = staging + (warp - 2) * 4096;
    const uint32_t tmem_empty_leader[2] = {map_to_cta(smem_u32(&tmem_empty[0]), 0),
                                           map_to_cta(smem_u32(&tmem_empty[1]), 0)};
    uint32_t lt = 0;
    for (int32_t st = group; st < super_tiles; st += p.groups, ++lt) {
      const uint32_t acc = lt & 1;
      const int32_t m0 = st * 2 * BM + (int32_t)rank * BM;
      const int64_t row = (int64_t)m0 + q * 32 + lane;
      const float* zrow = nullptr;
      bool uniform = false;
      if (has_add) {
        const int64_t rc = max((int64_t)0, min(row, p.M - 1));
        const int32_t my_req = p.row2req ? p.row2req[rc] : (int32_t)rc;
        const int32_t slab_req = __shfl_sync(0xffffffffu, my_req, 0);
        uniform = __all_sync(0xffffffffu, my_req == slab_req);
        // shared-memory copy when this row belongs to the slab's first request, global otherwise
        zrow = (my_req == slab_req) ? (z_smem + ((lt % kZBufs) * 4 + q) * BN) : (p.add + (int64_t)my_req * p.ld_add + n0);
        if (!mbar_wait(&z_full[lt % kZBufs], (lt / kZBufs) & 1, abort_flag, p.status, kStatusWs2 | 7)) break;
      }
      if (!mbar_wait(&tmem_full[acc], (lt >> 1) & 1, abort_flag, p.status, kStatusWs2 | 4)) break;
      tc_fence_after_sync();
      // the TMA stores of the previous tile have finished reading this warp's staging boxes
      if (lane == 0) tma_store_wait_read<0>();
      __syncwarp();
      const uint32_t t_row = tmem_base + acc * BN + half * 128 + ((uint32_t)(q * 32) << 16);
      float st_sum = 0.f, st_sq = 0.f;  // this row's 128 output columns, for a normalisation that follows (Eq. 7)
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
          if (lane == 0) mbar_arrive_cluster_relaxed(tmem_empty_leader[acc]);
        }
        float f[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) f[i] = __uint_as_float(v[i]);
        if (has_add) {
          if (uniform) {
#pragma unroll
            for (int i = 0; i < 64; i += 4) {  // one broadcast read per 16 bytes (columns past d_out hold zeros)
              const float4 z = lds128(zrow + colL + i);
              f[i] += z.x; f[i + 1] += z.y; f[i + 2] += z.z; f[i + 3] += z.w;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 64; i += 4) {
              if (n0 + colL + i < p.d_out) {
                const float4 z = *reinterpret_cast<const float4*>(zrow + colL + i);
                f[i] += z.x; f[i + 1] += z.y; f[i + 2] += z.z; f[i + 3] += z.w;
              }
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
        if (p.stat_partials != nullptr) {  // columns past d_out hold zeros and add nothing
#pragma unroll
          for (int i = 0; i < 64; ++i) {
            st_sum += f[i];
            st_sq = fmaf(f[i], f[i], st_sq);
          }
        }
        if (c == 1) {  // the store of the first chunk has finished reading the box
          if (lane == 0) tma_store_wait_read<0>();
          __syncwarp();
        }
        uint8_t* row_ptr = my_stage + lane * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {  // eight 16-byte pieces per 128-byte row, XOR-swizzled by row
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
          if (n0 + half * 128 + c * 64 < p.d_out && (int64_t)m0 + q * 32 < p.M)
            tma_store_2d(&map_y, my_stage, n0 + half * 128 + c * 64, m0 + q * 32);
          tma_store_commit();
        }
      }
      if (p.stat_partials != nullptr && row < p.M)
        p.stat_partials[row * (2 * p.n_slices) + slice * 2 + half] = make_float2(st_sum, st_sq);
      if (lane == 0 && has_add) mbar_arrive(&z_empty[lt % kZBufs]);
    }
    if (lane == 0) tma_store_wait_all<0>();
  }

  tc_fence_before_sync();
  cluster_sync_all();  // neither CTA leaves while the pair's MMAs or remote arrivals may still touch it
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 2 * BN);
  }
}

int sm_count_ws2() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

}  // namespace

bool umma_linear_ws2_supported(int64_t M, int32_t d_in, int32_t d_out, bool out_f32) {
  if (out_f32 || d_in < 8 || d_in > 256 || d_out < 64 || d_out % 8 != 0) return false;
  if (M < 512 || M > 0x7fffff00LL) return false;
  return 2 * ((d_out + BN - 1) / BN) <= sm_count_ws2();
}

rocs_status_t umma_linear_ws2(int64_t M, int32_t d_in, int32_t d_out, const void* X, int64_t ld_x, const void* W,
                              int64_t ld_w, const float* bias, const float* add, int64_t ld_add,
                              const int32_t* row2req, int act, void* Y, int64_t ld_y, cudaStream_t stream,
                              bool add_from_previous_launch, float2* stat_partials, int64_t add_rows) {
  const int32_t k_blocks = (d_in + BK - 1) / BK;
  CUtensorMap map_x, map_w, map_z, map_y;
  if (!make_tensor_map_2d(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_in, (uint64_t)ld_x,
                          BM, BK, true) ||
      !make_tensor_map_2d(&map_w, W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)d_out, (uint64_t)d_in,
                          (uint64_t)ld_w, BN / 2, BK, true) ||
      !make_tensor_map_2d(&map_y, Y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)M, (uint64_t)d_out, (uint64_t)ld_y,
                          32, 64, true))
    return ROCS_ERR_CUDA;
  if (add != nullptr) {
    const int64_t z_rows = add_rows > 0 ? add_rows : M;   // a row past the last request reads as zero fill
    if (!make_tensor_map_2d(&map_z, add, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, (uint64_t)z_rows, (uint64_t)d_out,
                            (uint64_t)ld_add, 1, BN, false))
      return ROCS_ERR_CUDA;
  } else {
    map_z = map_x;
  }
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  Ws2Params p{};
  p.M = M; p.d_in = d_in; p.d_out = d_out;
  p.n_slices = (d_out + BN - 1) / BN;
  const int32_t super_tiles = (int32_t)((M + 2 * BM - 1) / (2 * BM));
  p.groups = std::max(1, std::min(super_tiles, (sm_count_ws2() / 2) / p.n_slices));
  const int fixed = k_blocks * kWBlockBytes + kStagingBytes + kZBufs * kZBufBytes + 512 + 1024;
  p.a_stages = std::min(10, (227 * 1024 - fixed) / kAStageBytes);
  p.bias = bias; p.add = add; p.ld_add = ld_add; p.row2req = row2req; p.act = act; p.status = status;
  p.wait_for_previous = (add_from_previous_launch && add != nullptr) ? 1 : 0;
  p.stat_partials = stat_partials;
  const int smem_bytes = fixed + p.a_stages * kAStageBytes;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(linear_ws2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * p.n_slices * p.groups);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.wait_for_previous ? 1 : 0;
  ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_ws2_kernel, map_x, map_w, map_z, map_y, p));
  return ROCS_OK;
}

}  // namespace rocs
