// Group-wise cross attention, candidate side (Eq. 13), with the request's K/V shared inside the
// kernel (Section 4.3.1):  O[i,t,h,:] = softmax_j(scale <Q[i,t,h,:], K[r,j,h,:]>) V[r,j,h,:],  r = m_i.
//
// Candidates of one request are stacked in the tile M dimension: a work item is one head of up to
// TWO 128-row query tiles (A and B) of the same request, so every 64-key block of K and V is loaded
// once and used by 256 query rows.  K/V are addressed per request through seq_offsets; nothing is
// replicated per candidate.
//
// Two persistent CTAs per SM (half the shared memory and half the TMEM columns each), so sixteen
// softmax warps keep the exponential unit fed while others wait on barriers.  Per CTA, 10 warps:
//   warp 0     TMA producer: Q tiles of the item, then (K_j, V_j) blocks of 64 keys through a ring
//   warp 1     tcgen05.mma issuer:  S_X = Q_X K_j^T  (128x64x64)  and  O_X = P_X V_j  (128x64x64)
//   warps 2-5  softmax group A,  warps 6-9  softmax group B: each thread owns one query row:
//              S from TMEM into registers (one read), reference max and sum in fp32 (exp2 on scaled
//              scores), P rounded to bf16 into shared memory (the A operand of the second MMA),
//              final 1/sum, bf16 store.
// O accumulates in TMEM across key blocks.  A row moves its reference max only when the block max
// exceeds it by more than 2^8; then O is rescaled in TMEM (read, multiply, write back) before the
// next P V is issued.  The decision is taken per row from that row's own scores; rows that keep
// their reference multiply by exactly 1, so a row's bits never depend on its neighbours.
// Q is double buffered and the producer runs one item ahead, so consecutive items overlap; the two
// groups run out of phase, so while one waits for its next S tile the other keeps the exponential
// unit busy.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr int DH = 64;            // head dimension handled here (128-byte rows)
constexpr int BQ = 128;           // query rows per tile
constexpr int BKV = 64;           // keys per block
constexpr int kThreads = 320;
constexpr int kKvStages = 3;
constexpr int kQSlots = 1;        // Q buffers per side (the second CTA on the SM covers the item change-over)
constexpr int kTmemCols = 256;    // per CTA; two CTAs share an SM
constexpr int kQBytes = BQ * DH * 2;          // 16 KB
constexpr int kKvStageBytes = 2 * BKV * DH * 2;  // K block + V block = 16 KB
constexpr int kPBytes = BQ * BKV * 2;         // 16 KB per side
constexpr int kSmemBytes = 2 * kQSlots * kQBytes + kKvStages * kKvStageBytes + 2 * kPBytes + 512;  // 1024-aligned base
constexpr float kRescaleThreshold = 8.f;  // log2 units
constexpr uint32_t kStatusDca = 0x400;
constexpr int kSideTmemStride = 128;  // side A: columns 0.., side B: columns 128..
constexpr int kOColOffset = BKV;      // S in [0, 64), O block in [64, 128) of the side

struct DcaParams {
  const DcaItem* items;
  int32_t num_items;
  int32_t n_q, H;
  float scale_log2e;  // scale * log2(e)
  const int32_t* seq_offsets;
  __nv_bfloat16* O;
  int64_t n_rows;     // N * n_q
  uint32_t* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed fp32 pairs (one instruction for two lanes of arithmetic) and the three-input maximum.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__global__ void __launch_bounds__(kThreads, 2)
dca_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const DcaParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];     // swizzled operand tiles need 1024-byte alignment
  uint8_t* q_smem = smem;                              // [slots][2 sides][128][64] bf16
  uint8_t* kv_smem = q_smem + 2 * kQSlots * kQBytes;   // [stages][K 8 KB | V 8 KB]
  uint8_t* p_smem = kv_smem + kKvStages * kKvStageBytes;  // [2][128 x 64] bf16, K-major swizzled
  uint64_t* q_full = reinterpret_cast<uint64_t*>(p_smem + 2 * kPBytes);  // [2]
  uint64_t* q_empty = q_full + 2;            // [2]
  uint64_t* kv_full = q_empty + 2;
  uint64_t* kv_empty = kv_full + kKvStages;
  uint64_t* s_full = kv_empty + kKvStages;   // [2]
  uint64_t* s_empty = s_full + 2;            // [2]
  uint64_t* p_full = s_empty + 2;            // [2]
  uint64_t* o_full = p_full + 2;             // [2]
  uint64_t* drain = o_full + 2;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles assume a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.status, 0u, kStatusDca | 15);
    return;
  }

  if (threadIdx.x == 0) {
    for (int x = 0; x < 2; ++x) {
      mbar_init(&q_full[x], 1);
      mbar_init(&q_empty[x], 1);
    }
    for (int s = 0; s < kKvStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(&s_full[x], 1);
      mbar_init(&s_empty[x], 4);
      mbar_init(&p_full[x], 4);
      mbar_init(&o_full[x], 1);
    }
    mbar_init(drain, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_ptr, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  const int32_t row_width = p.H * DH;  // elements per query / key row over all heads

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      uint32_t kv_it = 0, n_work = 0;
      bool ok = true;
      for (int32_t i = blockIdx.x; i < p.num_items && ok; i += gridDim.x) {
        const DcaItem item = p.items[i];
        const int32_t s0 = p.seq_offsets[item.req];
        const int32_t L = p.seq_offsets[item.req + 1] - s0;
        if (L == 0) continue;  // nobody touches a barrier for an item without keys
        const uint32_t slot = n_work % kQSlots;
        if (!mbar_wait_paced(&q_empty[slot], ((n_work / kQSlots) & 1) ^ 1, abort_flag, p.status, kStatusDca | 1)) { ok = false; break; }
        ++n_work;
        const int32_t sides = item.count_b > 0 ? 2 : 1;
        uint8_t* qs = q_smem + slot * 2 * kQBytes;
        mbar_expect_tx(&q_full[slot], sides * kQBytes);
        tma_load_2d(qs, &map_q, &q_full[slot], item.head * DH, item.cand0 * p.n_q);
        if (sides == 2) tma_load_2d(qs + kQBytes, &map_q, &q_full[slot], item.head * DH, (item.cand0 + item.count_a) * p.n_q);
        const int32_t nblk = (L + BKV - 1) / BKV;
        for (int32_t j = 0; j < nblk; ++j, ++kv_it) {
          const int s = kv_it % kKvStages;
          if (!mbar_wait_paced(&kv_empty[s], ((kv_it / kKvStages) & 1) ^ 1, abort_flag, p.status, kStatusDca | 2)) { ok = false; break; }
          uint8_t* st = kv_smem + s * kKvStageBytes;
          mbar_expect_tx(&kv_full[s], kKvStageBytes);
          tma_load_2d(st, &map_k, &kv_full[s], item.head * DH, s0 + j * BKV);
          tma_load_2d(st + BKV * DH * 2, &map_v, &kv_full[s], item.head * DH, s0 + j * BKV);
        }
      }
      if (!ok) {
        for (int s = 0; s < kKvStages; ++s) {
          const uint32_t n_issued = kv_it / kKvStages + (((int)(kv_it % kKvStages) > s) ? 1 : 0);
          if (n_issued == 0) continue;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&kv_full[s], (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ---------------------------------------------
    constexpr uint32_t idesc_s = umma_idesc_bf16(BQ, BKV, false, false);  // S = Q K^T, both K-major
    constexpr uint32_t idesc_o = umma_idesc_bf16(BQ, DH, false, true);    // O = P V, V is MN-major
    uint32_t kv_it = 0, n_work = 0;           // n_work: items that had keys (phase of q_full)
    uint32_t cnt_p[2] = {0, 0};               // phases of p_full per side
    bool ok = true;
    uint32_t cnt_se[2] = {0, 0};              // phases of s_empty per side
    auto issue_s = [&](int side, int stage, uint32_t slot) {
      const uint32_t d = tmem_base + side * kSideTmemStride;
      const uint64_t a_desc = smem_desc_sw128(smem_u32(q_smem + (slot * 2 + side) * kQBytes), 1024, 16);
      const uint64_t b_desc = smem_desc_sw128(smem_u32(kv_smem + stage * kKvStageBytes), 1024, 16);
#pragma unroll
      for (int k = 0; k < DH / 16; ++k) umma_ss(d, a_desc + 2 * k, b_desc + 2 * k, idesc_s, k != 0 ? 1u : 0u);
      umma_commit(&s_full[side]);
    };
    auto issue_pv = [&](int side, int stage, bool first_block) {
      const uint32_t d = tmem_base + side * kSideTmemStride + kOColOffset;
      const uint32_t p_addr = smem_u32(p_smem + side * kPBytes);
      const uint32_t v_addr = smem_u32(kv_smem + stage * kKvStageBytes + BKV * DH * 2);
#pragma unroll
      for (int k = 0; k < BKV / 16; ++k) {
        // P: K-major, one 64-key block (128 rows x 128 bytes), 32 bytes per 16 keys
        const uint64_t a_desc = smem_desc_sw128(p_addr + k * 32, 1024, 16);
        // V: rows are keys (K), 128 bytes = 64 head dims (N): 16 keys = 2048 bytes further on
        const uint64_t b_desc = smem_desc_sw128(v_addr + k * 16 * 128, 1024, 16);
        umma_ss(d, a_desc, b_desc, idesc_o, (k != 0 || !first_block) ? 1u : 0u);
      }
      umma_commit(&o_full[side]);
    };
    for (int32_t i = blockIdx.x; i < p.num_items && ok; i += gridDim.x) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      if (L == 0) continue;
      const int32_t sides = item.count_b > 0 ? 2 : 1;
      const int32_t nblk = (L + BKV - 1) / BKV;
      const uint32_t slot = n_work % kQSlots;
      if (!mbar_wait_paced(&q_full[slot], (n_work / kQSlots) & 1, abort_flag, p.status, kStatusDca | 3)) { ok = false; break; }
      ++n_work;
      // first key block: S for both sides (their S tiles were drained at the end of the previous item)
      if (!mbar_wait_paced(&kv_full[kv_it % kKvStages], (kv_it / kKvStages) & 1, abort_flag, p.status, kStatusDca | 4)) { ok = false; break; }
      tc_fence_after_sync();
      if (lane == 0) {
        for (int x = 0; x < sides; ++x) issue_s(x, kv_it % kKvStages, slot);
        if (nblk == 1) umma_commit(&q_empty[slot]);
      }
      __syncwarp();
      for (int32_t j = 0; j < nblk && ok; ++j, ++kv_it) {
        const int stage = kv_it % kKvStages;
        const int next_stage = (kv_it + 1) % kKvStages;
        if (j + 1 < nblk) {
          if (!mbar_wait_paced(&kv_full[next_stage], ((kv_it + 1) / kKvStages) & 1, abort_flag, p.status, kStatusDca | 5)) { ok = false; break; }
          // S_{j+1} as soon as the side has pulled S_j into registers
          for (int x = 0; x < sides; ++x) {
            if (!mbar_wait_paced(&s_empty[x], cnt_se[x] & 1, abort_flag, p.status, kStatusDca | 11)) { ok = false; break; }
            ++cnt_se[x];
            tc_fence_after_sync();
            if (lane == 0) issue_s(x, next_stage, slot);
            __syncwarp();
          }
          if (!ok) break;
          if (j + 2 == nblk && lane == 0) umma_commit(&q_empty[slot]);  // last S of the item: Q slot is free
          __syncwarp();
        } else {
          // keep the s_empty phases in step: the sides still signal after reading the last S
          for (int x = 0; x < sides; ++x) {
            if (!mbar_wait_paced(&s_empty[x], cnt_se[x] & 1, abort_flag, p.status, kStatusDca | 12)) { ok = false; break; }
            ++cnt_se[x];
          }
          if (!ok) break;
        }
        for (int x = 0; x < sides; ++x) {
          // P_j of this side is in shared memory (and O has been rescaled if it had to be)
          if (!mbar_wait_paced(&p_full[x], cnt_p[x] & 1, abort_flag, p.status, kStatusDca | 6)) { ok = false; break; }
          ++cnt_p[x];
          tc_fence_after_sync();
          if (lane == 0) issue_pv(x, stage, j == 0);
          __syncwarp();
        }
        if (ok && lane == 0) umma_commit(&kv_empty[stage]);  // K_j and V_j are no longer needed
        __syncwarp();
      }
    }
    if (!ok && lane == 0) {
      umma_commit(drain);
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(drain, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ------------------------------ softmax groups -----------------------------------------
    const int side = (warp - 2) / 4;
    const int q = warp % 4;                 // TMEM lane quadrant
    const int row = q * 32 + lane;          // query row of the tile = TMEM lane
    const uint32_t t_s = tmem_base + side * kSideTmemStride + ((uint32_t)(q * 32) << 16);
    const uint32_t t_o = t_s + kOColOffset;
    uint8_t* p_row = p_smem + side * kPBytes + row * 128;
    uint32_t cnt_s = 0, cnt_o = 0;
    for (int32_t i = blockIdx.x; i < p.num_items; i += gridDim.x) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      const int32_t my_count = side == 0 ? item.count_a : item.count_b;
      const int32_t cand_first = side == 0 ? item.cand0 : item.cand0 + item.count_a;
      const int32_t rows_valid = my_count * p.n_q;
      __nv_bfloat16* out = p.O + ((int64_t)cand_first * p.n_q + row) * row_width + item.head * DH;
      bool aborted = false;
      float m_ref = -INFINITY, l_run = 0.f;
      if (my_count > 0 && L > 0) {
        const int32_t nblk = (L + BKV - 1) / BKV;
        for (int32_t j = 0; j < nblk; ++j) {
          const int32_t valid = min(BKV, L - j * BKV);  // keys of this block that exist
          if (!mbar_wait_paced(&s_full[side], cnt_s & 1, abort_flag, p.status, kStatusDca | 7)) { aborted = true; break; }
          ++cnt_s;
          tc_fence_after_sync();
          uint32_t sv[BKV];
#pragma unroll
          for (int c = 0; c < BKV; c += 32) tmem_ld_32x32b_x32(t_s + c, sv + c);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s_empty[side]);  // S_{j+1} may overwrite the tile now
          if (valid < BKV) {
#pragma unroll
            for (int e = 0; e < BKV; ++e)
              if (e >= valid) sv[e] = 0xff800000u;  // -inf: the key does not exist
          }
          float mx4[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) mx4[u] = fmaxf(__uint_as_float(sv[2 * u]), __uint_as_float(sv[2 * u + 1]));
#pragma unroll
          for (int e = 8; e < BKV; e += 2)  // four short chains of three-input maxima
            mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
          float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          mx *= p.scale_log2e;
          // this row's own decision: move the reference only for a jump of more than 2^8
          const bool move = mx > m_ref + kRescaleThreshold;
          const float m_new = move ? mx : m_ref;
          const float alpha = move ? ex2(m_ref - m_new) : 1.f;  // 0 on the first block
          m_ref = m_new;
          if (j > 0) {
            // P V of the previous block is complete: O is stable and P's buffer may be rewritten
            if (!mbar_wait_paced(&o_full[side], cnt_o & 1, abort_flag, p.status, kStatusDca | 8)) { aborted = true; break; }
            ++cnt_o;
            tc_fence_after_sync();
            if (__any_sync(0xffffffffu, move)) {
#pragma unroll
              for (int c = 0; c < DH; c += 16) {
                uint32_t v[16];
                tmem_ld_32x32b_x16(t_o + c, v);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                tmem_st_32x32b_x16(t_o + c, v);
              }
              tmem_st_wait();
            }
          }
          const uint64_t c2 = pack2(p.scale_log2e, p.scale_log2e), m2 = pack2(-m_new, -m_new);
          uint64_t sum2 = pack2(0.f, 0.f);
#pragma unroll
          for (int c = 0; c < BKV; c += 8) {
            float pe[8];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              float x0, x1;
              unpack2(ffma2(pack2(__uint_as_float(sv[c + e]), __uint_as_float(sv[c + e + 1])), c2, m2), x0, x1);
              pe[e] = ex2(x0);
              pe[e + 1] = ex2(x1);
              sum2 = fadd2(sum2, pack2(pe[e], pe[e + 1]));
            }
            uint4 w;
            __nv_bfloat162 h2;
            h2 = __floats2bfloat162_rn(pe[0], pe[1]); w.x = *reinterpret_cast<uint32_t*>(&h2);
            h2 = __floats2bfloat162_rn(pe[2], pe[3]); w.y = *reinterpret_cast<uint32_t*>(&h2);
            h2 = __floats2bfloat162_rn(pe[4], pe[5]); w.z = *reinterpret_cast<uint32_t*>(&h2);
            h2 = __floats2bfloat162_rn(pe[6], pe[7]); w.w = *reinterpret_cast<uint32_t*>(&h2);
            // 8 keys = one 16-byte chunk of this row
            *reinterpret_cast<uint4*>(p_row + (((c / 8) ^ (row & 7)) << 4)) = w;
          }
          float sum_lo, sum_hi;
          unpack2(sum2, sum_lo, sum_hi);
          const float sum = sum_lo + sum_hi;
          l_run = l_run * alpha + sum;
          fence_proxy_async_smem();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_full[side]);
        }
        if (!aborted) {
          if (!mbar_wait_paced(&o_full[side], cnt_o & 1, abort_flag, p.status, kStatusDca | 9)) {
            aborted = true;
          } else {
            ++cnt_o;
            tc_fence_after_sync();
            const float inv = 1.f / l_run;
#pragma unroll
            for (int c = 0; c < DH; c += 32) {
              uint32_t v[32];
              tmem_ld_32x32b_x32(t_o + c, v);
              tmem_ld_wait();
              if (row < rows_valid) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                  uint4 w;
                  __nv_bfloat162 h2;
                  h2 = __floats2bfloat162_rn(__uint_as_float(v[e + 0]) * inv, __uint_as_float(v[e + 1]) * inv); w.x = *reinterpret_cast<uint32_t*>(&h2);
                  h2 = __floats2bfloat162_rn(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv); w.y = *reinterpret_cast<uint32_t*>(&h2);
                  h2 = __floats2bfloat162_rn(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv); w.z = *reinterpret_cast<uint32_t*>(&h2);
                  h2 = __floats2bfloat162_rn(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv); w.w = *reinterpret_cast<uint32_t*>(&h2);
                  *reinterpret_cast<uint4*>(out + c + e) = w;
                }
              }
            }
          }
        }
      } else if (my_count > 0 && row < rows_valid) {
        // a request without keys: zero rows
#pragma unroll
        for (int c = 0; c < DH; c += 8) *reinterpret_cast<uint4*>(out + c) = make_uint4(0u, 0u, 0u, 0u);
      }
      if (aborted) break;
      tc_fence_before_sync();  // the next item's first P V overwrites O
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

int sm_count_dca() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

}  // namespace

bool umma_dca_supported(int32_t n_q, int32_t H, int32_t dh) {
  return dh == DH && n_q >= 1 && n_q <= BQ && H >= 1 && H <= 65535;
}

rocs_status_t umma_dca(const rocs_plan* plan, int32_t n_q, int32_t H, int32_t dh, float scale, const void* Q,
                       const void* K, const void* V, const int32_t* seq_offsets, int64_t T, void* O,
                       cudaStream_t stream) {
  (void)dh;
  if (plan->N == 0) return ROCS_OK;
  DcaItemList items;
  rocs_status_t st = plan_dca_items(plan, BQ / n_q, H, stream, &items);
  if (st != ROCS_OK) return st;
  if (items.num == 0) return ROCS_OK;
  const uint64_t width = (uint64_t)H * DH;
  CUtensorMap map_q, map_k, map_v;
  if (!make_tensor_map_2d(&map_q, Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)plan->N * n_q, width, width, BQ, DH,
                          true))
    return ROCS_ERR_CUDA;
  if (T > 0) {
    if (!make_tensor_map_2d(&map_k, K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)T, width, width, BKV, DH, true) ||
        !make_tensor_map_2d(&map_v, V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)T, width, width, BKV, DH, true))
      return ROCS_ERR_CUDA;
  } else {
    map_k = map_q;  // every sequence is empty: the kernel only writes zeros
    map_v = map_q;
  }
  uint32_t* status = device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  DcaParams p{};
  p.items = items.dev;
  p.num_items = items.num;
  p.n_q = n_q;
  p.H = H;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.seq_offsets = seq_offsets;
  p.O = (__nv_bfloat16*)O;
  p.n_rows = plan->N * n_q;
  p.status = status;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(dca_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  const int grid = std::min(items.num, 2 * sm_count_dca());  // two CTAs per SM
  dca_umma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_q, map_k, map_v, p);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
