// Group-wise cross attention, candidate side (Eq. 13), with the request's K/V shared inside the
// kernel (Section 4.3.1):  O[i,t,h,:] = softmax_j(scale <Q[i,t,h,:], K[r,j,h,:]>) V[r,j,h,:],  r = m_i.
//
// Candidates of one request are stacked in the tile M dimension: a work item is one head of up to
// TWO 128-row query tiles (sides A and B) of the same request, so every 128-key block of K and V is
// loaded once and used by 256 query rows.  K/V are addressed per request through seq_offsets;
// nothing is replicated per candidate.
//
// One persistent CTA per SM, 20 warps:
//   warp 16     TMA producer: Q tiles of the item (double buffered, one item ahead), then
//               (K_j, V_j) blocks of 128 keys through a ring
//   warps 17,18 tcgen05.mma issuers, one per side:  S_X = Q_X K_j^T (128x128x64, operands in shared
//               memory) and O_X += P_X V_j (128x64x128, P read from tensor memory, V from shared memory)
//   warps 0-15  softmax: 8 warps per side, TWO threads per query row, each owning 64 of the 128
//               key columns of a block: S from TMEM into registers (one read), block maximum
//               (the two halves of a row exchange theirs through shared memory), exp2 on scaled
//               scores, fp32 partial sums, P rounded to bf16 and stored to tensor memory.
// Tensor memory per side (256 columns): S [0,128) fp32, P [128,192) bf16 pairs, O [192,256) fp32.
// P has its own columns, so S_{j+1} is issued as soon as S_j sits in registers and the only wait
// on P V_{j-1} comes after the exponentials of block j, just before P_j overwrites P_{j-1}: no
// product and no hand-shake is on the softmax warps' critical path, they run back to back on the
// exponential unit while the tensor pipe works one block ahead (S) and one behind (P V).
//
// O accumulates in TMEM across key blocks.  A row keeps an integer-valued reference maximum and
// moves it only when a block maximum exceeds it by more than 2^8; then O is rescaled in TMEM
// before the next P V is issued.  The decision is taken per row from that row's own scores; rows
// that keep their reference multiply by exactly 1, so a row's bits never depend on its neighbours.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

#ifdef ROCS_DCA_TRACE
extern "C" void* rocs_dca_trace_buffer = nullptr;
#endif

namespace rocs {
namespace {

using namespace ptx;

constexpr int DH = 64;            // head dimension handled here (128-byte rows)
constexpr int BQ = 128;           // query rows per tile
constexpr int BKV = 128;          // keys per block
constexpr int kSoftmaxWarps = 16; // 8 per side
constexpr int kControlWarp0 = kSoftmaxWarps;   // warps 16, 19: TMA producers of sides A, B; 17, 18: their MMA issuers
constexpr int kThreads = (kSoftmaxWarps + 4) * 32;
constexpr int kKvStages = 3;        // per side
constexpr int kQSlots = 1;         // Q buffers per side (freed when the item's last S is issued, a block before its end)
constexpr int kTmemCols = 512;
constexpr int kQBytes = BQ * DH * 2;            // 16 KB
constexpr int kKBytes = BKV * DH * 2;           // 16 KB
constexpr int kKvStageBytes = 2 * kKBytes;      // K block + V block
constexpr int kXchgBytes = 2 * 2 * BQ * 4;  // partial sums of the two halves of a row [side][half][row]
constexpr int kNumBarriers = 2 * (2 * kQSlots + 2 * kKvStages) + 8 + 8 + 2;
constexpr int kSmemBytes = 2 * (kQSlots * kQBytes + kKvStages * kKvStageBytes) + kXchgBytes + kNumBarriers * 8 + 16;
constexpr float kRescaleThreshold = 8.f;  // log2 units
constexpr uint32_t kStatusDca = 0x400;
constexpr int kSideTmemStride = 256;
constexpr int kPColOffset = 128;
constexpr int kOColOffset = 192;

struct DcaParams {
  const DcaItem* items;
  int32_t num_items;
  int32_t n_q, H;
  float scale_log2e;  // scale * log2(e)
  const int32_t* seq_offsets;
  const __nv_bfloat16 *Q, *K, *V;  // plain pointers for rows that are computed by hand
  __nv_bfloat16* O;
  uint32_t* status;
#ifdef ROCS_DCA_TRACE
  long long* trace;
#endif
};

__device__ __forceinline__ float ex2(float x) {
#ifdef ROCS_DCA_PROBE_NOEXP
  return x * 0.001f;  // timing probe only: wrong results
#else
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
#endif
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
__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi) {
  const __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h2);
}

// D[tmem] (+)= A[tmem] * B[smem]: A holds bf16 pairs in 32-bit columns (16 keys = 8 columns).
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x32b_x32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
      "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
      "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

// One query row of one head, 32 of its 64 output columns, in plain fp32 with the row's true maximum as
// reference: q and k point at the head's 64 values of the row / of the request's first key, v at the
// 32 columns wanted; consecutive keys are `stride` elements apart.
__device__ __forceinline__ void row_by_hand(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                         int32_t stride, int32_t L, float scale_log2e, __nv_bfloat16* out) {
  auto score = [&](int32_t j) {
    float s = 0.f;
    for (int d = 0; d < DH; ++d) s = fmaf(__bfloat162float(q[d]), __bfloat162float(k[(int64_t)j * stride + d]), s);
    return s * scale_log2e;
  };
  float m = -INFINITY;
  for (int32_t j = 0; j < L; ++j) m = fmaxf(m, score(j));
  float acc[32], l = 0.f;
  for (int d = 0; d < 32; ++d) acc[d] = 0.f;
  for (int32_t j = 0; j < L; ++j) {
    const float pj = exp2f(score(j) - m);
    l += pj;
    for (int d = 0; d < 32; ++d) acc[d] = fmaf(pj, __bfloat162float(v[(int64_t)j * stride + d]), acc[d]);
  }
  const float inv = 1.f / l;
  for (int d = 0; d < 32; ++d) out[d] = __float2bfloat16_rn(acc[d] * inv);
}

// A short burst of probes before the paced wait: for hand-offs that complete within a few dozen cycles.
__device__ __forceinline__ bool mbar_wait_spin(uint64_t* bar, uint32_t parity, AbortFlag* abort_flag, uint32_t* status,
                                               uint32_t code) {
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait_brief(bar, parity)) return true;
  return mbar_wait_paced(bar, parity, abort_flag, status, code);
}

#ifdef ROCS_DCA_TRACE
// event stamps of CTA 0: [role 0..3][block 0..kTraceBlocks)[event 0..8)
constexpr int kTraceBlocks = 96;
#define TRACE_EV(role, ev) do { if (p.trace && blockIdx.x == 0 && lane == 0 && tr_blk < kTraceBlocks) p.trace[((role) * kTraceBlocks + tr_blk) * 8 + (ev)] = clock64(); } while (0)
#else
#define TRACE_EV(role, ev)
#endif

__global__ void __launch_bounds__(kThreads, 1)
dca_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const DcaParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];     // swizzled operand tiles need 1024-byte alignment
  uint8_t* q_smem = smem;                                // [2 sides][slots][128][64] bf16
  uint8_t* kv_smem = q_smem + 2 * kQSlots * kQBytes;     // [2 sides][stages][K 16 KB | V 16 KB]
  float* l_x = reinterpret_cast<float*>(kv_smem + 2 * kKvStages * kKvStageBytes);  // [2 sides][2 halves][128]
  uint64_t* q_full = reinterpret_cast<uint64_t*>(l_x + 2 * 2 * BQ);  // [2 sides][slots]
  uint64_t* q_empty = q_full + 2 * kQSlots;      // [2][slots]
  uint64_t* kv_full = q_empty + 2 * kQSlots;     // [2][stages]
  uint64_t* kv_empty = kv_full + 2 * kKvStages;  // [2][stages]
  uint64_t* s_full = kv_empty + 2 * kKvStages;   // [2]
  uint64_t* s_empty = s_full + 2;            // [2]
  uint64_t* p_full = s_empty + 2;            // [2]
  uint64_t* o_full = p_full + 2;             // [2]
  uint64_t* pair_bar = o_full + 2;           // [8]: the two warps that share 32 query rows
  uint64_t* drain = pair_bar + 8;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(drain + 2);
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles assume a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.status, 0u, kStatusDca | 15);
    return;
  }

  if (threadIdx.x == 0) {
    for (int x = 0; x < 2 * kQSlots; ++x) {
      mbar_init(&q_full[x], 1);
      mbar_init(&q_empty[x], 1);
    }
    for (int s = 0; s < 2 * kKvStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(&s_full[x], 1);
      mbar_init(&s_empty[x], kSoftmaxWarps / 2);
      mbar_init(&p_full[x], kSoftmaxWarps / 2);
      mbar_init(&o_full[x], 1);
    }
    for (int x = 0; x < 8; ++x) mbar_init(&pair_bar[x], 2);
    mbar_init(&drain[0], 1);
    mbar_init(&drain[1], 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == kControlWarp0 + 1) {
    tmem_alloc(tmem_ptr, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  const int32_t row_width = p.H * DH;  // elements per query / key row over all heads

  // Each side is a stream of its own: items 2 b + side, 2 b + side + 2 grid, ... of CTA b.
  const int32_t item0 = 2 * (int32_t)blockIdx.x, item_step = 2 * (int32_t)gridDim.x;

  if (warp == kControlWarp0 || warp == kControlWarp0 + 3) {
    // ------------------------------ TMA producers: one warp per side --------------------------
    const int side = warp == kControlWarp0 ? 0 : 1;
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      uint64_t* qf = q_full + side * kQSlots;
      uint64_t* qe = q_empty + side * kQSlots;
      uint64_t* kf = kv_full + side * kKvStages;
      uint64_t* ke = kv_empty + side * kKvStages;
      uint8_t* kv_side = kv_smem + side * kKvStages * kKvStageBytes;
      uint32_t kv_it = 0, n_work = 0;
      bool ok = true;
      for (int32_t i = item0 + side; i < p.num_items && ok; i += item_step) {
        const DcaItem item = p.items[i];
        const int32_t s0 = p.seq_offsets[item.req];
        const int32_t L = p.seq_offsets[item.req + 1] - s0;
        if (L == 0) continue;  // nobody touches a barrier for an item without keys
        const uint32_t slot = n_work % kQSlots;
        if (!mbar_wait_paced(&qe[slot], ((n_work / kQSlots) & 1) ^ 1, abort_flag, p.status, kStatusDca | 1)) { ok = false; break; }
        ++n_work;
        mbar_expect_tx(&qf[slot], kQBytes);
        tma_load_2d(q_smem + (side * kQSlots + slot) * kQBytes, &map_q, &qf[slot], item.head * DH, item.cand0 * p.n_q);
        const int32_t nblk = (L + BKV - 1) / BKV;
        for (int32_t j = 0; j < nblk; ++j, ++kv_it) {
          const int s = kv_it % kKvStages;
          if (!mbar_wait_paced(&ke[s], ((kv_it / kKvStages) & 1) ^ 1, abort_flag, p.status, kStatusDca | 2)) { ok = false; break; }
          uint8_t* st = kv_side + s * kKvStageBytes;
          mbar_expect_tx(&kf[s], kKvStageBytes);
          tma_load_2d(st, &map_k, &kf[s], item.head * DH, s0 + j * BKV);
          tma_load_2d(st + kKBytes, &map_v, &kf[s], item.head * DH, s0 + j * BKV);
        }
      }
      if (!ok) {
        // let the loads in flight land before the CTA's shared memory goes away
        for (int s = 0; s < kKvStages; ++s) {
          const uint32_t n_issued = kv_it / kKvStages + (((int)(kv_it % kKvStages) > s) ? 1 : 0);
          if (n_issued == 0) continue;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&kf[s], (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp >= kControlWarp0) {
    // ------------------------------ MMA issuers: one warp per side ---------------------------
    const int side = warp - (kControlWarp0 + 1);
    constexpr uint32_t idesc_s = umma_idesc_bf16(BQ, BKV, false, false);  // S = Q K^T, both K-major
    constexpr uint32_t idesc_o = umma_idesc_bf16(BQ, DH, false, true);    // O = P V, V is MN-major
    uint64_t* qf = q_full + side * kQSlots;
    uint64_t* qe = q_empty + side * kQSlots;
    uint64_t* kf = kv_full + side * kKvStages;
    uint64_t* ke = kv_empty + side * kKvStages;
    uint8_t* kv_side = kv_smem + side * kKvStages * kKvStageBytes;
    uint32_t kv_it = 0, n_work = 0;           // n_work: items that had keys (phase of q_full)
    uint32_t cnt_p = 0, cnt_se = 0;           // phases of p_full and s_empty of this side
    bool ok = true;
#ifdef ROCS_DCA_TRACE
    int tr_blk = 0;
#endif
    const uint32_t t_s = tmem_base + side * kSideTmemStride;
    // Descriptors are formed by the whole warp ahead of the barrier waits; the elected lane then only
    // issues the products.
    auto desc_q = [&](uint32_t slot) { return smem_desc_sw128(smem_u32(q_smem + (side * kQSlots + slot) * kQBytes), 1024, 16); };
    auto desc_k = [&](int stage) { return smem_desc_sw128(smem_u32(kv_side + stage * kKvStageBytes), 1024, 16); };
    auto desc_v = [&](int stage) { return smem_desc_sw128(smem_u32(kv_side + stage * kKvStageBytes + kKBytes), 1024, 16); };
    auto issue_s = [&](uint64_t a_desc, uint64_t b_desc) {
#pragma unroll
      for (int k = 0; k < DH / 16; ++k) umma_ss(t_s, a_desc + 2 * k, b_desc + 2 * k, idesc_s, k != 0 ? 1u : 0u);
      umma_commit(&s_full[side]);
    };
    auto issue_pv = [&](uint64_t b_desc, bool first_block) {
      // P: 16 keys = 8 columns of bf16 pairs in tensor memory
      // V: rows are keys (K), 128 bytes = 64 head dims (N): 16 keys = 2048 bytes further on
#pragma unroll
      for (int k = 0; k < BKV / 16; ++k)
        umma_ts(t_s + kOColOffset, t_s + kPColOffset + k * 8, b_desc + k * (16 * 128 / 16), idesc_o,
                (k != 0 || !first_block) ? 1u : 0u);
      umma_commit(&o_full[side]);
    };
    // The last block of a sequence may reach past it into the next request's rows (or past the
    // tensor, where TMA fills zeros).  Scores of such keys are masked to -inf by the softmax warps,
    // so P is exactly 0 there; the V rows are zeroed here so that 0 x (Inf or NaN of a foreign
    // request) cannot reach this request's output.
    auto zero_v_tail = [&](int stage, int32_t valid) {
      uint8_t* v = kv_side + stage * kKvStageBytes + kKBytes;
      for (int idx = valid * 8 + lane; idx < BKV * 8; idx += 32)
        *reinterpret_cast<uint4*>(v + idx * 16) = make_uint4(0u, 0u, 0u, 0u);
      fence_proxy_async_smem();
      __syncwarp();
    };
    for (int32_t i = item0 + side; i < p.num_items && ok; i += item_step) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      if (L == 0) continue;
      const int32_t nblk = (L + BKV - 1) / BKV;
      const int32_t tail_valid = L - (nblk - 1) * BKV;  // keys of the last block that exist
      const uint32_t slot = n_work % kQSlots;
      if (!mbar_wait_paced(&qf[slot], (n_work / kQSlots) & 1, abort_flag, p.status, kStatusDca | 3)) { ok = false; break; }
      ++n_work;
      // first key block (the S tile was drained at the end of the previous item)
      if (!mbar_wait_paced(&kf[kv_it % kKvStages], (kv_it / kKvStages) & 1, abort_flag, p.status, kStatusDca | 4)) { ok = false; break; }
      if (nblk == 1 && tail_valid < BKV) zero_v_tail(kv_it % kKvStages, tail_valid);
      tc_fence_after_sync();
      const uint64_t dq = desc_q(slot);
      if (lane == 0) {
        issue_s(dq, desc_k(kv_it % kKvStages));
        if (nblk == 1) umma_commit(&qe[slot]);
      }
      __syncwarp();
      for (int32_t j = 0; j < nblk && ok; ++j, ++kv_it) {
        const int stage = kv_it % kKvStages;
        const int next_stage = (kv_it + 1) % kKvStages;
        const uint64_t dk_next = desc_k(next_stage), dv = desc_v(stage);
        TRACE_EV(2 + side, 0);
        if (j + 1 < nblk) {
          if (!mbar_wait_paced(&kf[next_stage], ((kv_it + 1) / kKvStages) & 1, abort_flag, p.status, kStatusDca | 5)) { ok = false; break; }
          TRACE_EV(2 + side, 1);
          if (j + 2 == nblk && tail_valid < BKV) zero_v_tail(next_stage, tail_valid);
        }
        // S_{j+1} as soon as the side has pulled S_j into registers
        if (!mbar_wait_paced(&s_empty[side], cnt_se & 1, abort_flag, p.status, kStatusDca | 11)) { ok = false; break; }
        ++cnt_se;
        TRACE_EV(2 + side, 2);
        if (j + 1 < nblk) {
          tc_fence_after_sync();
          if (lane == 0) {
            issue_s(dq, dk_next);
            if (j + 2 == nblk) umma_commit(&qe[slot]);  // last S of the item: Q slot is free
          }
          __syncwarp();
          TRACE_EV(2 + side, 3);
        }
        // P_j of this side is in tensor memory
        if (!mbar_wait_paced(&p_full[side], cnt_p & 1, abort_flag, p.status, kStatusDca | 6)) { ok = false; break; }
        ++cnt_p;
        TRACE_EV(2 + side, 4);
        tc_fence_after_sync();
        if (lane == 0) {
          issue_pv(dv, j == 0);
          umma_commit(&ke[stage]);  // K_j and V_j are no longer needed
        }
        __syncwarp();
        TRACE_EV(2 + side, 5);
#ifdef ROCS_DCA_TRACE
        ++tr_blk;
#endif
      }
    }
    if (!ok && lane == 0) {
      umma_commit(&drain[side]);
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(&drain[side], 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ------------------------------ softmax warps ------------------------------------------
    const int sw = warp;
    const int side = sw >> 3;
    const int half = (sw >> 2) & 1;         // which 64 of the block's 128 key columns
    const int q = warp & 3;                 // TMEM lane quadrant this warp may touch
    const int row = q * 32 + lane;          // query row of the tile = TMEM lane
    const uint32_t t_side = tmem_base + side * kSideTmemStride + ((uint32_t)(q * 32) << 16);
    const uint32_t t_s = t_side + half * 64;
    const uint32_t t_row = t_side;                   // all 128 S columns of the row
    const uint32_t t_p = t_side + kPColOffset + half * 32;
    const uint32_t t_o = t_side + kOColOffset + half * 32;
    uint64_t* my_pair = &pair_bar[side * 4 + q];
    uint32_t cnt_s = 0, cnt_o = 0, cnt_pair = 0;
#ifdef ROCS_DCA_TRACE
    int tr_blk = 0;
    const int tr_role = sw == 0 ? 0 : sw == 8 ? 1 : -1;
#define TRACE_SM(ev) do { if (tr_role >= 0) TRACE_EV(tr_role, ev); } while (0)
#else
#define TRACE_SM(ev)
#endif
    for (int32_t i = item0 + side; i < p.num_items; i += item_step) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      const int32_t my_count = item.count_a;
      const int32_t cand_first = item.cand0;
      const int32_t rows_valid = my_count * p.n_q;
      const int32_t head = item.head;
      auto out_ptr = [&]() { return p.O + ((int64_t)cand_first * p.n_q + row) * row_width + head * DH + half * 32; };
      bool aborted = false;
      if (my_count > 0 && L > 0) {
        const int32_t nblk = (L + BKV - 1) / BKV;
        float m_ref, l_run = 0.f;
        // ---- reference of the row: the maximum of its first block, rounded up to an integer.
        // Both threads of a row scan all 128 columns, so they get bitwise the same value without
        // talking to each other.  It is never moved: later blocks use the same reference, whatever
        // their scores (see the end of the item for rows whose scores grow past fp32's range).
        TRACE_SM(0);
        if (!mbar_wait_spin(&s_full[side], cnt_s & 1, abort_flag, p.status, kStatusDca | 7)) { aborted = true; break; }
        tc_fence_after_sync();
        {
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < BKV; c += 32) {
            uint32_t ov[32];
            tmem_ld_32x32b_x32(t_row + c, ov);
            tmem_ld_wait();
            if (L < c + 32) {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (c + e >= L) ov[e] = 0xff800000u;  // -inf: the key does not exist
            }
#pragma unroll
            for (int e = 0; e < 32; e += 2)  // four short chains of three-input maxima
              mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], __uint_as_float(ov[e]), __uint_as_float(ov[e + 1]));
          }
          m_ref = ceilf(fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2e);
        }
        const uint64_t c2 = pack2(p.scale_log2e, p.scale_log2e), m2 = pack2(-m_ref, -m_ref);
        uint64_t sum2 = pack2(0.f, 0.f);
        for (int32_t j = 0; j < nblk; ++j) {
          if (j > 0) {
            TRACE_SM(0);
            if (!mbar_wait_spin(&s_full[side], cnt_s & 1, abort_flag, p.status, kStatusDca | 7)) { aborted = true; break; }
            tc_fence_after_sync();
          }
          ++cnt_s;
          TRACE_SM(1);
          uint32_t sv[64];  // this thread's 64 scores of the block
          tmem_ld_32x32b_x32(t_s, sv);
          tmem_ld_32x32b_x32(t_s + 32, sv + 32);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s_empty[side]);  // S_{j+1} may overwrite the tile now
          const int32_t valid = L - j * BKV - half * 64;  // columns of this thread's half that are keys of the request
          if (valid < 64) {
#pragma unroll
            for (int e = 0; e < 64; ++e)
              if (e >= valid) sv[e] = 0xff800000u;  // -inf: the key does not exist
          }
          TRACE_SM(2);
          uint32_t pk[16];  // P of 32 keys of this row, bf16 pairs; stored in two halves
          auto exp_pair = [&](int e) {
            float x0, x1;
            unpack2(ffma2(pack2(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1])), c2, m2), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            sum2 = fadd2(sum2, pack2(p0, p1));
            pk[(e / 2) & 15] = bf16x2_bits(p0, p1);
          };
#pragma unroll
          for (int e = 0; e < 32; e += 2) exp_pair(e);
          TRACE_SM(3);
          if (j > 0) {
            // P V of the previous block has read P_{j-1} (it was issued most of a block ago): from here
            // on this thread's P columns may be rewritten
            if (!mbar_wait_spin(&o_full[side], cnt_o & 1, abort_flag, p.status, kStatusDca | 8)) { aborted = true; break; }
            ++cnt_o;
            tc_fence_after_sync();
          }
          TRACE_SM(4);
          tmem_st_32x32b_x16(t_p, pk);
#pragma unroll
          for (int e = 32; e < 64; e += 2) exp_pair(e);
          TRACE_SM(5);
          tmem_st_32x32b_x16(t_p + 16, pk);
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_full[side]);
          TRACE_SM(6);
#ifdef ROCS_DCA_TRACE
          ++tr_blk;
#endif
        }
        if (!aborted) {
          float sum_lo, sum_hi;
          unpack2(sum2, sum_lo, sum_hi);
          l_run = sum_lo + sum_hi;
          float* l_mine = l_x + (side * 2 + half) * BQ + row;
          const float* l_other = l_x + (side * 2 + (half ^ 1)) * BQ + row;
          *l_mine = l_run;
          __syncwarp();
          if (lane == 0) mbar_arrive(my_pair);
          if (!mbar_wait_paced(my_pair, cnt_pair & 1, abort_flag, p.status, kStatusDca | 14) ||
              !mbar_wait_paced(&o_full[side], cnt_o & 1, abort_flag, p.status, kStatusDca | 9)) {
            aborted = true;
          } else {
            ++cnt_pair;
            ++cnt_o;
            tc_fence_after_sync();
            const float l_o = *l_other;
            const float l_tot = half == 0 ? l_run + l_o : l_o + l_run;  // same order in both halves
            const float inv = 1.f / l_tot;
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_o, v);
            tmem_ld_wait();
            // Scores that outgrow the first block's maximum by 2^128 or so overflow fp32 (and so can
            // a sum of products with huge values): the row then holds Inf or NaN instead of a result.
            float probe = l_tot * 0.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) probe = fmaf(__uint_as_float(v[e]), 0.f, probe);
            if (row < rows_valid) {
              __nv_bfloat16* out = out_ptr();
              if (probe == 0.f) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                  uint4 w;
                  w.x = bf16x2_bits(__uint_as_float(v[e + 0]) * inv, __uint_as_float(v[e + 1]) * inv);
                  w.y = bf16x2_bits(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
                  w.z = bf16x2_bits(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv);
                  w.w = bf16x2_bits(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv);
                  *reinterpret_cast<uint4*>(out + e) = w;
                }
              } else {
                // such a row is computed again here, by this thread alone, with a reference that is
                // its true maximum (plain fp32 loops over the request's keys: slow, and reached only
                // by inputs whose scores span more than fp32's exponent range)
                const int64_t q_row = (int64_t)cand_first * p.n_q + row;
                row_by_hand(p.Q + q_row * row_width + head * DH, p.K + ((int64_t)p.seq_offsets[item.req] * p.H + head) * DH,
                            p.V + ((int64_t)p.seq_offsets[item.req] * p.H + head) * DH + half * 32, row_width, L,
                            p.scale_log2e, out);
              }
            }
          }
        }
      } else if (my_count > 0 && row < rows_valid) {
        // a request without keys: zero rows
        __nv_bfloat16* out = out_ptr();
#pragma unroll
        for (int c = 0; c < 32; c += 8) *reinterpret_cast<uint4*>(out + c) = make_uint4(0u, 0u, 0u, 0u);
      }
      if (aborted) break;
      tc_fence_before_sync();  // the next item's first P V overwrites O
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == kControlWarp0 + 1) {
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
  rocs_status_t st = plan_dca_items(plan, BQ / n_q, H, /*tiles_per_item=*/1, stream, &items);
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
  p.Q = (const __nv_bfloat16*)Q;
  p.K = (const __nv_bfloat16*)K;
  p.V = (const __nv_bfloat16*)V;
  p.O = (__nv_bfloat16*)O;
  p.status = status;
#ifdef ROCS_DCA_TRACE
  p.trace = (long long*)rocs_dca_trace_buffer;
#endif
  ROCS_CUDA_TRY(cudaFuncSetAttribute(dca_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  const int grid = std::min((items.num + 1) / 2, sm_count_dca());  // one CTA per SM, two item streams per CTA
  dca_umma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_q, map_k, map_v, p);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}

}  // namespace rocs
