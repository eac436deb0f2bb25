// Group-wise cross attention, candidate side (Eq. 13), with the request's K/V shared inside the
// kernel (Section 4.3.1):  O[i,t,h,:] = softmax_j(scale <Q[i,t,h,:], K[r,j,h,:]>) V[r,j,h,:],  r = m_i.
//
// Candidates of one request are stacked in the tile M dimension: a work item is one head of one
// 128-row query tile of a request; K/V are addressed per request through seq_offsets and read in
// 128-key blocks, nothing is replicated per candidate (tiles of the same request and head are
// consecutive items, so their K/V blocks are read from L2 at about the same time).
//
// Head dimensions 64 (128-key blocks), 128 (64-key blocks: tensor memory holds S, P and O of both
// sides in 512 columns either way) and 32 (128-key blocks, operand rows of 64 bytes under the 64-byte
// swizzle); the description below gives the figures of the first.
//
// One persistent CTA per SM runs TWO independent item streams (sides A and B), 20 warps:
//   warps 16,19 TMA producers of sides A, B: the Q tile of the item, then (K_j, V_j) blocks through a ring
//   warps 17,18 tcgen05.mma issuers of sides A, B:  S = Q K_j^T (128x128x64, operands in shared memory)
//               and O += P V_j (128x64x128, P read from tensor memory, V from shared memory)
//   warps 0-15  softmax: 8 warps per side, TWO threads per query row, each owning 64 of the 128 key
//               columns of a block: S from TMEM into registers (one read), exp2 on scaled scores,
//               fp32 partial sums, P rounded to bf16 and stored to tensor memory.
// Tensor memory per side (256 columns): S [0,128) fp32, P [128,192) bf16 pairs, O [192,256) fp32.
// P has its own columns, so S_{j+1} is issued as soon as S_j sits in registers, and the wait on
// P V_{j-1} comes in the middle of block j, just before P_j starts to overwrite P_{j-1}.
//
// Reference of the softmax: the maximum of the row's FIRST block, rounded up to an integer, found
// by both threads of the row (each scans all 128 columns, so they agree bit for bit without
// talking) and never moved: later blocks need no maximum, no rescaling of O and no exchange.
// fp32 holds 2^x up to x = 128, so a row overflows only if a later score exceeds its first block's
// maximum by about 88 nats; such a row shows Inf/NaN in its sums at the end of the item and is then
// computed again by its two threads alone in plain fp32 loops (slow, correct, reached only by inputs
// whose scores span more than fp32's exponent range).  Every decision is taken per row from that
// row's own values, so a row's bits never depend on its neighbours.
#include <algorithm>

#include "rocs_internal.h"
#include "sm100_ptx.cuh"

#ifdef ROCS_DCA_TRACE
extern "C" void* rocs_dca_trace_buffer = nullptr;
#endif

namespace rocs {
namespace {

using namespace ptx;

constexpr int BQ = 128;           // query rows per tile
constexpr int kSoftmaxWarps = 16; // 8 per side
constexpr int kControlWarp0 = kSoftmaxWarps;   // warps 16, 19: TMA producers of sides A, B; 17, 18: their MMA issuers
constexpr int kThreads = (kSoftmaxWarps + 4) * 32;
constexpr int kTmemCols = 512;
constexpr uint32_t kStatusDca = 0x400;
constexpr int kSideTmemStride = 256;

// Everything that depends on the head dimension DH and the keys per block BKV.  Operand tiles are kept
// as boxes of 64 columns (128-byte rows, 128-byte swizzle): a tile of DH columns is DH / 64 boxes; a head
// dimension of 32 is one box of 32 columns (64-byte rows, 64-byte swizzle).
template <int DH_, int BKV_>
struct DcaCfg {
  static constexpr int DH = DH_, BKV = BKV_;
  static constexpr int kBoxCols = DH < 64 ? DH : 64;         // columns of a box = output columns per P V product
  static constexpr int kRowBytes = kBoxCols * 2;             // 128 or 64: also the swizzle span
  static constexpr int kBoxes = DH / kBoxCols;
  static_assert(kRowBytes == 128 || kRowBytes == 64, "operand rows");
  static constexpr int kCols = BKV / 2;                      // score columns per softmax thread
  static constexpr int kOutCols = DH / 2;                    // output columns per softmax thread
  static constexpr int kKvStages = DH == 128 ? 2 : DH == 64 ? 3 : 4;  // per side
  static constexpr int kQBoxBytes = BQ * kRowBytes, kQBytes = kBoxes * kQBoxBytes;
  static constexpr int kKvBoxBytes = BKV * kRowBytes, kKBytes = kBoxes * kKvBoxBytes;
  // operand descriptor of a tile of 8-row groups, rows of kRowBytes
  __device__ static uint64_t desc(uint32_t addr) {
    return kRowBytes == 128 ? smem_desc_sw128(addr, 1024, 16) : smem_desc_sw64(addr, 512, 16);
  }
  static constexpr int kKvStageBytes = 2 * kKBytes;          // K block + V block
  // tensor memory per side: S [0, BKV) fp32, P [BKV, BKV + BKV/2) bf16 pairs, O [.., + DH) fp32
  static constexpr int kPColOffset = BKV, kOColOffset = BKV + BKV / 2;
  static_assert(kOColOffset + DH <= kSideTmemStride, "tensor memory columns of a side");
  static_assert(kCols == 32 || kCols == 64, "score columns per thread");
  // Shared-memory map (byte offsets from the 1024-byte aligned base); per side: one Q tile (freed when
  // the item's last S is issued, a block before its end) and a ring of K/V stages.
  static constexpr uint32_t kOffQ = 0;                                          // [2 sides][boxes][128][64] bf16
  static constexpr uint32_t kOffKv = kOffQ + 2 * kQBytes;                       // [2 sides][stages][K | V]
  static constexpr uint32_t kOffL = kOffKv + 2 * kKvStages * kKvStageBytes;     // partial sums [2 sides][2 halves][128] fp32
  static constexpr uint32_t kOffBar = kOffL + 2 * 2 * BQ * 4;
  // barriers, 8 bytes each, [side] innermost where there are two
  static constexpr uint32_t kBarQFull = kOffBar;                    // [2]
  static constexpr uint32_t kBarQEmpty = kBarQFull + 16;            // [2]
  static constexpr uint32_t kBarKvFull = kBarQEmpty + 16;           // [2][stages]
  static constexpr uint32_t kBarKvEmpty = kBarKvFull + 16 * kKvStages;
  static constexpr uint32_t kBarSFull = kBarKvEmpty + 16 * kKvStages;  // [2]
  static constexpr uint32_t kBarSEmpty = kBarSFull + 16;
  static constexpr uint32_t kBarPFull = kBarSEmpty + 16;
  static constexpr uint32_t kBarOFull = kBarPFull + 16;
  static constexpr uint32_t kBarPair = kBarOFull + 16;              // [8]: the two warps that share 32 query rows
  static constexpr uint32_t kBarDrain = kBarPair + 64;              // [2]
  static constexpr uint32_t kOffTmemPtr = kBarDrain + 16;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 4;
  static constexpr int kSmemBytes = kOffAbort + 12;
  static_assert(kSmemBytes <= 232448, "shared memory of one SM");
};

#ifndef ROCS_DCA_EMU
#define ROCS_DCA_EMU 0
#endif
// Of every 8 column pairs of a row, this many take 2^x from a cubic on the FMA pipe instead of the
// exponential unit (which pairs is fixed by the column index, so a row's bits do not depend on its
// neighbours): 2^x = 2^n 2^r, n = round(x), |r| <= 1/2, 2^r by a polynomial with relative error
// 7.5e-5, far below the rounding of P to bf16.  Off by default: with the rest of the loop as it is
// the exponential unit is not what limits the kernel (measured).
constexpr int kEmuPairs = ROCS_DCA_EMU;
constexpr float kMagic = 12582912.f;  // 1.5 * 2^23: adding it rounds to an integer kept in the low mantissa bits
constexpr float kPoly0 = 0.9999280572f, kPoly1 = 0.6932609677f, kPoly2 = 0.2426111251f, kPoly3 = 0.0551716685f;

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
__device__ __forceinline__ float fmax_nan(float a, float b) {  // NaN if either input is NaN
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
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

__device__ __forceinline__ void tmem_st_32x32b_x8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// One query row of one head, half of its DH output columns, in plain fp32 with the row's true maximum
// as reference: q and k point at the head's DH values of the row / of the request's first key, v at the
// DH / 2 columns wanted; consecutive keys are `stride` elements apart.  Inlined on purpose: as a called
// function it forces the caller's hot loop to keep its registers where the calling convention wants
// them, and the loop spills.
template <int DH>
__device__ __forceinline__ void row_by_hand(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                            int32_t stride, int32_t L, float scale_log2e, __nv_bfloat16* out) {
  auto score = [&](int32_t j) {
    float s = 0.f;
    for (int d = 0; d < DH; ++d) s = fmaf(__bfloat162float(q[d]), __bfloat162float(k[(int64_t)j * stride + d]), s);
    return s * scale_log2e;
  };
  float m = -INFINITY;
  for (int32_t j = 0; j < L; ++j) m = fmaxf(m, score(j));
  float acc[DH / 2], l = 0.f;
  for (int d = 0; d < DH / 2; ++d) acc[d] = 0.f;
  for (int32_t j = 0; j < L; ++j) {
    const float pj = exp2f(score(j) - m);
    l += pj;
    for (int d = 0; d < DH / 2; ++d) acc[d] = fmaf(pj, __bfloat162float(v[(int64_t)j * stride + d]), acc[d]);
  }
  const float inv = 1.f / l;
  for (int d = 0; d < DH / 2; ++d) out[d] = __float2bfloat16_rn(acc[d] * inv);
}

// A short burst of probes before the paced wait: for hand-offs that are usually complete already.
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, AbortFlag* abort_flag, uint32_t* status,
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
#define TRACE_NEXT() ++tr_blk
#else
#define TRACE_EV(role, ev)
#define TRACE_NEXT()
#endif

template <int DH, int BKV>
__global__ void __launch_bounds__(kThreads, 1)
dca_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const DcaParams p) {
  using C = DcaCfg<DH, BKV>;
  constexpr int kKvStages = C::kKvStages, kBoxes = C::kBoxes, kCols = C::kCols, kOutCols = C::kOutCols;
  constexpr int kQBytes = C::kQBytes, kKBytes = C::kKBytes, kKvStageBytes = C::kKvStageBytes;
  constexpr int kPColOffset = C::kPColOffset, kOColOffset = C::kOColOffset;
  constexpr uint32_t kOffQ = C::kOffQ, kOffKv = C::kOffKv, kOffL = C::kOffL, kBarQFull = C::kBarQFull,
                     kBarQEmpty = C::kBarQEmpty, kBarKvFull = C::kBarKvFull, kBarKvEmpty = C::kBarKvEmpty,
                     kBarSFull = C::kBarSFull, kBarSEmpty = C::kBarSEmpty, kBarPFull = C::kBarPFull,
                     kBarOFull = C::kBarOFull, kBarPair = C::kBarPair, kBarDrain = C::kBarDrain,
                     kOffTmemPtr = C::kOffTmemPtr, kOffAbort = C::kOffAbort;
  extern __shared__ __align__(1024) uint8_t smem[];     // swizzled operand tiles need 1024-byte alignment
  const uint32_t sb = smem_u32(smem);                   // every shared-memory address below is sb + constant
  AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(smem + kOffAbort);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if ((sb & 1023u) != 0) {  // the swizzled tiles assume a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.status, 0u, kStatusDca | 15);
    return;
  }

  if (threadIdx.x == 0) {
    auto init = [&](uint32_t off, int n, uint32_t count) {
      for (int x = 0; x < n; ++x) mbar_init(reinterpret_cast<uint64_t*>(smem + off + 8 * x), count);
    };
    init(kBarQFull, 2, 1);
    init(kBarQEmpty, 2, 1);
    init(kBarKvFull, 2 * kKvStages, 1);
    init(kBarKvEmpty, 2 * kKvStages, 1);
    init(kBarSFull, 2, 1);
    init(kBarSEmpty, 2, kSoftmaxWarps / 2);
    init(kBarPFull, 2, kSoftmaxWarps / 2);
    init(kBarOFull, 2, 1);
    init(kBarPair, 8, 2);
    init(kBarDrain, 2, 1);
    abort_flag->v = 0;
    fence_mbar_init();
  }
  if (warp == kControlWarp0 + 1) {
    tmem_alloc(reinterpret_cast<uint32_t*>(smem + kOffTmemPtr), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *reinterpret_cast<const uint32_t*>(smem + kOffTmemPtr);
  // launched as a programmatic dependent: the set-up above may overlap the end of the kernel in front;
  // global memory is touched only from here on, and the kernel behind this one is released after the wait
  griddep_wait();
  griddep_launch_dependents();
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
      const uint32_t q_full = sb + kBarQFull + 8 * side, q_empty = sb + kBarQEmpty + 8 * side;
      const uint32_t kv_full = sb + kBarKvFull + 8 * kKvStages * side, kv_empty = sb + kBarKvEmpty + 8 * kKvStages * side;
      const uint32_t q_dst = sb + kOffQ + side * kQBytes, kv_dst = sb + kOffKv + side * kKvStages * kKvStageBytes;
      uint32_t kv_it = 0, n_work = 0;
      bool ok = true;
      for (int32_t i = item0 + side; i < p.num_items && ok; i += item_step) {
        const DcaItem item = p.items[i];
        const int32_t s0 = p.seq_offsets[item.req];
        const int32_t L = p.seq_offsets[item.req + 1] - s0;
        if (L == 0) continue;  // nobody touches a barrier for an item without keys
        if (!mbar_wait_paced(q_empty, (n_work & 1) ^ 1, abort_flag, p.status, kStatusDca | 1)) { ok = false; break; }
        ++n_work;
        mbar_expect_tx(q_full, kQBytes);
#pragma unroll
        for (int bx = 0; bx < kBoxes; ++bx)
          tma_load_2d(q_dst + bx * C::kQBoxBytes, &map_q, q_full, item.head * DH + bx * C::kBoxCols, item.cand0 * p.n_q);
        const int32_t nblk = (L + BKV - 1) / BKV;
        for (int32_t j = 0; j < nblk; ++j, ++kv_it) {
          const uint32_t s = kv_it % kKvStages;
          if (!mbar_wait_paced(kv_empty + 8 * s, ((kv_it / kKvStages) & 1) ^ 1, abort_flag, p.status, kStatusDca | 2)) { ok = false; break; }
          mbar_expect_tx(kv_full + 8 * s, kKvStageBytes);
#pragma unroll
          for (int bx = 0; bx < kBoxes; ++bx) {
            tma_load_2d(kv_dst + s * kKvStageBytes + bx * C::kKvBoxBytes, &map_k, kv_full + 8 * s,
                        item.head * DH + bx * C::kBoxCols, s0 + j * BKV);
            tma_load_2d(kv_dst + s * kKvStageBytes + kKBytes + bx * C::kKvBoxBytes, &map_v, kv_full + 8 * s,
                        item.head * DH + bx * C::kBoxCols, s0 + j * BKV);
          }
        }
      }
      if (!ok) {
        // let the loads in flight land before the CTA's shared memory goes away
        for (uint32_t s = 0; s < kKvStages; ++s) {
          const uint32_t n_issued = kv_it / kKvStages + ((kv_it % kKvStages > s) ? 1 : 0);
          if (n_issued == 0) continue;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait_brief(kv_full + 8 * s, (n_issued - 1) & 1) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp >= kControlWarp0) {
    // ------------------------------ MMA issuers: one warp per side ---------------------------
    const int side = warp - (kControlWarp0 + 1);
    constexpr uint32_t idesc_s = umma_idesc_bf16(BQ, BKV, false, false);  // S = Q K^T, both K-major
    constexpr uint32_t idesc_o = umma_idesc_bf16(BQ, C::kBoxCols, false, true);  // O = P V per box of output columns, V is MN-major
    const uint32_t q_full = sb + kBarQFull + 8 * side, q_empty = sb + kBarQEmpty + 8 * side;
    const uint32_t kv_full = sb + kBarKvFull + 8 * kKvStages * side, kv_empty = sb + kBarKvEmpty + 8 * kKvStages * side;
    const uint32_t s_full = sb + kBarSFull + 8 * side, s_empty = sb + kBarSEmpty + 8 * side;
    const uint32_t p_full = sb + kBarPFull + 8 * side, o_full = sb + kBarOFull + 8 * side;
    const uint32_t kv_base = sb + kOffKv + side * kKvStages * kKvStageBytes;
    uint32_t kv_it = 0, n_work = 0;           // n_work: items that had keys (phase of q_full)
    uint32_t cnt_p = 0, cnt_se = 0;           // phases of p_full and s_empty of this side
    bool ok = true;
#ifdef ROCS_DCA_TRACE
    int tr_blk = 0;
#endif
    const uint32_t t_s = tmem_base + side * kSideTmemStride;
    // Q tile of this side, K block and V block of a stage as shared-memory operand descriptors
    const uint64_t dq = C::desc(sb + kOffQ + side * kQBytes);
    auto desc_k = [&](uint32_t stage) { return C::desc(kv_base + stage * kKvStageBytes); };
    auto desc_v = [&](uint32_t stage) { return C::desc(kv_base + stage * kKvStageBytes + kKBytes); };
    auto issue_s = [&](uint64_t b_desc) {
#pragma unroll
      for (int k = 0; k < DH / 16; ++k) {  // 16 columns of dh per step: box k / kPerBox, 32 bytes further on inside it
        constexpr int kPerBox = C::kBoxCols / 16;
        umma_ss(t_s, dq + (k / kPerBox) * (C::kQBoxBytes >> 4) + 2 * (k % kPerBox),
                b_desc + (k / kPerBox) * (C::kKvBoxBytes >> 4) + 2 * (k % kPerBox), idesc_s, k != 0 ? 1u : 0u);
      }
      umma_commit(s_full);
    };
    auto issue_pv = [&](uint64_t b_desc, bool first_block) {
      // P: 16 keys = 8 columns of bf16 pairs in tensor memory
      // V: rows are keys (K), one row = a box of head dims (N): 16 keys = 16 rows further on
#pragma unroll
      for (int k = 0; k < BKV / 16; ++k)
#pragma unroll
        for (int bx = 0; bx < kBoxes; ++bx)  // one box of output columns per product
          umma_ts(t_s + kOColOffset + bx * C::kBoxCols, t_s + kPColOffset + k * 8,
                  b_desc + bx * (C::kKvBoxBytes >> 4) + k * (16 * C::kRowBytes / 16), idesc_o, (k != 0 || !first_block) ? 1u : 0u);
      umma_commit(o_full);
    };
    // The last block of a sequence may reach past it into the next request's rows (or past the
    // tensor, where TMA fills zeros).  Scores of such keys are masked to -inf by the softmax warps,
    // so P is exactly 0 there; the V rows are zeroed here so that 0 x (Inf or NaN of a foreign
    // request) cannot reach this request's output.
    auto zero_v_tail = [&](uint32_t stage, int32_t valid) {
      uint8_t* v = smem + kOffKv + (side * kKvStages + stage) * kKvStageBytes + kKBytes;
      for (int bx = 0; bx < kBoxes; ++bx)
        for (int idx = valid * (C::kRowBytes / 16) + lane; idx < BKV * (C::kRowBytes / 16); idx += 32)
          *reinterpret_cast<uint4*>(v + bx * C::kKvBoxBytes + idx * 16) = make_uint4(0u, 0u, 0u, 0u);
      fence_proxy_async_smem();
      __syncwarp();
    };
    for (int32_t i = item0 + side; i < p.num_items && ok; i += item_step) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      if (L == 0) continue;
      const int32_t nblk = (L + BKV - 1) / BKV;
      const int32_t tail_valid = L - (nblk - 1) * BKV;  // keys of the last block that exist
      if (!mbar_wait_paced(q_full, n_work & 1, abort_flag, p.status, kStatusDca | 3)) { ok = false; break; }
      ++n_work;
      // first key block (the S tile was drained at the end of the previous item)
      if (!mbar_wait_paced(kv_full + 8 * (kv_it % kKvStages), (kv_it / kKvStages) & 1, abort_flag, p.status, kStatusDca | 4)) { ok = false; break; }
      if (nblk == 1 && tail_valid < BKV) zero_v_tail(kv_it % kKvStages, tail_valid);
      tc_fence_after_sync();
      if (lane == 0) {
        issue_s(desc_k(kv_it % kKvStages));
        if (nblk == 1) umma_commit(q_empty);
      }
      __syncwarp();
      for (int32_t j = 0; j < nblk && ok; ++j, ++kv_it) {
        const uint32_t stage = kv_it % kKvStages;
        const uint32_t next_stage = (kv_it + 1) % kKvStages;
        const uint64_t dk_next = desc_k(next_stage), dv = desc_v(stage);
        TRACE_EV(2 + side, 0);
        if (j + 1 < nblk) {
          if (!mbar_wait_paced(kv_full + 8 * next_stage, ((kv_it + 1) / kKvStages) & 1, abort_flag, p.status, kStatusDca | 5)) { ok = false; break; }
          TRACE_EV(2 + side, 1);
          if (j + 2 == nblk && tail_valid < BKV) zero_v_tail(next_stage, tail_valid);
        }
        // S_{j+1} as soon as the side has pulled S_j into registers
        if (!mbar_wait_paced(s_empty, cnt_se & 1, abort_flag, p.status, kStatusDca | 11)) { ok = false; break; }
        ++cnt_se;
        TRACE_EV(2 + side, 2);
        if (j + 1 < nblk) {
          tc_fence_after_sync();
          if (lane == 0) {
            issue_s(dk_next);
            if (j + 2 == nblk) umma_commit(q_empty);  // last S of the item: the Q tile is free
          }
          __syncwarp();
          TRACE_EV(2 + side, 3);
        }
        // P_j of this side is in tensor memory
        if (!mbar_wait_paced(p_full, cnt_p & 1, abort_flag, p.status, kStatusDca | 6)) { ok = false; break; }
        ++cnt_p;
        TRACE_EV(2 + side, 4);
        tc_fence_after_sync();
        if (lane == 0) {
          issue_pv(dv, j == 0);
          umma_commit(kv_empty + 8 * stage);  // K_j and V_j are no longer needed
        }
        __syncwarp();
        TRACE_EV(2 + side, 5);
        TRACE_NEXT();
      }
    }
    if (!ok && lane == 0) {
      umma_commit(sb + kBarDrain + 8 * side);
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait_brief(sb + kBarDrain + 8 * side, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ------------------------------ softmax warps ------------------------------------------
    const int side = warp >> 3;
    const int half = (warp >> 2) & 1;       // which half of the block's key columns
    const int q = warp & 3;                 // TMEM lane quadrant this warp may touch
    const int row = q * 32 + lane;          // query row of the tile = TMEM lane
    const uint32_t t_row = tmem_base + side * kSideTmemStride + ((uint32_t)(q * 32) << 16);  // S columns of the row
    const uint32_t t_s = t_row + half * kCols;
    const uint32_t t_p = t_row + kPColOffset + half * (kCols / 2);
    const uint32_t t_o = t_row + kOColOffset + half * kOutCols;
    const uint32_t s_full = sb + kBarSFull + 8 * side, s_empty = sb + kBarSEmpty + 8 * side;
    const uint32_t p_full = sb + kBarPFull + 8 * side, o_full = sb + kBarOFull + 8 * side;
    const uint32_t my_pair = sb + kBarPair + 8 * (side * 4 + q);
    uint32_t cnt_s = 0, cnt_o = 0, cnt_pair = 0;
#ifdef ROCS_DCA_TRACE
    int tr_blk = 0;
    const int tr_role = warp == 0 ? 0 : warp == 8 ? 1 : -1;
#define TRACE_SM(ev) do { if (tr_role >= 0) TRACE_EV(tr_role, ev); } while (0)
#else
#define TRACE_SM(ev)
#endif
    for (int32_t i = item0 + side; i < p.num_items; i += item_step) {
      const DcaItem item = p.items[i];
      const int32_t L = p.seq_offsets[item.req + 1] - p.seq_offsets[item.req];
      const int32_t rows_valid = item.count_a * p.n_q;
      // this thread's half of the output columns of its row
      auto out_ptr = [&]() { return p.O + ((int64_t)item.cand0 * p.n_q + row) * row_width + item.head * DH + half * kOutCols; };
      bool aborted = false;
      if (L > 0) {
        const int32_t nblk = (L + BKV - 1) / BKV;
        // ---- reference of the row: the maximum of its first block, rounded up to an integer
        TRACE_SM(0);
        if (!mbar_wait_spin(s_full, cnt_s & 1, abort_flag, p.status, kStatusDca | 7)) break;
        tc_fence_after_sync();
        float m_ref;
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
        // the polynomial path: x = s c - m_ref with m_ref an integer, so n = round(x) comes out of one
        // fused multiply-add against kMagic - m_ref; scores are clamped from below at x = -126 (2^x is
        // nothing there) and must stay below x = 126, which is checked per block
        const float k_off = kMagic - m_ref;
        const float s_lo = (m_ref - 126.f) / p.scale_log2e;
        bool by_hand = kEmuPairs > 0 && !(fabsf(m_ref) < 1048576.f);  // kMagic - m_ref must be exact
        float g_max = -INFINITY;                     // largest raw score that went through the polynomial
        uint64_t sum2 = pack2(0.f, 0.f);
        for (int32_t j = 0; j < nblk; ++j) {
          if (j > 0) {
            TRACE_SM(0);
            if (!mbar_wait_spin(s_full, cnt_s & 1, abort_flag, p.status, kStatusDca | 7)) { aborted = true; break; }
            tc_fence_after_sync();
          }
          ++cnt_s;
          TRACE_SM(1);
          uint32_t sv[kCols];  // this thread's scores of the block
#pragma unroll
          for (int c = 0; c < kCols; c += 32) tmem_ld_32x32b_x32(t_s + c, sv + c);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty);  // S_{j+1} may overwrite the tile now
          const int32_t valid = L - j * BKV - half * kCols;  // columns of this thread's half that are keys of the request
          if (valid < kCols) {
#pragma unroll
            for (int e = 0; e < kCols; ++e)
              if (e >= valid) sv[e] = 0xff800000u;  // -inf: the key does not exist
          }
          TRACE_SM(2);
          uint32_t pk[kCols / 4];  // P of half of this thread's keys, bf16 pairs; stored in two halves
          auto store_p = [&](uint32_t taddr) {
            if constexpr (kCols == 64) tmem_st_32x32b_x16(taddr, pk); else tmem_st_32x32b_x8(taddr, pk);
          };
          auto exp_pair = [&](int e) {
            float p0, p1;
            if (((e >> 1) & 7) < kEmuPairs) {
              const uint64_t k2 = pack2(k_off, k_off);
              const float s0 = __uint_as_float(sv[e]), s1 = __uint_as_float(sv[e + 1]);
              g_max = fmax3(g_max, s0, s1);
              const uint64_t s2 = pack2(fmax_nan(s0, s_lo), fmax_nan(s1, s_lo));
              const uint64_t xf2 = ffma2(s2, c2, k2);                        // kMagic + n
              const uint64_t w2 = ffma2(xf2, pack2(-1.f, -1.f), k2);          // -(n + m_ref)
              const uint64_t r2 = ffma2(s2, c2, w2);                         // x - n
              uint64_t q2 = ffma2(r2, pack2(kPoly3, kPoly3), pack2(kPoly2, kPoly2));
              q2 = ffma2(q2, r2, pack2(kPoly1, kPoly1));
              q2 = ffma2(q2, r2, pack2(kPoly0, kPoly0));
              float q0, q1, f0, f1;
              unpack2(q2, q0, q1);
              unpack2(xf2, f0, f1);
              p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(f0) << 23));  // 2^r scaled by 2^n
              p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(f1) << 23));
            } else {
              float x0, x1;
              unpack2(ffma2(pack2(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1])), c2, m2), x0, x1);
              p0 = ex2(x0);
              p1 = ex2(x1);
            }
            sum2 = fadd2(sum2, pack2(p0, p1));
            pk[(e / 2) % (kCols / 4)] = bf16x2_bits(p0, p1);
          };
#pragma unroll
          for (int e = 0; e < kCols / 2; e += 2) exp_pair(e);
          TRACE_SM(3);
          if (j > 0) {
            // P V of the previous block has read P_{j-1} (it was issued most of a block ago): from here
            // on this thread's P columns may be rewritten
            if (!mbar_wait_spin(o_full, (cnt_o & 1) ^ 1, abort_flag, p.status, kStatusDca | 8)) { aborted = true; break; }
            tc_fence_after_sync();
          }
          ++cnt_o;
          TRACE_SM(4);
          store_p(t_p);
#pragma unroll
          for (int e = kCols / 2; e < kCols; e += 2) exp_pair(e);
          TRACE_SM(5);
          store_p(t_p + kCols / 4);
          if (kEmuPairs > 0 && g_max * p.scale_log2e - m_ref > 126.f) by_hand = true;  // 2^n would leave fp32's exponent field
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(p_full);
          TRACE_SM(6);
          TRACE_NEXT();
        }
        if (aborted) break;
        float sum_lo, sum_hi;
        unpack2(sum2, sum_lo, sum_hi);
        const float l_run = sum_lo + sum_hi;
        float* l_x = reinterpret_cast<float*>(smem + kOffL);
        l_x[(side * 2 + half) * BQ + row] = by_hand ? __int_as_float(0x7fc00000) : l_run;  // NaN tells the other half of the row too
        __syncwarp();
        if (lane == 0) mbar_arrive(my_pair);
        if (!mbar_wait_paced(my_pair, cnt_pair & 1, abort_flag, p.status, kStatusDca | 14) ||
            !mbar_wait_paced(o_full, (cnt_o & 1) ^ 1, abort_flag, p.status, kStatusDca | 9))
          break;
        ++cnt_pair;
        tc_fence_after_sync();
        const float l_o = l_x[(side * 2 + (half ^ 1)) * BQ + row];
        const float l_tot = half == 0 ? l_run + l_o : l_o + l_run;  // same order in both halves
        const float inv = 1.f / l_tot;
        uint32_t v[kOutCols];
        if constexpr (kOutCols == 16) {
          tmem_ld_32x32b_x16(t_o, v);
        } else {
#pragma unroll
          for (int c = 0; c < kOutCols; c += 32) tmem_ld_32x32b_x32(t_o + c, v + c);
        }
        tmem_ld_wait();
        // Scores that outgrow the first block's maximum by 2^128 or so overflow fp32 (and so can
        // a sum of products with huge values): the row then holds Inf or NaN instead of a result.
        float probe = l_tot * 0.f;
#pragma unroll
        for (int e = 0; e < kOutCols; ++e) probe = fmaf(__uint_as_float(v[e]), 0.f, probe);
        if (row < rows_valid) {
          __nv_bfloat16* out = out_ptr();
          if (probe == 0.f && !by_hand) {
#pragma unroll
            for (int e = 0; e < kOutCols; e += 8) {
              uint4 w;
              w.x = bf16x2_bits(__uint_as_float(v[e + 0]) * inv, __uint_as_float(v[e + 1]) * inv);
              w.y = bf16x2_bits(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
              w.z = bf16x2_bits(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv);
              w.w = bf16x2_bits(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv);
              *reinterpret_cast<uint4*>(out + e) = w;
            }
          } else {
            // such a row is computed again here, by this thread alone, with its true maximum as reference
            const int64_t q_row = (int64_t)item.cand0 * p.n_q + row;
            const int64_t kv0 = ((int64_t)p.seq_offsets[item.req] * p.H + item.head) * DH;
            row_by_hand<DH>(p.Q + q_row * row_width + item.head * DH, p.K + kv0, p.V + kv0 + half * kOutCols, row_width,
                            L, p.scale_log2e, out);
          }
        }
      } else if (row < rows_valid) {
        // a request without keys: zero rows
        __nv_bfloat16* out = out_ptr();
#pragma unroll
        for (int c = 0; c < kOutCols; c += 8) *reinterpret_cast<uint4*>(out + c) = make_uint4(0u, 0u, 0u, 0u);
      }
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
  return (dh == 32 || dh == 64 || dh == 128) && n_q >= 1 && n_q <= BQ && H >= 1 && H <= 65535;
}

template <int DH, int BKV>
static rocs_status_t launch_dca(const rocs_plan* plan, int32_t n_q, int32_t H, float scale, const void* Q,
                                const void* K, const void* V, const int32_t* seq_offsets, int64_t T, void* O,
                                cudaStream_t stream) {
  using C = DcaCfg<DH, BKV>;
  DcaItemList items;
  rocs_status_t st = plan_dca_items(plan, BQ / n_q, H, /*tiles_per_item=*/1, stream, &items);
  if (st != ROCS_OK) return st;
  if (items.num == 0) return ROCS_OK;
  const uint64_t width = (uint64_t)H * DH;
  CUtensorMap map_q, map_k, map_v;
  constexpr bool sw64 = C::kRowBytes == 64;
  if (!make_tensor_map_2d(&map_q, Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)plan->N * n_q, width, width, BQ,
                          C::kBoxCols, true, sw64))
    return ROCS_ERR_CUDA;
  if (T > 0) {
    if (!make_tensor_map_2d(&map_k, K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)T, width, width, BKV, C::kBoxCols,
                            true, sw64) ||
        !make_tensor_map_2d(&map_v, V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)T, width, width, BKV, C::kBoxCols,
                            true, sw64))
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
  auto kernel = dca_umma_kernel<DH, BKV>;
  ROCS_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
  const int grid = std::min((items.num + 1) / 2, sm_count_dca());  // one CTA per SM, two item streams per CTA
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ROCS_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_q, map_k, map_v, p));
  return ROCS_OK;
}

rocs_status_t umma_dca(const rocs_plan* plan, int32_t n_q, int32_t H, int32_t dh, float scale, const void* Q,
                       const void* K, const void* V, const int32_t* seq_offsets, int64_t T, void* O,
                       cudaStream_t stream) {
  if (plan->N == 0) return ROCS_OK;
  if (dh == 64) return launch_dca<64, 128>(plan, n_q, H, scale, Q, K, V, seq_offsets, T, O, stream);
  if (dh == 32) return launch_dca<32, 128>(plan, n_q, H, scale, Q, K, V, seq_offsets, T, O, stream);
  return launch_dca<128, 64>(plan, n_q, H, scale, Q, K, V, seq_offsets, T, O, stream);
}

}  // namespace rocs
