// Decode GEMV (M <= 8) against packed RaZeR weights for sm_100a: TMA-fed register-fragment kernel.
//
//   y[m, n] = bf16( ts * sum_k x[m, k] * D1[n, k] ),   D1 = block_scale * element (exact bf16)
//
// The path is bound by the instructions that decode the 4.5-bit weights, so everything around the decode is
// kept off the decoding warps: one producer warp moves packed weights and activations into a shared-memory
// ring with bulk copies (cp.async.bulk + mbarrier, no per-lane copy instructions), one epilogue warp adds the
// warps' partial sums, writes y and runs the cross-CTA combination, and the CW consumer warps only wait for a
// stage, decode their slice of it in registers (razer_decode.cuh) and feed it to warp-level m16n8k16 MMAs as
// the A fragment (B fragment = the activation slice, 8 tokens along n; FP32 accumulators).  Sec. 4.3 of the
// paper describes this fragment-matched style for its weight-only kernel; App. E its partition.
//
// Work: a unit is TM strips of 16 weight rows over the whole of K; a slice is one unit x one 64-column chunk.
// A stage of the ring holds CW consecutive slices of one unit (one per consumer warp) and the matching
// activation columns.  Two CTAs fit on an SM (half the shared memory and registers each), so that the CTAs of
// the next launch in the stream become resident, fill their rings and wait (programmatic dependent launch)
// while this launch drains.
// Partition (host, stream_plan): either every CTA takes whole units only, or every CTA takes q whole units
// and the remaining units are cut along K into equal slice ranges, one range per CTA, processed FIRST: a
// unit shared by several CTAs is combined through FP32 slots in the workspace by the last CTA to arrive (one
// counter per unit, slots added in CTA order: a fixed summation order), which then happens in the shadow of
// the whole units that follow.  This is the stripe partition with a global reduction of Sec. 4.3 / App. E,
// arranged so that the reduction is off the critical path.
//
// Every wait is bounded: on expiry the thread records a code in the workspace status word and the CTA drains
// its copies and exits.
#include <cuda.h>
#include <algorithm>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_decode.cuh"
#include "razer_ptx.cuh"

namespace razer {

namespace stream_path {

#ifndef STREAM_CW
#define STREAM_CW 8
#endif
constexpr int CW = STREAM_CW;                       // consumer warps; a stage holds CW * SPW slices, SPW per warp
constexpr int THREADS = 32 * (CW + 2);              // + producer warp + epilogue warp
constexpr int MAX_STAGES = 8;
constexpr int MAX_M = 8;
#ifndef STREAM_OCC
#define STREAM_OCC 2
#endif
#ifndef STREAM_TABLE_SHIFT
#define STREAM_TABLE_SHIFT 2
#endif
constexpr int OCC = STREAM_OCC;                     // CTAs per SM the kernel is built for
constexpr int TABLE_SHIFT = STREAM_TABLE_SHIFT;     // 1: 16 copies of each entry, 2: 8 copies, 3: 4 copies
constexpr int TABLE_COPIES = 32 >> TABLE_SHIFT;
constexpr int TABLE_BYTES = 256 * TABLE_COPIES * 8; // 256 scale bytes x copies x {scale, special value}
constexpr int RED_STRIDE = 36;                      // floats per (warp, token) in the partial-sum buffers
constexpr int SLOT_FLOATS = 32 * MAX_M;             // one CTA's partial result of a unit
constexpr int SMEM_BYTES = (OCC == 2 ? 112 : 74) * 1024;   // OCC CTAs per SM (each also holds 1 KB of system shared memory)
constexpr int BAR_BYTES = (2 * MAX_STAGES + 4) * 8 + 32;

template <int TM, int SPW>
struct Cfg {
  static constexpr int ROWS = 16 * TM;
  static constexpr int CPS = CW * SPW;                     // chunks (slices) per stage
  static constexpr int STRIP_BYTES = CPS * PIECE_BYTES;    // one strip's pieces of a stage
  static constexpr int W_BYTES = TM * STRIP_BYTES;         // weights of a stage
  static constexpr int XS = CPS * 128 + 16;                // bytes between tokens in a stage (16 mod 128: no bank conflicts)
  static_assert(XS % 16 == 0, "bulk copies land on 16-byte boundaries");
};

struct Args {
  const uint8_t* packed;
  const __nv_bfloat16* x;    // [M][K]
  __nv_bfloat16* y;          // [M][N]
  float* slots;              // [grid][SLOT_FLOATS]
  uint32_t* counters;        // one per split unit, zero between calls
  uint32_t* status;          // device status word
  const float* extra_scale;  // optional device scalar multiplied into the tensor scale
  int N, K, kc, M;
  int units;                 // units of TM strips that hold rows < N
  int whole_base, whole_per_cta;   // CTA b owns the whole units whole_base + b * whole_per_cta .. (clipped to units)
  int rem_ctas;              // CTAs that share the split units [0, whole_base): pieces_per_unit each; 0 = nothing is split
  int pieces_per_unit;       // a split unit is cut along K into this many equal pieces, one per CTA
  float sv0, sv1, tensor_scale;
  uint32_t mul_lo, mul_hi;   // 2^6 + 2^12 and 2^2 + 2^8 (razer_decode.cuh)
};

// D (+)= A(16 x 16, row) * B(16 x 8, col), bf16 inputs, FP32 accumulation.
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <int OFF>
__device__ __forceinline__ uint32_t lds16_at(uint32_t base) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1+%2];" : "=r"(v) : "r"(base), "n"(OFF) : "memory");
  return v;
}
template <int OFF>
__device__ __forceinline__ uint2 lds64_at(uint32_t base) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(base), "n"(OFF) : "memory");
  return v;
}
template <int OFF>
__device__ __forceinline__ uint4 lds128_at(uint32_t base) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4+%5];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(base), "n"(OFF)
               : "memory");
  return v;
}
__device__ __forceinline__ void sts128_zero(uint32_t addr) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One segment of a CTA's work: chunks [c0, c1) of one unit.
struct Seg {
  int unit, c0, c1;
};

// A CTA's list of segments: at most one piece of a split unit, then its whole units.
struct Work {
  int n_rem, n_seg;
  int u0, a0, a1;            // the piece of a split unit: unit, chunk range
  int wu0;                   // first whole unit
  int kc;
  __device__ __forceinline__ Seg seg(int i) const {
    Seg s;
    if (i < n_rem) {
      s.unit = u0; s.c0 = a0; s.c1 = a1;
    } else {
      s.unit = wu0 + (i - n_rem);
      s.c0 = 0;
      s.c1 = kc;
    }
    return s;
  }
};

__device__ __forceinline__ Work make_work(const Args& a, int b) {
  Work w;
  w.kc = a.kc;
  w.n_rem = 0;
  w.u0 = w.a0 = w.a1 = 0;
  if (b < a.rem_ctas) {
    // piece j of unit u: chunks [kc j / p, kc (j + 1) / p)
    w.u0 = b / a.pieces_per_unit;
    const int j = b - w.u0 * a.pieces_per_unit;
    w.a0 = (a.kc * j) / a.pieces_per_unit;
    w.a1 = (a.kc * (j + 1)) / a.pieces_per_unit;
    w.n_rem = 1;
  }
  w.wu0 = a.whole_base + b * a.whole_per_cta;
  int n_whole = a.units - w.wu0;
  n_whole = n_whole < 0 ? 0 : (n_whole > a.whole_per_cta ? a.whole_per_cta : n_whole);
  w.n_seg = w.n_rem + n_whole;
  return w;
}

// Four stored nibbles of each 16-bit half of `w` -> four bf16x2 registers (elements 2p, 2p + 1 of the word in
// register p), each the exact product value x scale with the block's sign.  The special value is the one
// nibble that is numerically zero when the isolated nibble is read as a bf16 pair: relu(nibble * -2^11 + sv')
// is sv' = sv x 2^-126 for it and 0 for every other nibble (the smallest, 2^-133, times 2^11 already exceeds
// the largest sv').
__device__ __forceinline__ void decode_word2(uint32_t w, uint32_t ss2, uint32_t svp, uint32_t mul_lo, uint32_t mul_hi,
                                             uint32_t* out) {
  constexpr uint32_t NEG = 0xC500C500u;               // (-2048, -2048) as bf16x2
  const uint32_t w8 = w >> 8;
  const uint32_t n0 = w & 0x000F000Fu, n1 = w & 0x00F000F0u;
  const uint32_t n2 = w8 & 0x000F000Fu, n3 = w8 & 0x00F000F0u;
  const uint32_t u0 = and_or(n0 * mul_lo, 0x81C081C0u, fma_relu_bf16x2(n0, NEG, svp));
  const uint32_t u1 = and_or(n1 * mul_hi, 0x81C081C0u, fma_relu_bf16x2(n1, NEG, svp));
  const uint32_t u2 = and_or(n2 * mul_lo, 0x81C081C0u, fma_relu_bf16x2(n2, NEG, svp));
  const uint32_t u3 = and_or(n3 * mul_hi, 0x81C081C0u, fma_relu_bf16x2(n3, NEG, svp));
  out[0] = mul_bf16x2(u0, ss2);
  out[1] = mul_bf16x2(u1, ss2);
  out[2] = mul_bf16x2(u2, ss2);
  out[3] = mul_bf16x2(u3, ss2);
}

// Wait for a barrier phase.  One cheap poll first; the slow path looks at the clock and the abort flag only once
// per 32 polls and, for the service warps (SLEEP_NS > 0), sleeps between polls, so that a waiting warp costs the
// decoding warps few issue slots.
template <int SLEEP_NS>
__device__ __noinline__ bool wait_phase_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  const uint64_t t0 = global_ns();
  for (uint32_t i = 0; i < (WAIT_LIMIT >> 5); ++i) {
#pragma unroll 1
    for (int j = 0; j < 32; ++j) {
      if (mbar_try_wait(bar, parity)) return true;
      if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    }
    if (*abort_flag) return false;
    if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
  }
  return false;
}
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_phase_slow<SLEEP_NS>(bar, parity, abort_flag);
}

// Per-lane constants of the consumer's reads from a stage.
struct LaneView {
  uint32_t h0, h1;           // code words of rows g and g + 8 of block t (offset inside the warp's piece)
  uint32_t sc;               // the two scale bytes of those blocks
  uint32_t xo;               // the lane's 16 activation columns of token g
  uint32_t tbl;              // (table address | lane copy * 8) << TABLE_SHIFT: the scale byte is dropped into bits 15:8
};

// One strip (16 rows) of one slice: decode the lane's two blocks, four MMAs (into one accumulator: separate
// accumulators per MMA measured no faster).
template <int OFF>
__device__ __forceinline__ void strip_step(float (&acc)[4], uint32_t piece, const LaneView& v, uint32_t mul_lo,
                                           uint32_t mul_hi, const uint32_t (&xq)[4][2]) {
  const uint2 c0 = lds64_at<OFF>(piece + v.h0), c1 = lds64_at<OFF>(piece + v.h1);
  const uint32_t sb = lds16_at<OFF>(piece + v.sc);
  // table entry of a scale byte b: table + (b * copies + copy) * 8 = {+-scale x 2^126, special value x 2^-126}
  const uint2 t0 = lds64(__byte_perm(sb, v.tbl, 0x7604) >> TABLE_SHIFT);
  const uint2 t1 = lds64(__byte_perm(sb, v.tbl, 0x7614) >> TABLE_SHIFT);
  uint32_t e0[8], e1[8];
  decode_word2(c0.x, t0.x, t0.y, mul_lo, mul_hi, e0);
  decode_word2(c0.y, t0.x, t0.y, mul_lo, mul_hi, e0 + 4);
  decode_word2(c1.x, t1.x, t1.y, mul_lo, mul_hi, e1);
  decode_word2(c1.y, t1.x, t1.y, mul_lo, mul_hi, e1 + 4);
#pragma unroll
  for (int q = 0; q < 4; ++q) mma_16816(acc, e0[2 * q], e1[2 * q], e0[2 * q + 1], e1[2 * q + 1], xq[q][0], xq[q][1]);
}

// The warp's slices J, J + 1, .. SPW - 1 of a stage (slice j is chunk c + j * CW): activation fragment, then decode
// + MMA for each of the unit's strips, fully unrolled with every shared-memory offset an immediate (a rolled
// loop over the slices, with or without loading a slice ahead, measured 6 to 15 % slower).
// CHECKED: the stage is the last of a segment and may hold fewer slices.
template <int TM, int SPW, int J, bool CHECKED>
__device__ __forceinline__ void slice_steps(float (&acc)[TM][4], uint32_t st, const LaneView& v, int c, int c1,
                                            uint32_t mul_lo, uint32_t mul_hi) {
  if constexpr (J < SPW) {
    if (!CHECKED || c + J * CW < c1) {
      uint32_t xq[4][2];
      const uint4 xa = lds128_at<J * CW * 128>(st + v.xo), xb = lds128_at<J * CW * 128 + 16>(st + v.xo);
      xq[0][0] = xa.x, xq[0][1] = xa.y, xq[1][0] = xa.z, xq[1][1] = xa.w;
      xq[2][0] = xb.x, xq[2][1] = xb.y, xq[3][0] = xb.z, xq[3][1] = xb.w;
      strip_step<J * CW * PIECE_BYTES>(acc[0], st, v, mul_lo, mul_hi, xq);
      if (TM == 2) strip_step<Cfg<TM, SPW>::STRIP_BYTES + J * CW * PIECE_BYTES>(acc[TM - 1], st, v, mul_lo, mul_hi, xq);
    }
    slice_steps<TM, SPW, J + 1, CHECKED>(acc, st, v, c, c1, mul_lo, mul_hi);
  }
}

template <int TM, int SPW>
__global__ void __launch_bounds__(THREADS, OCC) razer_stream_kernel(const Args a) {
  using C = Cfg<TM, SPW>;
  constexpr int CPS = C::CPS, XS = C::XS;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __shared__ uint32_t abort_word, never_set;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x;
  const Work work = make_work(a, b);

  // ---- carve the dynamic shared memory: the decode table sits on a 32 KB boundary of the shared window; the
  // barriers and partial-sum buffers go in front of it, ring stages fill what is left before and behind it ----
  const uint32_t base = smem_addr(smem_raw);
  const uint32_t table = (base + TABLE_BYTES - 1) & ~(uint32_t)(TABLE_BYTES - 1);
  uint32_t lo0 = base, lo1 = table, hi0 = table + TABLE_BYTES, hi1 = base + SMEM_BYTES;
  const uint32_t red_bytes = 2u * CW * a.M * RED_STRIDE * 4u;
  const uint32_t fixed = (BAR_BYTES + red_bytes + 15u) & ~15u;
  const uint32_t stage_bytes = (uint32_t)C::W_BYTES + (uint32_t)a.M * XS;
  uint32_t fixed_at;
  bool layout_ok = hi1 >= hi0 && table >= base;
  if (layout_ok && lo1 - lo0 >= fixed) { fixed_at = lo0; lo0 += fixed; }
  else { fixed_at = hi0; hi0 += fixed; layout_ok = layout_ok && hi0 <= hi1; }
  const int n_lo = layout_ok ? (int)((lo1 - lo0) / stage_bytes) : 0;
  const int n_hi = layout_ok ? (int)((hi1 - hi0) / stage_bytes) : 0;
  const int stages = min(MAX_STAGES, n_lo + n_hi);
  auto stage_addr = [&](int s) -> uint32_t { return s < n_lo ? lo0 + (uint32_t)s * stage_bytes : hi0 + (uint32_t)(s - n_lo) * stage_bytes; };
  const uint32_t bar_full = fixed_at, bar_empty = bar_full + 8 * MAX_STAGES;
  const uint32_t bar_red_full = bar_empty + 8 * MAX_STAGES, bar_red_free = bar_red_full + 16;
  const uint32_t red = fixed_at + BAR_BYTES;                 // [2][CW][M][RED_STRIDE] floats
  volatile uint32_t* abort_flag = &abort_word;

  // ---- producer state: stage k of this CTA's work (k counts stages over all segments) is (segment, first chunk) ----
  const size_t strip_run = (size_t)a.kc * PIECE_BYTES;        // bytes of one strip's K run
  struct Walk { int seg_i, c, c1, unit, slot, phase; };
  auto walk_start = [&](Walk& w) {
    w.seg_i = 0; w.slot = 0; w.phase = 0; w.c = w.c1 = w.unit = 0;
    if (work.n_seg > 0) { const Seg s = work.seg(0); w.c = s.c0; w.c1 = s.c1; w.unit = s.unit; }
  };
  auto walk_next = [&](Walk& w) {
    w.c += CPS;
    if (w.c >= w.c1 && ++w.seg_i < work.n_seg) { const Seg s = work.seg(w.seg_i); w.c = s.c0; w.c1 = s.c1; w.unit = s.unit; }
    if (++w.slot == stages) { w.slot = 0; w.phase ^= 1; }
  };
  auto issue_w = [&](const Walk& w) {
    const uint32_t st = stage_addr(w.slot), bar = bar_full + 8 * w.slot;
    const int n = min(CPS, w.c1 - w.c);
    const uint32_t wb = (uint32_t)n * PIECE_BYTES;
    const uint32_t xb = (uint32_t)min(n * CHUNK_K, a.K - w.c * CHUNK_K) * 2u, full = (uint32_t)n * 128u;
    if (xb < full) {
      // K ends inside the stage's last chunk: the columns beyond it multiply zero blocks, but must be finite.
      // Written before this thread's arrival on the barrier, which publishes them to the consumers.
      for (int m = 0; m < a.M; ++m)
        for (uint32_t o = xb; o < full; o += 16) sts128_zero(st + C::W_BYTES + m * XS + o);   // K % 16 == 0: xb is a multiple of 32
      fence_proxy_async();
    }
    mbar_expect_tx(bar, TM * wb + (uint32_t)a.M * xb);
    const uint8_t* src = a.packed + (size_t)(w.unit * TM) * strip_run + (size_t)w.c * PIECE_BYTES;
#pragma unroll
    for (int tm = 0; tm < TM; ++tm) bulk_copy_g2s(st + tm * C::STRIP_BYTES, src + tm * strip_run, wb, bar);
  };
  auto issue_x = [&](const Walk& w) {
    const uint32_t st = stage_addr(w.slot) + C::W_BYTES, bar = bar_full + 8 * w.slot;
    const int n = min(CPS, w.c1 - w.c);
    const uint32_t xb = (uint32_t)min(n * CHUNK_K, a.K - w.c * CHUNK_K) * 2u;
    const __nv_bfloat16* src = a.x + (size_t)w.c * CHUNK_K;
    for (int m = 0; m < a.M; ++m) bulk_copy_g2s(st + m * XS, src + (size_t)m * a.K, xb, bar);
  };

  // ---- warp 0 sets up the barriers and sends out the first ring of weight copies (lane k: stage k) before the
  // CTA meets: they depend on nothing, and the first HBM round trip is the longest wait of a short launch ----
  Walk mine;                                                  // warp 0: the lane's stage of the first ring
  bool mine_valid = false;
  if (warp == 0) {
    if (lane == 0) {
      abort_word = 0;
      never_set = 0;
      for (int i = 0; i < MAX_STAGES; ++i) {
        mbar_init(bar_full + 8 * i, 1);
        mbar_init(bar_empty + 8 * i, CW);
      }
      for (int i = 0; i < 2; ++i) {
        mbar_init(bar_red_full + 8 * i, CW);
        mbar_init(bar_red_free + 8 * i, 1);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (stages >= 2) {
      walk_start(mine);
      for (int j = 0; j < lane && mine.seg_i < work.n_seg; ++j) walk_next(mine);
      mine_valid = lane < stages && mine.seg_i < work.n_seg;
      if (mine_valid) issue_w(mine);
    }
  }
  grid_dep_launch();                                          // the next launch of the stream may become resident
  __syncthreads();
  if (stages < 2) {                                           // cannot happen with the sizes the host admits
    if (threadIdx.x == 0) { grid_dep_wait(); atomicCAS(a.status, 0u, 20u); }
    return;
  }

  auto fail = [&](uint32_t code) {
    *abort_flag = 1;
    grid_dep_wait();                                          // the status word lives in the (possibly shared) workspace
    atomicCAS(a.status, 0u, code);
  };

  if (warp == 0) {
    // ===================== producer: bulk copies into the ring =====================
    grid_dep_wait();                                          // activations may belong to the preceding kernel
    if (mine_valid) issue_x(mine);
    const int first = (int)__popc(__ballot_sync(0xFFFFFFFFu, mine_valid));   // stages of the first ring
    if (lane == 0) {
      Walk head = mine;                                       // stage 0; move on to the first stage not yet issued
      int issued = first;
      for (int j = 0; j < first; ++j) walk_next(head);
      for (; head.seg_i < work.n_seg; ++issued, walk_next(head)) {
        if (!wait_phase<100>(bar_empty + 8 * head.slot, (uint32_t)head.phase ^ 1u, abort_flag)) { fail(1); break; }
        issue_w(head);
        issue_x(head);
      }
      // Drain: copies still in flight must land before this CTA's shared memory is released.  Waiting for the
      // last `stages` issued stages covers everything that can still be in flight.
      {
        int slot = 0, phase = 0;
        const int skip = issued > stages ? issued - stages : 0;
        for (int i = 0; i < issued; ++i) {
          if (i >= skip) wait_phase<100>(bar_full + 8 * slot, (uint32_t)phase, &never_set);
          if (++slot == stages) { slot = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== epilogue: add the consumer warps' partial sums, write y, combine split units =====================
    grid_dep_wait();                                          // y, workspace and the scale scalar may belong to the preceding kernel
    float ts = a.tensor_scale;
    if (a.extra_scale) ts *= *a.extra_scale;
    constexpr int ROWS = C::ROWS;
    const int outputs = ROWS * a.M;                           // output o = token (o / ROWS), row (o % ROWS)
    for (int i = 0; i < work.n_seg; ++i) {
      const Seg s = work.seg(i);
      const int buf = i & 1;
      const bool got = wait_phase<32>(bar_red_full + 8 * buf, (uint32_t)(i >> 1) & 1u, abort_flag);
      if (!got) fail(10);
      if (!__all_sync(0xFFFFFFFFu, got)) break;
      float v[MAX_M];
#pragma unroll
      for (int j = 0; j < MAX_M; ++j) {
        const int o = lane + 32 * j;
        float sum = 0.0f;
        if (o < outputs) {
          const int m = o / ROWS, row = o % ROWS;
          const uint32_t src = red + (uint32_t)(((buf * CW) * a.M + m) * RED_STRIDE + row) * 4u;
#pragma unroll
          for (int w = 0; w < CW; ++w) sum += __uint_as_float(lds32(src + (uint32_t)(w * a.M * RED_STRIDE) * 4u));   // warp order
        }
        v[j] = sum;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_red_free + 8 * buf);
      const int n0 = s.unit * ROWS;
      const bool whole = s.c0 == 0 && s.c1 == a.kc;
      if (whole) {
#pragma unroll
        for (int j = 0; j < MAX_M; ++j) {
          const int o = lane + 32 * j;
          if (o < outputs) {
            const int m = o / ROWS, n = n0 + o % ROWS;
            if (n < a.N) a.y[(size_t)m * a.N + n] = __float2bfloat16_rn(ts * v[j]);
          }
        }
        continue;
      }
      // ---- a piece of a split unit: publish, count, the last arrival adds the pieces in CTA order ----
      float* mine = a.slots + (size_t)b * SLOT_FLOATS;
#pragma unroll
      for (int j = 0; j < MAX_M; ++j)
        if (lane + 32 * j < outputs) mine[lane + 32 * j] = v[j];
      __syncwarp();
      const int c_first = s.unit * a.pieces_per_unit, c_last = c_first + a.pieces_per_unit - 1;
      uint32_t last = 0;
      if (lane == 0) {
        uint32_t prev;
        // release: this warp's slot stores (ordered before by the warp barrier) become visible with the count;
        // acquire: the last arrival sees every earlier arrival's slot stores
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(a.counters + s.unit) : "memory");
        last = (prev + 1 == (uint32_t)a.pieces_per_unit) ? 1u : 0u;
        if (last) a.counters[s.unit] = 0;                     // leave the counter ready for the next call
      }
      last = __shfl_sync(0xFFFFFFFFu, last, 0);
      if (!last) continue;
      float acc[MAX_M];
#pragma unroll
      for (int j = 0; j < MAX_M; ++j) acc[j] = 0.0f;
      // CTA order (a fixed summation order); the loads of four CTAs' slots are in flight together
      for (int cb = c_first; cb <= c_last; cb += 4) {
#pragma unroll
        for (int j = 0; j < MAX_M; ++j) {
          if (lane + 32 * j < outputs) {
            float part[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) part[u] = __ldcg(a.slots + (size_t)min(cb + u, c_last) * SLOT_FLOATS + lane + 32 * j);
#pragma unroll
            for (int u = 0; u < 4; ++u)
              if (cb + u <= c_last) acc[j] += part[u];
          }
        }
      }
#pragma unroll
      for (int j = 0; j < MAX_M; ++j) {
        const int o = lane + 32 * j;
        if (o < outputs) {
          const int m = o / ROWS, n = n0 + o % ROWS;
          if (n < a.N) a.y[(size_t)m * a.N + n] = __float2bfloat16_rn(ts * acc[j]);
        }
      }
    }
  } else {
    // ===================== consumers: decode + MMA =====================
    // the table must be complete before the first decode; the consumer warps fill it themselves
    const int cw = warp - 2;
    {
      const int tid = cw * 32 + lane;
      for (int e = tid; e < 256 * (TABLE_COPIES / 4); e += CW * 32) {
        const uint32_t idx = (uint32_t)e / (TABLE_COPIES / 4);   // packed scale byte [select | negate | code]
        // scale x 2^126 has four significant bits: the upper half of the FP32 pattern is the exact bf16
        const float sc = scale_value(idx & 0x3Fu) * 8.50705917e37f;
        const uint32_t sb = (__float_as_uint(sc) >> 16) | ((idx & PACKED_NEGATE) << 9);
        const float sv = (idx & PACKED_SELECT) ? a.sv1 : a.sv0;
        const uint32_t pv = __float_as_uint(sv * 1.17549435e-38f) >> 16;      // sv x 2^-126
        const uint32_t e0 = sb | (sb << 16), e1 = pv | (pv << 16);
        const uint32_t dst = table + (uint32_t)e * 32;            // four copies per iteration
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %1, %2};" ::"r"(dst), "r"(e0), "r"(e1) : "memory");
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %1, %2};" ::"r"(dst + 16), "r"(e0), "r"(e1) : "memory");
      }
      asm volatile("bar.sync 1, %0;" ::"n"(CW * 32) : "memory");   // consumer warps only
    }
    // The activations of the first stages arrive only after the preceding kernel has finished; waiting for that
    // here (the producer has the weights in flight meanwhile) keeps it out of the bounded waits below.
    grid_dep_wait();
    const int g = lane >> 2, t = lane & 3;
    LaneView v;
    {
      const uint32_t slot = (uint32_t)(g ^ (4 * t));          // row g of block t; row g + 8 sits in slot ^ 8
      const uint32_t piece = (uint32_t)cw * PIECE_BYTES;
      v.h0 = piece + t * 128 + slot * 8;
      v.h1 = piece + t * 128 + (slot ^ 8u) * 8;
      v.sc = piece + PIECE_CODE_BYTES + g * 8 + t * 2;
      // B-fragment column g is token g; a lane without a token reads the last token's columns instead: its
      // products land in accumulator columns that are never stored
      v.xo = (uint32_t)C::W_BYTES + (uint32_t)min(g, a.M - 1) * XS + cw * 128 + t * 32;
      v.tbl = (table << TABLE_SHIFT) | ((uint32_t)(lane & (TABLE_COPIES - 1)) << (3 + TABLE_SHIFT));
    }
    const uint32_t mul_lo = a.mul_lo, mul_hi = a.mul_hi;
    const bool t_ok0 = 2 * t < a.M, t_ok1 = 2 * t + 1 < a.M;    // which of the lane's two accumulator columns are tokens
    float acc[TM][4];
#pragma unroll
    for (int tm = 0; tm < TM; ++tm)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[tm][j] = 0.0f;
    int slot = 0;
    uint32_t phase = 0;
    bool alive = true;
    for (int i = 0; alive && i < work.n_seg; ++i) {
      const Seg s = work.seg(i);
      // stages of CPS chunks; in a stage that starts at chunk c0 this warp's slices are chunks c0 + cw, c0 + cw + CW, ...
      const int n_full = (s.c1 - s.c0) / CPS;
      const bool ragged = (s.c1 - s.c0) % CPS != 0;
#pragma unroll 1
      for (int k = 0; k < n_full + (ragged ? 1 : 0); ++k) {
        if (!wait_phase(bar_full + 8 * slot, phase, abort_flag)) { fail(2); alive = false; }
        if (!__all_sync(0xFFFFFFFFu, alive)) { alive = false; break; }
        const uint32_t st = stage_addr(slot);
        if (k < n_full) slice_steps<TM, SPW, 0, false>(acc, st, v, 0, 0, mul_lo, mul_hi);
        else slice_steps<TM, SPW, 0, true>(acc, st, v, s.c0 + k * CPS + cw, s.c1, mul_lo, mul_hi);
        __syncwarp();                                         // every lane has read the stage
        if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
        if (++slot == stages) { slot = 0; phase ^= 1u; }
      }
      if (!alive) break;
      // ---- end of a segment: leave this warp's partial sums for the epilogue warp ----
      const int buf = i & 1;
      if (!wait_phase(bar_red_free + 8 * buf, ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_flag)) { fail(3); alive = false; }
      if (!__all_sync(0xFFFFFFFFu, alive)) { alive = false; break; }
      // element (token m, row r) of warp cw at ((buf * CW + cw) * M + m) * RED_STRIDE + r
      const uint32_t dst = red + (uint32_t)((buf * CW + cw) * a.M * RED_STRIDE) * 4u;
#pragma unroll
      for (int tm = 0; tm < TM; ++tm) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int m = 2 * t + (j & 1), row = 16 * tm + 8 * (j >> 1) + g;
          if ((j & 1) ? t_ok1 : t_ok0)
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst + (uint32_t)(m * RED_STRIDE + row) * 4u), "f"(acc[tm][j]) : "memory");
          acc[tm][j] = 0.0f;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_red_full + 8 * buf);
    }
  }
  __syncthreads();
}

}  // namespace stream_path

// ------------------------------------------------------------------ host side
static int stream_sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

struct StreamPlan {
  int TM, SPW, grid, units, kc;
  int whole_base, whole_per_cta, rem_ctas, pieces_per_unit;
  double cost;
  size_t counters_bytes, slots_bytes;
};

static size_t align256s(size_t v) { return (v + 255) / 256 * 256; }

// One candidate: units of TM strips; every CTA takes whole units only (split == false), or q whole units after a
// piece of one of the remaining units, each of which is cut along K into equal pieces (processed first, combined
// through the workspace).  The cost is the busiest CTA's work in strip-slices: a slice of TM strips costs TM plus
// what is per slice (activation fragment, loop), and a split whose combination nothing follows (q == 0) pays
// for it at the end of the launch.
static StreamPlan stream_candidate(const razer_desc* d, int M, int G, int TM, bool split) {
  using namespace stream_path;
  StreamPlan p;
  const Geometry g = make_geometry(d->N, d->K);
  const int strips = (d->N + STRIP_ROWS - 1) / STRIP_ROWS;
  p.TM = TM;
  p.units = (strips + TM - 1) / TM;
  p.kc = g.k_chunks;
  // slices per warp and stage: as many as leave three stages in what a CTA has for its ring
  p.SPW = 1;
  const int ring_bytes = SMEM_BYTES - TABLE_BYTES - 2 * CW * M * RED_STRIDE * 4 - 2048;
  for (int spw = (TM == 1 ? 4 : 2); spw >= 1; spw >>= 1) {
    const int stage = TM * CW * spw * PIECE_BYTES + M * (CW * spw * 128 + 16);
    if (3 * stage <= ring_bytes) { p.SPW = spw; break; }
  }
  const double per_slice = TM + 0.12 + 0.04 * M;
  const int q = p.units / G, rem = p.units - q * G;
  if (split && rem > 0) {
    int pieces = G / rem;                                               // >= 1
    pieces = std::max(1, std::min(pieces, p.kc / CW));                  // a piece is at least one slice per warp
    p.whole_base = rem;
    p.whole_per_cta = q;
    p.pieces_per_unit = pieces;
    p.rem_ctas = rem * pieces;
    p.grid = q > 0 ? G : p.rem_ctas;
    p.cost = ((double)q * p.kc + (p.kc + pieces - 1) / pieces) * per_slice + (q == 0 && pieces > 1 ? 40.0 : 0.0);
  } else {
    const int qa = (p.units + G - 1) / G;
    p.whole_base = 0;
    p.whole_per_cta = qa;
    p.pieces_per_unit = 1;
    p.rem_ctas = 0;
    p.grid = (p.units + qa - 1) / qa;
    p.cost = (double)qa * p.kc * per_slice;
  }
  p.counters_bytes = align256s((size_t)G * sizeof(uint32_t));           // at most G - 1 split units
  p.slots_bytes = (size_t)G * SLOT_FLOATS * sizeof(float);
  return p;
}

// The cheapest of the four candidates (one or two strips per unit, with or without a split).
static StreamPlan stream_plan(const razer_desc* d, int M) {
  using namespace stream_path;
  static const int per_sm = [] { const char* e = getenv("RAZER_STREAM_CTAS"); const int v = e ? atoi(e) : 0; return v >= 1 && v <= OCC ? v : OCC; }();   // tuning aids
  static const char force_split = [] { const char* e = getenv("RAZER_STREAM_SPLIT"); return e ? e[0] : '\0'; }();
  static const char force_tm = [] { const char* e = getenv("RAZER_STREAM_TM"); return e ? e[0] : '\0'; }();
  const int G = per_sm * stream_sm_count();
  StreamPlan best;
  bool have = false;
  for (int TM = 1; TM <= 2; ++TM) {
    if ((force_tm == '1' && TM != 1) || (force_tm == '2' && TM != 2)) continue;
    for (int split = 0; split <= 1; ++split) {
      if (force_split == '0' && split) continue;
      const StreamPlan c = stream_candidate(d, M, G, TM, split != 0);
      if (force_split == '1' && !split && c.units % G != 0) continue;
      if (!have || c.cost < best.cost) { best = c; have = true; }
    }
  }
  if (!have) best = stream_candidate(d, M, G, 1, false);
  return best;
}

bool gemv_stream_supported(const razer_desc* d, int M) {
  (void)d;
  return M >= 1 && M <= stream_path::MAX_M;
}

size_t gemv_stream_workspace_bytes(const razer_desc* d, int M) {
  const StreamPlan p = stream_plan(d, M);
  return WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
}

template <int TM, int SPW>
static int launch_stream_cfg(const stream_path::Args& a, int grid, cudaStream_t st) {
  auto kern = stream_path::razer_stream_kernel<TM, SPW>;
  static bool attr_set = false;
  if (!attr_set) {
    RAZER_TRY(check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, stream_path::SMEM_BYTES),
                         "cudaFuncSetAttribute(max dynamic shared memory)"));
    attr_set = true;
  }
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(stream_path::THREADS);
  cfg.dynamicSmemBytes = stream_path::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, a);
  count_launches(1);
  return check_cuda(e, "razer_stream_kernel launch");
}

int launch_gemv_stream(const razer_desc* d, const void* packed, const void* x, int M, float extra_scale,
                       const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  const StreamPlan p = stream_plan(d, M);
  const size_t need = WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
  if (!ws || ws_bytes < need)
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  stream_path::Args a;
  a.packed = (const uint8_t*)packed;
  a.x = (const __nv_bfloat16*)x;
  a.y = (__nv_bfloat16*)y;
  a.status = (uint32_t*)ws;
  a.counters = (uint32_t*)((char*)ws + WS_STATUS_BYTES);
  a.slots = (float*)((char*)ws + WS_STATUS_BYTES + p.counters_bytes);
  a.extra_scale = extra_scale_dev;
  a.N = d->N;
  a.K = d->K;
  a.kc = p.kc;
  a.M = M;
  a.units = p.units;
  a.whole_base = p.whole_base;
  a.whole_per_cta = p.whole_per_cta;
  a.rem_ctas = p.rem_ctas;
  a.pieces_per_unit = p.pieces_per_unit;
  a.sv0 = d->sv_mag[0];
  a.sv1 = d->sv_mag[1];
  a.tensor_scale = d->tensor_scale * extra_scale;
  a.mul_lo = (1u << 6) + (1u << 12);
  a.mul_hi = (1u << 2) + (1u << 8);
  if (p.TM == 2) return p.SPW == 2 ? launch_stream_cfg<2, 2>(a, p.grid, st) : launch_stream_cfg<2, 1>(a, p.grid, st);
  return p.SPW == 4 ? launch_stream_cfg<1, 4>(a, p.grid, st)
                    : p.SPW == 2 ? launch_stream_cfg<1, 2>(a, p.grid, st) : launch_stream_cfg<1, 1>(a, p.grid, st);
}

}  // namespace razer
