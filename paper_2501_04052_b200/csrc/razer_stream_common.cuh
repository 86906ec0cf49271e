// Declarations of the decode kernel (razer_gemv_stream.cu): configuration,
// kernel arguments, the list of a CTA's work segments, bounded barrier waits, shared-memory access helpers, the
// epilogue warp's loop and the host-side partition plan.
#pragma once

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
  float* slots;              // [grid][2][SLOT_FLOATS]
  uint32_t* counters;        // one per split unit, zero between calls
  uint32_t* status;          // device status word
  const float* extra_scale;  // optional device scalar multiplied into the tensor scale
  int N, K, kc, M;
  int units;                 // units of TM strips that hold rows < N
  int whole_base, whole_per_cta;   // CTA b owns the whole units whole_base + b * whole_per_cta .. (clipped to units)
  int rem_ctas;              // CTAs that share the split units [0, whole_base); 0 = nothing is split
  int pieces_per_unit;       // a split unit is cut along K into this many equal pieces; the pieces of all split units,
                             // in unit order, are dealt out to the rem_ctas CTAs in equal contiguous ranges
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

// A CTA's list of segments: its range of pieces of split units (at most two units), then its whole units.
struct Work {
  int n_rem, n_seg;
  int u0, a0, a1;            // first split segment: unit, chunk range
  int u1, b1;                // second split segment: unit, chunks [0, b1)
  int wu0;                   // first whole unit
  int kc;
  __device__ __forceinline__ Seg seg(int i) const {
    Seg s;
    if (i < n_rem) {
      if (i == 0) { s.unit = u0; s.c0 = a0; s.c1 = a1; }
      else { s.unit = u1; s.c0 = 0; s.c1 = b1; }
    } else {
      s.unit = wu0 + (i - n_rem);
      s.c0 = 0;
      s.c1 = kc;
    }
    return s;
  }
};

// Piece range of CTA c: pieces [P c / ctas, P (c + 1) / ctas) of the P = units * pieces_per_unit pieces
// (P * ctas stays far below 2^32: at most a few hundred units, eight pieces each, a few hundred CTAs).
__device__ __forceinline__ int piece_begin(const Args& a, int c) {
  const uint32_t P = (uint32_t)(a.whole_base * a.pieces_per_unit);
  if (P == (uint32_t)a.rem_ctas) return c;                   // one piece per CTA
  return (int)((P * (uint32_t)c) / (uint32_t)a.rem_ctas);
}
// CTA that owns piece i (the inverse of piece_begin).
__device__ __forceinline__ int cta_of_piece(const Args& a, int i) {
  const uint32_t P = (uint32_t)(a.whole_base * a.pieces_per_unit);
  if (P == (uint32_t)a.rem_ctas) return i;
  return (int)((((uint32_t)(i + 1) * (uint32_t)a.rem_ctas) - 1u) / P);
}

__device__ __forceinline__ Work make_work(const Args& a, int b) {
  Work w;
  w.kc = a.kc;
  w.n_rem = 0;
  w.u0 = w.a0 = w.a1 = w.u1 = w.b1 = 0;
  if (b < a.rem_ctas) {
    // piece j of a unit: chunks [kc j / p, kc (j + 1) / p)
    const int p = a.pieces_per_unit;
    const int i0 = piece_begin(a, b), i1 = piece_begin(a, b + 1);       // i1 > i0: there are at least as many pieces as CTAs
    w.u0 = i0 / p;
    w.u1 = (i1 - 1) / p;
    w.n_rem = w.u1 > w.u0 ? 2 : 1;
    w.a0 = (a.kc * (i0 - w.u0 * p)) / p;
    w.a1 = w.n_rem == 2 ? a.kc : (a.kc * (i1 - w.u0 * p)) / p;
    w.b1 = (a.kc * (i1 - w.u1 * p)) / p;
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

// The epilogue warp's loop over the CTA's segments: add the consumer warps' partial sums of a segment in warp order,
// then either write y (whole unit) or publish the piece, count, and let the last arrival add the pieces in CTA order.
// `ts` multiplies every output.  `fail(code)` records a wait that gave up.
template <int ROWS, class Fail>
__device__ __forceinline__ void epilogue_loop(const Args& a, const Work& work, int b, int lane, uint32_t red,
                                              uint32_t bar_red_full, uint32_t bar_red_free, volatile uint32_t* abort_flag,
                                              float ts, Fail fail) {
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
    float* mine = a.slots + ((size_t)b * 2 + i) * SLOT_FLOATS;          // split segments come first: i is 0 or 1
#pragma unroll
    for (int j = 0; j < MAX_M; ++j)
      if (lane + 32 * j < outputs) mine[lane + 32 * j] = v[j];
    __syncwarp();
    const int c_first = cta_of_piece(a, s.unit * a.pieces_per_unit);
    const int c_last = cta_of_piece(a, (s.unit + 1) * a.pieces_per_unit - 1);
    uint32_t last = 0;
    if (lane == 0) {
      uint32_t prev;
      // release: this warp's slot stores (ordered before by the warp barrier) become visible with the count;
      // acquire: the last arrival sees every earlier arrival's slot stores
      asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(a.counters + s.unit) : "memory");
      last = (prev + 1 == (uint32_t)(c_last - c_first + 1)) ? 1u : 0u;
      if (last) a.counters[s.unit] = 0;                     // leave the counter ready for the next call
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) continue;
    float acc[MAX_M];
#pragma unroll
    for (int j = 0; j < MAX_M; ++j) acc[j] = 0.0f;
    // CTA order (a fixed summation order); the loads of four CTAs' slots are in flight together
    for (int cb = c_first; cb <= c_last; cb += 4) {
      const float* src[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = min(cb + u, c_last);
        const int sl = piece_begin(a, c) / a.pieces_per_unit == s.unit ? 0 : 1;   // the unit is that CTA's first or second segment
        src[u] = a.slots + ((size_t)c * 2 + sl) * SLOT_FLOATS;
      }
#pragma unroll
      for (int j = 0; j < MAX_M; ++j) {
        if (lane + 32 * j < outputs) {
          float part[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) part[u] = __ldcg(src[u] + lane + 32 * j);
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
}

}  // namespace stream_path

// ------------------------------------------------------------------ host side
static inline int stream_sm_count() {
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

static inline size_t align256s(size_t v) { return (v + 255) / 256 * 256; }

// One candidate: units of TM strips; every CTA takes whole units only (split == false), or q whole units after a
// piece of one of the remaining units, each of which is cut along K into equal pieces (processed first, combined
// through the workspace).  The cost is the busiest CTA's work in strip-slices: a slice of TM strips costs TM plus
// what is per slice (activation fragment, loop), and a split whose combination nothing follows (q == 0) pays
// for it at the end of the launch.
static inline StreamPlan stream_candidate(const razer_desc* d, int M, int G, int TM, bool split) {
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
    // pieces per unit: the count that leaves the busiest CTA the least to do; every further segment of a CTA costs a
    // little (partial sums, combination), so ties go to fewer pieces
    int best_p = 1;
    double best_cost = 0;
    const int max_p = std::max(1, std::min(8, p.kc / CW));              // a piece is at least one slice per warp
    for (int pc = 1; pc <= max_p; ++pc) {
      const int ctas = std::min(G, rem * pc);
      const int most = (rem * pc + ctas - 1) / ctas;                    // pieces of the busiest CTA
      const double c = most * ((p.kc + pc - 1) / pc) * per_slice + (most > 1 ? 4.0 : 0.0) + 0.5 * pc;
      if (pc == 1 || c < best_cost) { best_cost = c; best_p = pc; }
    }
    p.whole_base = rem;
    p.whole_per_cta = q;
    p.pieces_per_unit = best_p;
    p.rem_ctas = std::min(G, rem * best_p);
    p.grid = q > 0 ? G : p.rem_ctas;
    p.cost = (double)q * p.kc * per_slice + best_cost + (q == 0 && best_p > 1 ? 40.0 : 0.0);
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
  p.slots_bytes = (size_t)G * 2 * SLOT_FLOATS * sizeof(float);
  return p;
}

// The cheapest of the four candidates (one or two strips per unit, with or without a split).
static inline StreamPlan stream_plan(const razer_desc* d, int M) {
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

}  // namespace razer
