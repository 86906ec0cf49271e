// Decode GEMV (M <= 16) against packed RaZeR weights for sm_100a: register-fragment tensor-core kernel with
// no exchange between CTAs.
//
//   y[m, n] = bf16( ts * sum_k x[m, k] * D1[n, k] ),   D1 = block_scale * element (exact bf16)
//
// Every weight byte is used exactly once.  Each warp streams "its" chunk slices through a small private
// ring in shared memory (cp.async, 16 bytes per lane, several slices ahead; only the warp itself waits on
// them), each lane decodes the code words of "its" blocks in registers (razer_decode.cuh) and feeds them
// as the A fragment of a warp-level m16n8k16 tensor-core MMA whose B fragment is the activation slice
// (8 tokens along n; a second fragment and accumulator for tokens 8..15), accumulated in FP32 registers.  Sec. 4.3 of the paper describes this style for its
// weight-only kernel (weights pre-shuffled so that each thread's loads match its MMA fragment).
//
// Work unit: 32 weight rows (two 16-row MMA tiles) over the whole of K.  A CTA (16 warps) takes a contiguous
// range of rows, in whole units or in 16-row halves, whichever the host's cost model prefers (with halves a unit
// at either end of the range may be shared with the neighbouring CTA, each doing its own tile).  Inside a unit warp w
// takes the chunks (64 columns) w, w + 16, ...  In a chunk, lane (g = lane / 4, t = lane % 4) decodes block t
// of rows g and g + 8 of each tile; MMA q (0..3) takes elements 4q .. 4q + 3 of every lane's block, i.e. the
// MMA's k slots are columns 16 t + 4 q + {0, 1, 2, 3}, for A and B alike.  At the end of a unit the 16 warps
// leave their partial sums in shared memory, and 32 x tokens threads add them in warp order, scale, round and store.
// Nothing is exchanged between CTAs, so there is no workspace, no counter and no wait on another CTA; the
// price is that the rows have to divide evenly enough over the SMs, which the host checks before it picks
// this kernel.
#include <cuda.h>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_decode.cuh"

namespace razer {

namespace direct_path {

constexpr int WARPS = 16;
constexpr int THREADS = 32 * WARPS;
constexpr int UNIT_ROWS = 32;                       // two 16-row MMA tiles
constexpr int DEPTH = 2;                            // chunk slices in flight per warp
// A warp's ring stage: the 32-row slice of one chunk, [blk 0..3][32 slots x 8 B] (blocks 2 and 3 sit 32 bytes
// further so that a half-warp's 8-byte reads, four blocks x four slots, cover all 32 banks), then
// [32 rows x 4 scale bytes], then per group of 8 tokens the activations of the chunk: lane l keeps its 16 columns
// (token l / 4 of the group, columns 16 (l % 4) ..) as two 16-byte halves at 16 l and 512 + 16 l.
constexpr int STAGE_CODE_BYTES = 4 * 256 + 32;
constexpr int STAGE_X_OFF = STAGE_CODE_BYTES + 128;
constexpr int TABLE_ALIGN = 16384;                  // decode_block_consts_rot() wants the tables on a 16 KB boundary
constexpr long long STEP_BYTES = (long long)WARPS * CHUNK_BYTES;   // a warp's next chunk of the same unit
static_assert(STAGE_X_OFF % 16 == 0 && DECODE_TABLE_BYTES % 16 == 0, "16-byte copies");

template <int NT>                                   // NT groups of 8 tokens
struct Cfg {
  static constexpr int TOKENS = 8 * NT;
  static constexpr int STAGE_BYTES = STAGE_X_OFF + 1024 * NT;
  static constexpr int RED_FLOATS = UNIT_ROWS * TOKENS;      // one warp's partial sums
  static constexpr int RED_BYTES = 2 * WARPS * RED_FLOATS * 4;
  static constexpr int RING_BYTES = WARPS * DEPTH * STAGE_BYTES;
  static constexpr size_t SMEM_BYTES = TABLE_ALIGN + DECODE_TABLE_BYTES + RING_BYTES + RED_BYTES;
  static_assert(RED_FLOATS <= THREADS && SMEM_BYTES <= 227 * 1024, "one thread per output of a unit; one CTA per SM");
};

__device__ __forceinline__ constexpr int stage_blk_off(int blk) { return blk * 256 + (blk >> 1) * 32; }

// 16 bytes to dst + DOFF from src + SOFF, of which only the first `bytes` (0 or 16) are read; the rest is written
// as zero.  The offsets are immediates of the instruction, so one base register serves several copies.
template <int DOFF, int SOFF>
__device__ __forceinline__ void cp_async16_cg(uint32_t dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.cg.shared.global [%0+%3], [%1+%4], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes), "n"(DOFF), "n"(SOFF)
               : "memory");
}
template <int DOFF, int SOFF>
__device__ __forceinline__ void cp_async16_ca(uint32_t dst, const void* src, uint32_t bytes) {   // kept in L1: re-read per unit
  asm volatile("cp.async.ca.shared.global [%0+%3], [%1+%4], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes), "n"(DOFF), "n"(SOFF)
               : "memory");
}
// shared-memory loads at base + OFF (immediate)
template <int OFF>
__device__ __forceinline__ uint32_t lds32_at(uint32_t base) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(base), "n"(OFF) : "memory");
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
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// D (+)= A(16 x 16, row) * B(16 x 8, col), bf16 inputs, FP32 accumulation.
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct Args {
  const uint8_t* packed;
  const __nv_bfloat16* x;    // [M][K]
  __nv_bfloat16* y;          // [M][N]
  const float* extra_scale;  // optional device scalar multiplied into the tensor scale
  Geometry g;
  float sv0, sv1, tensor_scale;
  uint32_t mul_lo, mul_hi;   // 2^6 + 2^12 and 2^2 + 2^8 (razer_decode.cuh)
  int M, halves;             // 16-row half units of the padded matrix
  int unit_aligned;          // CTA ranges are whole 32-row units (else 16-row halves)
};

// One chunk slice of MMA tile TILE (16 rows): decode the lane's two blocks, four MMAs.
// codes_h0 / codes_h1: the lane's code words of rows g / g + 8 of tile 0 in the stage; scales: row g's scale word.
// rot = (8 t + 25) % 32 turns a row's scale word so that block t's byte sits on bits 14:7.
template <int TILE, int NT>
__device__ __forceinline__ void tile_step(float (&acc)[NT][4], uint32_t codes_h0, uint32_t codes_h1, uint32_t scales,
                                          uint32_t rot, const DecodeTables& dt, uint32_t mul_lo, uint32_t mul_hi,
                                          const uint32_t (&xq)[NT][4][2]) {
  const uint2 c0 = lds64_at<128 * TILE>(codes_h0), c1 = lds64_at<128 * TILE>(codes_h1);
  const uint32_t s0 = lds32_at<64 * TILE>(scales), s1 = lds32_at<64 * TILE + 32>(scales);
  uint32_t e[2][8];
  {
    uint32_t ss2;
    SvConsts svc;
    decode_block_consts_rot(dt, __funnelshift_r(s0, s0, rot), ss2, svc);
    decode_word(c0.x, ss2, svc, mul_lo, mul_hi, e[0]);
    decode_word(c0.y, ss2, svc, mul_lo, mul_hi, e[0] + 4);
  }
  {
    uint32_t ss2;
    SvConsts svc;
    decode_block_consts_rot(dt, __funnelshift_r(s1, s1, rot), ss2, svc);
    decode_word(c1.x, ss2, svc, mul_lo, mul_hi, e[1]);
    decode_word(c1.y, ss2, svc, mul_lo, mul_hi, e[1] + 4);
  }
#pragma unroll
  for (int q = 0; q < 4; ++q)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
      mma_16816(acc[nt], e[0][2 * q], e[1][2 * q], e[0][2 * q + 1], e[1][2 * q + 1], xq[nt][q][0], xq[nt][q][1]);
}

template <int NT>
__global__ void __launch_bounds__(THREADS, 1) razer_direct_kernel(const Args a) {
  using C = Cfg<NT>;
  constexpr int TOKENS = C::TOKENS, STAGE_BYTES = C::STAGE_BYTES, RED_FLOATS = C::RED_FLOATS, RING_BYTES = C::RING_BYTES;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  // tables first, on a 16 KB boundary of the shared window; then the rings; then the reduction buffers
  const uint32_t raw_addr = smem_addr(smem_raw);
  uint8_t* tables = smem_raw + (((raw_addr + TABLE_ALIGN - 1) & ~(uint32_t)(TABLE_ALIGN - 1)) - raw_addr);
  uint8_t* ring_base = tables + DECODE_TABLE_BYTES;
  float* red = reinterpret_cast<float*>(ring_base + RING_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int kc = a.g.k_chunks;                               // >= WARPS (host check): every warp has chunks
  const int per_unit = (kc - warp + WARPS - 1) / WARPS;      // this warp's chunks of a unit: warp, warp + 16, ...
  // this CTA's rows: a contiguous range of 16-row halves; a 32-row unit at either end may be shared with a neighbour
  int h_begin, h_end;
  if (a.unit_aligned) {
    const int units = a.halves >> 1;
    h_begin = 2 * (int)(((long long)units * blockIdx.x) / gridDim.x);
    h_end = 2 * (int)(((long long)units * (blockIdx.x + 1)) / gridDim.x);
  } else {
    h_begin = (int)(((long long)a.halves * blockIdx.x) / gridDim.x);
    h_end = (int)(((long long)a.halves * (blockIdx.x + 1)) / gridDim.x);
  }
  const int u_begin = h_begin >> 1, u_end = (h_end + 1) >> 1;
  auto unit_mask = [&](int u) -> uint32_t {                  // which MMA tiles of unit u are this CTA's
    return (2 * u >= h_begin && 2 * u < h_end ? 1u : 0u) | (2 * u + 1 >= h_begin && 2 * u + 1 < h_end ? 2u : 0u);
  };

  grid_dep_launch();
  decode_tables_fill(tables, a.sv0, a.sv1, threadIdx.x, THREADS);

  const uint32_t ring = smem_addr(ring_base) + (uint32_t)warp * (DEPTH * STAGE_BYTES);
  bool has_token[NT];                                        // token g of group nt exists
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) has_token[nt] = 8 * nt + g < a.M;
  const bool k_tail = (a.g.K % CHUNK_K) != 0;                // only then can a chunk hold absent columns
  // ---- copy side: what this lane copies for every chunk slice ----
  // two 16-byte pieces of code words (blocks cblk and cblk + 2, slots 2 piece and + 1), 16 bytes of scale
  // words (lanes 0..7) and its own 32 bytes of activations; a size of 0 writes zeros and reads nothing
  const int piece = lane & 15, cblk = lane >> 4;
  const uint32_t dst_codes = ring + stage_blk_off(cblk) + piece * 16;       // blocks cblk + 2: 544 bytes further
  const uint32_t dst_lane = ring + lane * 16;                                 // + STAGE_CODE_BYTES: scales, + STAGE_X_OFF: activations
  const uint8_t* src_codes;                                                   // blocks cblk + 2: 2048 bytes further
  const uint8_t* src_scales;
  const __nv_bfloat16* src_x;                                                 // token g; token g + 8: 8 K elements further
  int col, cp_unit, cp_left;                                                  // first activation column; unit; chunks of it still to copy
  uint32_t sz_codes, sz_scales;
  auto cursor_to_unit = [&](int u) {
    const int n0 = u * UNIT_ROWS, tile = n0 / TILE_ROWS, r0 = n0 % TILE_ROWS;
    const uint8_t* ck = a.packed + ((size_t)tile * kc + warp) * CHUNK_BYTES;
    const uint32_t mask = u < u_end ? unit_mask(u) : 0u;
    src_codes = ck + r0 * 8 + cblk * 1024 + piece * 16;
    src_scales = ck + CHUNK_CODE_BYTES + r0 * 4 + (lane & 7) * 16;
    src_x = a.x + (size_t)(has_token[0] ? g : 0) * a.g.K + warp * CHUNK_K + 16 * t;
    col = warp * CHUNK_K + 16 * t;
    cp_unit = u;
    cp_left = per_unit;
    sz_codes = ((mask >> (piece >> 3)) & 1u) ? 16u : 0u;
    sz_scales = ((mask >> ((lane & 7) >> 2)) & 1u) ? 16u : 0u;
  };
  auto copy_weights = [&](uint32_t so) {                     // weights: no dependency on earlier kernels
    if (cp_unit < u_end) {
      const uint32_t dc = dst_codes + so;
      cp_async16_cg<0, 0>(dc, src_codes, sz_codes);
      cp_async16_cg<544, 2048>(dc, src_codes, sz_codes);
      if (lane < 8) cp_async16_cg<STAGE_CODE_BYTES, 0>(dst_lane + so, src_scales, sz_scales);
    }
  };
  auto copy_x = [&](uint32_t so) {
    if (cp_unit < u_end) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (has_token[nt]) {
          const __nv_bfloat16* src = src_x + (size_t)nt * 8 * a.g.K;
          uint32_t sz = 16u;
          if (k_tail && col >= a.g.K) {                      // K is a multiple of 16: a 16-column group is whole or absent
            src = a.x;
            sz = 0u;
          }
          if (nt == 0) {
            cp_async16_ca<STAGE_X_OFF, 0>(dst_lane + so, src, sz);
            cp_async16_ca<STAGE_X_OFF + 512, 16>(dst_lane + so, src, sz);
          } else {
            cp_async16_ca<STAGE_X_OFF + 1024, 0>(dst_lane + so, src, sz);
            cp_async16_ca<STAGE_X_OFF + 1536, 16>(dst_lane + so, src, sz);
          }
        }
      }
    }
  };
  auto cursor_next = [&]() {
    if (--cp_left > 0) {
      src_codes += STEP_BYTES;
      src_scales += STEP_BYTES;
      src_x += WARPS * CHUNK_K;
      col += WARPS * CHUNK_K;
    } else {
      cursor_to_unit(cp_unit + 1);
    }
  };

  // lanes without a token never copy activations: their slots stay zero
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
    if (!has_token[nt]) {
      uint8_t* mine = ring_base + (size_t)warp * (DEPTH * STAGE_BYTES) + STAGE_X_OFF + 1024 * nt + lane * 16;
#pragma unroll
      for (int d = 0; d < DEPTH; ++d) {
        *reinterpret_cast<uint4*>(mine + d * STAGE_BYTES) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(mine + d * STAGE_BYTES + 512) = make_uint4(0, 0, 0, 0);
      }
    }

  // ---------------- prologue: the first DEPTH slices' weights, then (after the dependency) their activations ----------------
  cursor_to_unit(u_begin);
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    copy_weights(d * STAGE_BYTES);
    cursor_next();
  }
  __syncthreads();                                           // tables are ready
  const DecodeTables dt = decode_tables_view(tables, lane);
  const uint32_t mul_lo = a.mul_lo, mul_hi = a.mul_hi;
  grid_dep_wait();                                           // activations and outputs may belong to the preceding kernel
  float ts = a.tensor_scale;
  if (a.extra_scale) ts *= *a.extra_scale;
  cursor_to_unit(u_begin);
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    copy_x(d * STAGE_BYTES);
    cp_async_commit();                                       // one group per position (the first also holds all the weights above)
    cursor_next();
  }

  // ---- compute side: this lane's reads from a stage ----
  const uint32_t lo = (t & 1) ? 64u : 0u;                    // odd blocks keep rows g and g + 8 the other way round
  const uint32_t rd_h0 = ring + stage_blk_off(t) + g * 8 + lo, rd_h1 = ring + stage_blk_off(t) + g * 8 + (64u - lo);
  const uint32_t rd_scales = ring + STAGE_CODE_BYTES + g * 4;
  const uint32_t rot = (uint32_t)(8 * t + 25) & 31u;
  float acc[2][NT][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[mt][nt][j] = 0.0f;

  uint32_t so = 0;                                           // byte offset of the current stage in the ring
  int buf = 0;
  for (int u = u_begin; u < u_end; ++u) {
    const uint32_t mask = unit_mask(u);
#pragma unroll 1
    for (int j = 0; j < per_unit; ++j) {
      cp_async_wait<DEPTH - 1>();                            // this lane's pieces of the oldest slice have landed
      __syncwarp();                                          // ... and so have the other lanes'
      const uint32_t bx = dst_lane + so, bh0 = rd_h0 + so, bh1 = rd_h1 + so, bs = rd_scales + so;
      uint32_t xq[NT][4][2];
      {
        const uint4 xa = lds128_at<STAGE_X_OFF>(bx), xb = lds128_at<STAGE_X_OFF + 512>(bx);
        xq[0][0][0] = xa.x, xq[0][0][1] = xa.y, xq[0][1][0] = xa.z, xq[0][1][1] = xa.w;
        xq[0][2][0] = xb.x, xq[0][2][1] = xb.y, xq[0][3][0] = xb.z, xq[0][3][1] = xb.w;
      }
      if (NT == 2) {
        const uint4 xa = lds128_at<STAGE_X_OFF + 1024>(bx), xb = lds128_at<STAGE_X_OFF + 1536>(bx);
        xq[NT - 1][0][0] = xa.x, xq[NT - 1][0][1] = xa.y, xq[NT - 1][1][0] = xa.z, xq[NT - 1][1][1] = xa.w;
        xq[NT - 1][2][0] = xb.x, xq[NT - 1][2][1] = xb.y, xq[NT - 1][3][0] = xb.z, xq[NT - 1][3][1] = xb.w;
      }
      if (mask & 1u) tile_step<0, NT>(acc[0], bh0, bh1, bs, rot, dt, mul_lo, mul_hi, xq);
      if (mask & 2u) tile_step<1, NT>(acc[1], bh0, bh1, bs, rot, dt, mul_lo, mul_hi, xq);
      __syncwarp();                                          // every lane has read the stage: refill it
      copy_weights(so);
      copy_x(so);
      cp_async_commit();
      cursor_next();
      if (DEPTH == 2) so ^= (uint32_t)STAGE_BYTES;
      else so = (so + STAGE_BYTES == DEPTH * STAGE_BYTES) ? 0u : so + STAGE_BYTES;
    }
    // End of the unit: leave this warp's partial sums, meet, and let 256 threads finish the rows.
    // Element (row, token) of the unit sits at row * TOKENS + token (8 tokens: a warp's 32 stores fall on 16 banks, two each; 8 stores per unit).
    float* mine = red + (buf * WARPS + warp) * RED_FLOATS;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          mine[(16 * mt + 8 * (j >> 1) + g) * TOKENS + 8 * nt + 2 * t + (j & 1)] = acc[mt][nt][j];
          acc[mt][nt][j] = 0.0f;
        }
    __syncthreads();                                         // the buffer written two units ago was read before the previous meeting
    if ((int)threadIdx.x < RED_FLOATS) {
      const float* src = red + buf * WARPS * RED_FLOATS + threadIdx.x;
      float s = 0.0f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) s += src[w * RED_FLOATS];      // warp order: a fixed summation order
      const int row = (int)threadIdx.x / TOKENS, m = (int)threadIdx.x % TOKENS;
      const int n = u * UNIT_ROWS + row;
      if (((mask >> (row >> 4)) & 1u) && m < a.M && n < a.g.N) a.y[(size_t)m * a.g.N + n] = __float2bfloat16_rn(ts * s);
    }
    buf ^= 1;
  }
  cp_async_wait<0>();
}

}  // namespace direct_path

// ------------------------------------------------------------------ host side
static int direct_sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

struct DirectPlan {
  int halves, grid, unit_aligned;
  double balance;            // useful share of the SMs' time: rows are not split over K
};

// Rows go to CTAs either in whole 32-row units or in 16-row halves.  Halves balance better, but a unit shared
// by two CTAs is walked by both, and every walk pays the per-chunk scaffolding again.  The busiest CTA's cost
// per chunk, in instructions (measured: about 110 of scaffolding per walk, 104 per 16-row tile), decides.
static DirectPlan direct_plan(const razer_desc* d) {
  const Geometry g = make_geometry(d->N, d->K);
  const int sms = direct_sm_count();
  const double walk = 110.0, tile = 104.0;
  DirectPlan p;
  p.halves = (g.row_tiles * TILE_ROWS) / 16;         // even: row tiles are 128 rows
  const int units = p.halves / 2;
  p.grid = units < sms ? units : sms;
  const int units_max = (units + p.grid - 1) / p.grid;
  const double cost_units = units_max * (walk + 2 * tile);
  double cost_halves = cost_units;
  if (units > sms) {
    const int halves_max = (p.halves + sms - 1) / sms;
    const int walks = halves_max / 2 + 1;            // worst case: a range that starts in the middle of a unit
    cost_halves = walks * walk + halves_max * tile;
  }
  p.unit_aligned = cost_units <= cost_halves ? 1 : 0;
  const double cost = p.unit_aligned ? cost_units : cost_halves;
  p.balance = p.halves * (tile + walk / 2) / (sms * cost);
  return p;
}

bool gemv_direct_supported(const razer_desc* d, int M) {
  const Geometry g = make_geometry(d->N, d->K);
  return M >= 1 && M <= 16 && g.k_chunks >= direct_path::WARPS &&
         (long long)g.row_tiles * g.k_chunks < (1ll << 30);
}

double gemv_direct_balance(const razer_desc* d) { return direct_plan(d).balance; }

template <int NT>
static int launch_direct_cfg(const direct_path::Args& a, int grid, cudaStream_t st) {
  using C = direct_path::Cfg<NT>;
  auto kern = direct_path::razer_direct_kernel<NT>;
  static bool attr_set = false;
  if (!attr_set) {
    RAZER_TRY(check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES),
                         "cudaFuncSetAttribute(max dynamic shared memory)"));
    attr_set = true;
  }
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(direct_path::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, a);
  count_launches(1);
  return check_cuda(e, "razer_direct_kernel launch");
}

int launch_gemv_direct(const razer_desc* d, const void* packed, const void* x, int M, float extra_scale,
                       const float* extra_scale_dev, void* y, cudaStream_t st) {
  const DirectPlan p = direct_plan(d);
  direct_path::Args a;
  a.packed = (const uint8_t*)packed;
  a.x = (const __nv_bfloat16*)x;
  a.y = (__nv_bfloat16*)y;
  a.extra_scale = extra_scale_dev;
  a.g = make_geometry(d->N, d->K);
  a.sv0 = d->sv_mag[0];
  a.sv1 = d->sv_mag[1];
  a.tensor_scale = d->tensor_scale * extra_scale;
  a.mul_lo = (1u << 6) + (1u << 12);
  a.mul_hi = (1u << 2) + (1u << 8);
  a.M = M;
  a.halves = p.halves;
  a.unit_aligned = p.unit_aligned;
  return M <= 8 ? launch_direct_cfg<1>(a, p.grid, st) : launch_direct_cfg<2>(a, p.grid, st);
}

}  // namespace razer
