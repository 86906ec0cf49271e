// Decode GEMV / very skinny GEMM (M <= 16) against packed RaZeR weights for sm_100a.
//
//   y[m, n] = bf16( ts * sum_k x[m, k] * D1[n, k] ),   D1 = block_scale * element (exact bf16)
//
// The path is bound by the stream of packed weights from HBM and, on the SM, by the
// instructions that decode them.  The decoded bf16 pairs therefore never leave registers:
// they are the A fragment of a warp-level m16n8k16 tensor-core MMA whose B fragment is the
// activation slice (tokens along n), so the multiply-accumulate costs one instruction per
// 256 weights and the accumulation is FP32.  Sec. 4.3 of the paper describes the same idea for
// its weight-only kernel (weights pre-shuffled so that each thread's loads match its fragment).
//
// Data movement: one producer warp streams stages of CH packed chunks (one bulk copy) plus
// the matching activation box (one tensor-map load, 128-byte swizzle) into a ring of shared
// memory stages guarded by full / empty mbarriers; eight compute warps consume them.
//
// Thread mapping inside a stage (128 weight rows x CH * 64 columns): compute warp w owns rows
// 32 * (w & 3) .. + 31 (two 16-row MMA tiles) and the chunks of parity w >> 2.  In a chunk,
// lane (g = lane / 4, t = lane % 4) decodes block t (16 columns) of rows g and g + 8 of each
// tile; MMA q (0..3) of the chunk takes elements 4q .. 4q + 3 of every lane's block, i.e. the
// MMA's 16 k slots are columns 16 t + 4 q + {0, 1, 2, 3}, t = 0..3, of the chunk, for A and B
// alike.  Each lane thus handles whole 16-element blocks and fetches a block's scale once.
//
// Work partition and reduction are those of the tcgen05 kernel (razer_gemm_umma.cu): stripes
// of (row tile, k stage) items, partial tiles through per-CTA FP32 slots, last arrival sums.
// Every wait is bounded and reports through the workspace status word.
#include <cuda.h>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_decode.cuh"

namespace razer {

namespace mma_path {

constexpr uint32_t WAIT_LIMIT = 1u << 26;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;
constexpr int COMPUTE_WARPS = 16;
constexpr int KQ = COMPUTE_WARPS / 4;                 // warps that share 32 rows split a stage's chunks KQ ways
constexpr int THREADS = 32 * (1 + COMPUTE_WARPS);
constexpr size_t WS_STATUS_BYTES = 256;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One poll of a barrier phase.  The hint lets the hardware park the thread until the phase
// completes (or about the hinted time passes) instead of spinning in the issue slots that
// the decoding warps need.
constexpr uint32_t WAIT_SLICE_NS = 1000000u;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(WAIT_SLICE_NS)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait; false = gave up (or another thread already flagged a failure).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();                     // only waits that already lasted a slice get here
  for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// D (+)= A(16 x 16, row) * B(16 x 8, col), bf16 inputs, FP32 accumulation.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct Args {
  const uint8_t* packed;
  __nv_bfloat16* y;
  float* slots;              // [grid][2][8 * NTILES][128] FP32 partial tiles
  uint32_t* counters;        // one per row tile, zero between calls
  uint32_t* status;          // device status word
  const float* extra_scale;  // optional device scalar multiplied into the tensor scale
  Geometry g;
  float sv0, sv1, tensor_scale;
  uint32_t mul_lo, mul_hi;   // 2^6 + 2^12 and 2^2 + 2^8 (razer_decode.cuh)
  int M, steps_per_tile, total_items;
  int x_map_3d;              // activation tensor map is the 3-D (64 k, tokens, k chunk) view
};

template <int NTILES, int CH, int STAGES>
struct Cfg {
  static constexpr int TOKENS = 8 * NTILES;
  static constexpr int W_PAD = (CH * CHUNK_BYTES + 1023) / 1024 * 1024;
  static constexpr int X_BOX_BYTES = TOKENS * 128;               // tokens x 64 k x 2 B
  static constexpr int STAGE_BYTES = W_PAD + CH * X_BOX_BYTES;
  static constexpr int NUM_BARS = 2 * STAGES + 2;
  static constexpr int RED_BYTES = (KQ - 1) * TILE_ROWS * TOKENS * 4;   // partial sums of the warps with kq > 0
  static constexpr size_t SMEM_BYTES =
      1024 + (size_t)STAGES * STAGE_BYTES + RED_BYTES + DECODE_TABLE_BYTES + NUM_BARS * 8 + 64;
};

__device__ __forceinline__ int cta_of_item(long long item, int grid, long long total) {
  return (int)((((item + 1) * grid) - 1) / total);
}

template <int NTILES, int CH, int STAGES>
__global__ void __launch_bounds__(THREADS, 1)
razer_mma_kernel(const __grid_constant__ CUtensorMap tmap_x, const Args a) {
  using C = Cfg<NTILES, CH, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  float* red = reinterpret_cast<float*>(smem + (size_t)STAGES * C::STAGE_BYTES);
  uint8_t* tables = reinterpret_cast<uint8_t*>(red) + C::RED_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tables + DECODE_TABLE_BYTES);
  uint32_t* flags = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
  volatile uint32_t* abort_flag = flags;
  uint32_t* bcast = flags + 1;

  const uint32_t bar_full = smem_u32(bars);             // [STAGES] TMA -> compute warps
  const uint32_t bar_empty = bar_full + 8 * STAGES;     // [STAGES] compute warps -> TMA (one arrival per warp)
  const uint32_t bar_all = bar_empty + 8 * STAGES;      // rendezvous of the 256 compute threads
  const uint32_t bar_epi = bar_all + 8;                 // rendezvous of the 128 epilogue threads

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grid = gridDim.x, cta = blockIdx.x;
  const int it_begin = (int)(((long long)a.total_items * cta) / grid);
  const int it_end = (int)(((long long)a.total_items * (cta + 1)) / grid);
  const int n_items = it_end - it_begin;
  const int spt = a.steps_per_tile;
  int tile = it_begin / spt, step = it_begin - tile * spt;
  int stage = 0, phase = 0;
  auto advance = [&]() {
    if (++step == spt) { step = 0; ++tile; }
    if (++stage == STAGES) { stage = 0; phase ^= 1; }
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, COMPUTE_WARPS);
    }
    mbar_init(bar_all, 32 * COMPUTE_WARPS);
    mbar_init(bar_epi, 128);
    flags[0] = 0;
    flags[2] = 0;                                       // a flag nobody sets (used by the drain waits)
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  auto fail = [&](uint32_t code) {
    *abort_flag = 1;
    grid_dep_wait();                                      // the status word lives in the (possibly shared) workspace
    atomicCAS(a.status, 0u, code);
  };
  // Producer state (thread 0).  Weights depend on nothing and start at once; activation boxes wait for
  // the preceding kernel of the stream (programmatic dependent launch).
  int issued = 0;
  auto produce_x = [&](int stg, int stp) {
    const int c0 = stp * CH;
    const int nch = min(CH, a.g.k_chunks - c0);
    const uint32_t st = smem_u32(smem) + (uint32_t)stg * C::STAGE_BYTES;
    const uint32_t bar = bar_full + 8 * stg;
    if (a.x_map_3d) {
      tma_load_3d(st + C::W_PAD, &tmap_x, 0, 0, c0, bar);
    } else {
      for (int c = 0; c < nch; ++c) tma_load_2d(st + C::W_PAD + c * C::X_BOX_BYTES, &tmap_x, (c0 + c) * CHUNK_K, 0, bar);
    }
  };
  auto produce = [&](bool with_x) {
    const int c0 = step * CH;
    const int nch = min(CH, a.g.k_chunks - c0);
    const uint32_t st = smem_u32(smem) + (uint32_t)stage * C::STAGE_BYTES;
    const uint32_t bar = bar_full + 8 * stage;
    const uint32_t n_x = a.x_map_3d ? CH : nch;           // the 3-D box always spans CH chunks (zero-filled past K)
    mbar_expect_tx(bar, (uint32_t)(nch * CHUNK_BYTES) + n_x * C::X_BOX_BYTES);
    bulk_copy_g2s(st, a.packed + ((size_t)tile * a.g.k_chunks + c0) * CHUNK_BYTES, (uint32_t)(nch * CHUNK_BYTES), bar);
    if (with_x) produce_x(stage, step);
    advance();
  };
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    grid_dep_launch();
    const int t0 = tile, s0 = step;
    for (; issued < n_items && issued < STAGES; ++issued) produce(false);
    grid_dep_wait();
    int t2 = t0, s2 = s0;
    for (int i = 0; i < issued; ++i) {
      produce_x(i, s2);
      if (++s2 == spt) { s2 = 0; ++t2; }
    }
    (void)t2;
  }
  if (warp != 0) decode_tables_fill(tables, a.sv0, a.sv1, threadIdx.x - 32, THREADS - 32);
  __syncthreads();

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      for (; issued < n_items; ++issued) {
        if (!mbar_wait(bar_empty + 8 * stage, (uint32_t)phase ^ 1u, abort_flag)) { fail(21); break; }
        produce(true);
      }
      // Drain: copies still in flight must land before this CTA's shared memory is released.
      const int pending = issued < STAGES ? issued : STAGES;
      for (int f = issued - pending; f < issued; ++f)
        mbar_wait(bar_full + 8 * (f % STAGES), (uint32_t)((f / STAGES) & 1), flags + 2);
    }
  } else {
    // ===================== compute warps =====================
    const int cw = warp - 1;
    const int rg = cw & 3, half = cw >> 2;              // half = kq: which share of the chunks
    const int g = lane >> 2, t = lane & 3;
    const bool epi_warp = (half == 0);
    const bool leader = (cw == 0 && lane == 0);
    const DecodeTables dt = decode_tables_view(tables, lane);
    const uint32_t mul_lo = a.mul_lo, mul_hi = a.mul_hi;
    float ts = a.tensor_scale;                           // (x extra scale: read after the grid dependency)
    bool dep_waited = false;
    uint32_t all_phase = 0, epi_phase = 0;
    auto wait_all = [&](uint32_t bar, uint32_t parity, uint32_t code) -> bool {
      const bool got = mbar_wait(bar, parity, abort_flag);
      if (!got) fail(code);
      return __all_sync(0xFFFFFFFFu, got);
    };
    auto sync_all = [&]() -> bool {                     // bounded rendezvous of the 256 compute threads
      mbar_arrive(bar_all);
      const bool got = wait_all(bar_all, all_phase & 1u, 22);
      ++all_phase;
      return got;
    };
    auto sync_epi = [&]() -> bool {                     // bounded rendezvous of the 128 epilogue threads
      mbar_arrive(bar_epi);
      const bool got = wait_all(bar_epi, epi_phase & 1u, 23);
      ++epi_phase;
      return got;
    };
    // byte offsets that do not change: this lane's code words of rows (g, g + 8) of both tiles in
    // block t, its rows' scale words, and its B-fragment positions inside an activation box
    int code_off[2][2], scale_off[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = 32 * rg + 16 * mt + 8 * h + g;
        code_off[mt][h] = packed_code_offset(t, r);
        scale_off[mt][h] = CHUNK_CODE_BYTES + r * 4;
      }
    int xb_off[NTILES][4];
#pragma unroll
    for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
      for (int q = 0; q < 4; ++q)                         // token 8 nt + g, columns 16 t + 4 q .. + 3, 128-byte swizzle
        xb_off[nt][q] = (8 * nt + g) * 128 + (((2 * t + (q >> 1)) ^ g) << 4) + 8 * (q & 1);

    float acc[2][NTILES][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[mt][nt][j] = 0.0f;

    for (int i = 0; i < n_items; ++i, advance()) {
      const bool seg_last = (i + 1 == n_items) || step == spt - 1;
      const int nch = min(CH, a.g.k_chunks - step * CH);
      if (!wait_all(bar_full + 8 * stage, (uint32_t)phase, 24)) break;
      const uint32_t st = smem_addr(smem) + (uint32_t)stage * C::STAGE_BYTES;
#pragma unroll
      for (int cc = 0; cc < (CH + KQ - 1) / KQ; ++cc) {
        const int c = KQ * cc + half;
        if (c < nch) {
          const uint32_t ck = st + c * CHUNK_BYTES;
          const uint32_t xk = st + C::W_PAD + c * C::X_BOX_BYTES;
          uint2 xb[NTILES][4];
#pragma unroll
          for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
            for (int q = 0; q < 4; ++q) xb[nt][q] = lds64(xk + xb_off[nt][q]);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            uint32_t e[2][8];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint2 cwd = lds64(ck + code_off[mt][h]);
              const uint32_t sb = lds32(ck + scale_off[mt][h]) >> (8 * t);
              uint32_t ss2;
              SvConsts svc;
              decode_block_consts_byte(dt, sb, ss2, svc);
              decode_word(cwd.x, ss2, svc, mul_lo, mul_hi, e[h]);
              decode_word(cwd.y, ss2, svc, mul_lo, mul_hi, e[h] + 4);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
              for (int nt = 0; nt < NTILES; ++nt)
                mma_16816(acc[mt][nt], e[0][2 * q], e[1][2 * q], e[0][2 * q + 1], e[1][2 * q + 1], xb[nt][q].x, xb[nt][q].y);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
      if (!seg_last) continue;

      // ---------------- end of a segment: fold the two chunk parities, then store or publish ----------------
      const int it = it_begin + i;
      const int tile_begin = tile * spt;
      const int seg_begin = it_begin > tile_begin ? it_begin : tile_begin;
      const bool complete = (seg_begin == tile_begin) && (step == spt - 1);
      if (half >= 1) {
        float* red_w = red + (half - 1) * (TILE_ROWS * C::TOKENS);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int r = 32 * rg + 16 * mt + 8 * (j >> 1) + g, m = 8 * nt + 2 * t + (j & 1);
              red_w[m * TILE_ROWS + r] = acc[mt][nt][j];
              acc[mt][nt][j] = 0.0f;
            }
      }
      if (!sync_all()) break;
      if (half == 0) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int r = 32 * rg + 16 * mt + 8 * (j >> 1) + g, m = 8 * nt + 2 * t + (j & 1);
              for (int q = 0; q < KQ - 1; ++q) acc[mt][nt][j] += red[q * (TILE_ROWS * C::TOKENS) + m * TILE_ROWS + r];
            }
      }
      if (!sync_all()) break;                               // `red` may be rewritten after this
      if (!epi_warp) continue;
      if (!dep_waited) {                                   // outputs, workspace and the scale scalar may belong to the preceding kernel
        grid_dep_wait();
        if (a.extra_scale) ts *= *a.extra_scale;
        dep_waited = true;
      }
      const int slot_idx = (seg_begin == it_begin) ? 0 : 1;           // first segment of the stripe or not
      float* my_slot = a.slots + ((size_t)cta * 2 + slot_idx) * (size_t)(C::TOKENS * TILE_ROWS);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int r = 32 * rg + 16 * mt + 8 * (j >> 1) + g, m = 8 * nt + 2 * t + (j & 1);
            const int n_out = tile * TILE_ROWS + r;
            if (complete) {
              if (n_out < a.g.N && m < a.M) a.y[(size_t)m * a.g.N + n_out] = __float2bfloat16_rn(ts * acc[mt][nt][j]);
            } else if (m < a.M) {
              my_slot[m * TILE_ROWS + r] = acc[mt][nt][j];
            }
            acc[mt][nt][j] = 0.0f;
          }
      if (complete) continue;
      // ---------------- partial tile: publish, count, last arrival reduces ----------------
      if (!sync_epi()) break;                                         // all slot stores of this CTA are done (CTA scope)
      const int tile_end = tile_begin + spt;
      const int c_first = cta_of_item(tile_begin, grid, a.total_items);
      const int c_last = cta_of_item(tile_end - 1, grid, a.total_items);
      if (leader) {
        const uint32_t parts = (uint32_t)(c_last - c_first + 1);
        // release: the CTA's slot stores become visible with the count; acquire: the last arrival sees all of them
        uint32_t prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(a.counters + tile) : "memory");
        const uint32_t last = (prev + 1 == parts) ? 1u : 0u;
        if (last) a.counters[tile] = 0;                               // leave the counter ready for the next call
        *bcast = last;
      }
      if (!sync_epi()) break;
      const bool finisher = *reinterpret_cast<volatile uint32_t*>(bcast) != 0;
      if (!sync_epi()) break;                                         // bcast may be rewritten after this
      if (!finisher) continue;
      {
        float sum[2][NTILES][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) sum[mt][nt][j] = 0.0f;
        // ascending CTA order (a fixed summation order); all of a CTA's values are loaded before they are added
        for (int c = c_first; c <= c_last; ++c) {
          const long long b_c = ((long long)a.total_items * c) / grid;
          const int sl = (b_c / spt == tile) ? 0 : 1;
          const float* src = a.slots + ((size_t)c * 2 + sl) * (size_t)(C::TOKENS * TILE_ROWS);
          float part[2][NTILES][4];
#pragma unroll
          for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int r = 32 * rg + 16 * mt + 8 * (j >> 1) + g, m = 8 * nt + 2 * t + (j & 1);
                part[mt][nt][j] = (m < a.M) ? __ldcg(src + m * TILE_ROWS + r) : 0.0f;
              }
#pragma unroll
          for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
              for (int j = 0; j < 4; ++j) sum[mt][nt][j] += part[mt][nt][j];
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int r = 32 * rg + 16 * mt + 8 * (j >> 1) + g, m = 8 * nt + 2 * t + (j & 1);
              const int n_out = tile * TILE_ROWS + r;
              if (n_out < a.g.N && m < a.M) a.y[(size_t)m * a.g.N + n_out] = __float2bfloat16_rn(ts * sum[mt][nt][j]);
            }
      }
      (void)it;
    }
  }
}

}  // namespace mma_path

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn mma_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

static int mma_sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

constexpr int MMA_CH = 4;

struct MmaPlan {
  int ntiles, steps_per_tile, total_items, grid;
  size_t counters_bytes, slots_bytes;
};

static MmaPlan mma_plan(const razer_desc* d, int M) {
  MmaPlan p;
  const Geometry g = make_geometry(d->N, d->K);
  p.ntiles = M <= 8 ? 1 : 2;
  p.steps_per_tile = (g.k_chunks + MMA_CH - 1) / MMA_CH;
  const long long items = (long long)g.row_tiles * p.steps_per_tile;
  p.total_items = (int)items;
  const int sms = mma_sm_count();
  p.grid = (int)(items < sms ? items : sms);
  p.counters_bytes = ((size_t)g.row_tiles * sizeof(uint32_t) + 255) / 256 * 256;
  p.slots_bytes = (size_t)p.grid * 2 * (8 * p.ntiles) * TILE_ROWS * sizeof(float);
  return p;
}

bool gemv_mma_supported(const razer_desc* d, int M) {
  const Geometry g = make_geometry(d->N, d->K);
  const long long items = (long long)g.row_tiles * ((g.k_chunks + MMA_CH - 1) / MMA_CH);
  return M >= 1 && M <= 16 && items < (1ll << 30);
}

size_t gemv_mma_workspace_bytes(const razer_desc* d, int M) {
  const MmaPlan p = mma_plan(d, M);
  const size_t slots = (size_t)(p.grid > 148 ? p.grid : 148) * 2 * (8 * p.ntiles) * TILE_ROWS * sizeof(float);
  return mma_path::WS_STATUS_BYTES + p.counters_bytes + slots;
}

size_t gemv_mma_workspace_zero_bytes(const razer_desc* d, int M) {
  return mma_path::WS_STATUS_BYTES + mma_plan(d, M).counters_bytes;
}

template <int NTILES, int CH, int STAGES>
static int mma_launch_cfg(const CUtensorMap& tmap, const mma_path::Args& args, int grid, cudaStream_t st) {
  using C = mma_path::Cfg<NTILES, CH, STAGES>;
  auto kern = mma_path::razer_mma_kernel<NTILES, CH, STAGES>;
  static bool attr_set = false;
  if (!attr_set) {
    RAZER_TRY(check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES),
                         "cudaFuncSetAttribute(max dynamic shared memory)"));
    attr_set = true;
  }
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(mma_path::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmap, args);
  count_launches(1);
  return check_cuda(e, "razer_mma_kernel launch");
}

int launch_gemv_mma(const razer_desc* d, const void* packed, const void* x, int M, float extra_scale,
                    const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  const Geometry g = make_geometry(d->N, d->K);
  const MmaPlan p = mma_plan(d, M);
  const size_t need = mma_path::WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
  if (!ws || ws_bytes < need)
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  EncodeTiledFn enc = mma_encode_fn();
  if (!enc) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const int tokens = 8 * p.ntiles;
  CUtensorMap tmap;
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = CUDA_ERROR_UNKNOWN;
  int map_3d = 0;
  if (d->K % CHUNK_K == 0) {
    const cuuint64_t dims[3] = {(cuuint64_t)CHUNK_K, (cuuint64_t)M, (cuuint64_t)(d->K / CHUNK_K)};
    const cuuint64_t strides[2] = {(cuuint64_t)d->K * 2, (cuuint64_t)CHUNK_K * 2};
    const cuuint32_t box[3] = {(cuuint32_t)CHUNK_K, (cuuint32_t)tokens, (cuuint32_t)MMA_CH};
    r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    map_3d = (r == CUDA_SUCCESS);
  }
  if (!map_3d) {
    const cuuint64_t dims[2] = {(cuuint64_t)d->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)d->K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)CHUNK_K, (cuuint32_t)tokens};
    r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);

  mma_path::Args a;
  a.packed = (const uint8_t*)packed;
  a.y = (__nv_bfloat16*)y;
  a.status = (uint32_t*)ws;
  a.counters = (uint32_t*)((char*)ws + mma_path::WS_STATUS_BYTES);
  a.slots = (float*)((char*)ws + mma_path::WS_STATUS_BYTES + p.counters_bytes);
  a.extra_scale = extra_scale_dev;
  a.g = g;
  a.sv0 = d->sv_mag[0];
  a.sv1 = d->sv_mag[1];
  a.tensor_scale = d->tensor_scale * extra_scale;
  a.mul_lo = (1u << 6) + (1u << 12);
  a.mul_hi = (1u << 2) + (1u << 8);
  a.M = M;
  a.steps_per_tile = p.steps_per_tile;
  a.total_items = p.total_items;
  a.x_map_3d = map_3d;
  if (p.ntiles == 1) return mma_launch_cfg<1, MMA_CH, 8>(tmap, a, p.grid, st);
  return mma_launch_cfg<2, MMA_CH, 7>(tmap, a, p.grid, st);
}

}  // namespace razer
