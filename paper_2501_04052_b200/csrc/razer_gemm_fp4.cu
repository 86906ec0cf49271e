// Two-pass block-scaled FP4 matmul of RaZeR weights against plain-NVFP4 activations (App. D.3) on the
// 5th-generation tensor core (tcgen05.mma kind::mxf4nvf4, block 16, UE4M3 scale factors).
//
//   y[m, n] = bf16( ts_w * ts_a * sum_k A[m, k] * (B_main[n, k] + B_comp[n, k]) )
//
// B_main keeps every ordinary code and puts a signed FP4 base value where the block's special value sits,
// B_comp holds the signed FP4 remainder there and zero elsewhere (base + remainder = special value).  Both
// share the block's scale byte: the 6-bit E3M3 code is an E4M3 code with a clear top bit, so the masked byte
// is the hardware's UE4M3 scale factor as it stands.  The two passes are two MMAs per 64-column chunk into
// the same TMEM accumulator; neither matrix exists in global memory.
//
// Mapping: the weight tile is the MMA's A operand (128 rows), the token tile its B operand (128 tokens, or 256
// when there are more than 128), both K-major FP4 in shared memory with the 128-byte swizzle (one row = 256
// codes = one stage of four chunks).  Warp 0 = weight producer (TMA box of packed bytes into a ring of its own,
// released by the remap warps as soon as they have read it), warp 1 = TMEM owner and MMA issuer, warps 2..17 =
// remap (thread = weight row and one of a stage's four chunks; all sixteen warps take every stage, alternating
// between two operand slots so that one stage is remapped while the previous one is multiplied)
// and epilogue, warp 18 = activation producer (codes by TMA, scale-factor tiles by bulk copy, into a ring
// released by the MMAs' completion).  A remap thread reads its row's packed blocks, finds the special-value
// nibbles (the only nibbles that are 0x0 in the packed form), builds the two code words with two integer
// multiply-adds, applies the block's stored-negated flag to the sign bits, and writes both rows plus the row's
// four scale bytes (scale-factor layout: 32 x 16-byte rows, row r % 32, word r / 32).  The MMA warp copies
// the scale factors of both operands to TMEM (tcgen05.cp) and issues main and comp MMAs.
//
// The activation operand is prepared by a small kernel before the matmul: codes padded to whole stages with
// the nibbles of every 32-bit word in the packed form's order (the contraction does not care about the order
// of k inside a block as long as both operands agree), scale bytes masked to 7 bits and laid out as the
// scale-factor tiles the MMA reads.
//
// Work partition, partial tiles and bounded waits are those of the bf16 tcgen05 kernel: a persistent grid,
// contiguous stripes of (tile, stage) items, partial tiles through FP32 slots and a per-tile counter.
#include <cuda.h>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_ptx.cuh"
#include "razer_tcgen05.cuh"

namespace razer {
namespace fp4_path {

constexpr int CH = 4;                                 // chunks per stage: 256 codes = one 128-byte swizzled row
constexpr int WSTAGES = 4;                            // packed-weight ring (released by the remap warps)
constexpr int ASTAGES = 2;                            // remapped-operand ring: one slot is remapped while the other is multiplied
constexpr int NRW = 16;                               // remap warps: four per chunk of a stage
constexpr int THREADS = 64 + 32 * NRW + 32;           // + W producer, MMA warp, X producer
constexpr int W_BYTES = CH * CHUNK_BYTES;             // 18432 packed weight bytes of a stage
constexpr int SF_TILE_BYTES = 512;                    // scale factors of 128 rows x one chunk
constexpr int SF_BYTES = CH * SF_TILE_BYTES;          // ... x one stage
constexpr int A_TILE_BYTES = TILE_ROWS * 128;         // 128 rows x 256 codes
constexpr int ASTAGE_BYTES = 2 * A_TILE_BYTES + SF_BYTES;

// NT = tokens per tile (the MMA's N): 128, or 256 when there are more than 128 tokens (half the weight traffic
// and remap work per flop).
template <int NT>
struct Cfg {
  static constexpr int XSTAGES = NT == 128 ? 3 : 2;               // activation ring (released by the MMAs' completion)
  static constexpr int X_CODE_BYTES = NT * 128;
  static constexpr int X_BYTES = X_CODE_BYTES + (NT / 128) * SF_BYTES;   // codes + scale-factor tiles
  static constexpr int NACC = NT == 128 ? 2 : 1;                  // accumulators (main / comp passes apart when they fit)
  static constexpr int ACC_COLS = NACC * NT;
  static constexpr int SFB_COLS = CH * 4 * (NT / 128);
  static constexpr int SF_COLS = CH * 4 + SFB_COLS;               // per operand ring slot: A and B scale factors of a stage
  static constexpr int TMEM_COLS = 512;
  static constexpr int NUM_BARS = 2 * WSTAGES + 2 * XSTAGES + 2 * ASTAGES + 4;
  static constexpr size_t SMEM_BYTES =
      1024 + (size_t)WSTAGES * W_BYTES + (size_t)XSTAGES * X_BYTES + (size_t)ASTAGES * ASTAGE_BYTES + NUM_BARS * 8 + 64;
  // E2M1 x E2M1 -> FP32, UE4M3 scale factors, both operands K-major, M = 128, N = NT
  static constexpr uint32_t IDESC = (1u << 7) | (1u << 10) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  static_assert(W_BYTES % 1024 == 0 && X_BYTES % 1024 == 0 && ASTAGE_BYTES % 1024 == 0, "swizzled tiles sit on 1024 bytes");
  static_assert(ACC_COLS + ASTAGES * SF_COLS <= TMEM_COLS, "TMEM budget");
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

struct Args {
  __nv_bfloat16* y;
  const uint8_t* sfb;        // activation scale factors: [128-token tile][stage][chunk] tiles of 512 bytes
  float* slots;              // [grid][2][NT][128] FP32 partial tiles
  uint32_t* counters;        // one per output tile, zero between calls
  uint32_t* status;          // device status word
  const float* extra_scale;  // device scalar multiplied into the tensor scale (the activations' tensor scale)
  Geometry g;
  float tensor_scale;
  uint32_t base0, rem0, base1, rem1;   // FP4 codes of the base value and the remainder for select 0 / 1
  int M, token_tiles, steps_per_tile;
  long long total_items;
};

// D[tmem] (+)= A[smem] * B[smem], FP4 operands with one UE4M3 scale factor per 16 elements read from TMEM.
__device__ __forceinline__ void mma_fp4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                        uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 ad, bd;\n\t"
      "setp.ne.b32 p, %7, 0;\n\t"
      "mov.b64 ad, {%1, %3};\n\t"
      "mov.b64 bd, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], ad, bd, %4, [%5], [%6], p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}
// 32 rows x 16 bytes of shared memory -> 4 TMEM columns, the same in all four 32-lane quarters.
__device__ __forceinline__ void copy_sf_to_tmem(uint32_t tmem, uint32_t saddr) {
  // no swizzle; eight 16-byte rows are contiguous, groups of eight rows 128 bytes apart
  const uint32_t lo = (saddr & 0x3FFFFu) >> 4;
  const uint32_t hi = (128u >> 4) | (1u << 14);
  asm volatile(
      "{\n\t.reg .b64 sd;\n\t"
      "mov.b64 sd, {%1, %2};\n\t"
      "tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], sd;\n\t}" ::"r"(tmem),
      "r"(lo), "r"(hi)
      : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// writes made through the generic proxy become visible to the tensor core's (asynchronous proxy) reads
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Upper half of an operand's shared-memory descriptor: 1024-byte group stride, descriptor version, 128-byte swizzle.
constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);

// Position of a role inside the CTA's stripe of work items, with the slot and parity of each ring.
template <int XSTAGES>
struct Cursor {
  int tile, step;
  int ws, wph, xs, xph, as, aph;
  __device__ __forceinline__ void next(int steps_per_tile) {
    if (++step == steps_per_tile) { step = 0; ++tile; }
    if (++ws == WSTAGES) { ws = 0; wph ^= 1; }
    if (++xs == XSTAGES) { xs = 0; xph ^= 1; }
    if (++as == ASTAGES) { as = 0; aph ^= 1; }
  }
};

template <int NT>
__global__ void __launch_bounds__(THREADS, 1)
razer_fp4_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const Args a) {
  using C = Cfg<NT>;
  constexpr int XSTAGES = C::XSTAGES;
  constexpr int X_WARP = 2 + NRW;                       // the activation producer
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem_w = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_x = smem_w + (size_t)WSTAGES * W_BYTES;
  uint8_t* smem_a = smem_x + (size_t)XSTAGES * C::X_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_a + (size_t)ASTAGES * ASTAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t bar_wfull = smem_u32(bars);            // [WSTAGES] TMA -> remap
  const uint32_t bar_wempty = bar_wfull + 8 * WSTAGES;  // [WSTAGES] remap warps -> TMA
  const uint32_t bar_xfull = bar_wempty + 8 * WSTAGES;  // [XSTAGES] TMA -> MMA
  const uint32_t bar_xempty = bar_xfull + 8 * XSTAGES;  // [XSTAGES] MMA commit -> TMA
  const uint32_t bar_afull = bar_xempty + 8 * XSTAGES;  // [ASTAGES] remap -> MMA
  const uint32_t bar_aempty = bar_afull + 8 * ASTAGES;  // [ASTAGES] MMA commit -> remap
  const uint32_t bar_accfull = bar_aempty + 8 * ASTAGES;
  const uint32_t bar_accempty = bar_accfull + 8;
  const uint32_t bar_epi = bar_accempty + 8;            // rendezvous of the epilogue threads
  const uint32_t bar_drain = bar_epi + 8;               // the MMA warp's own MMAs have all completed

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grid = gridDim.x, cta = blockIdx.x;
  const int it_begin = (int)((a.total_items * cta) / grid);
  const int it_end = (int)((a.total_items * (cta + 1)) / grid);
  const int n_items = it_end - it_begin;
  const int spt = a.steps_per_tile;
  Cursor<XSTAGES> cur;
  cur.tile = it_begin / spt;
  cur.step = it_begin - cur.tile * spt;
  cur.ws = cur.wph = cur.xs = cur.xph = cur.as = cur.aph = 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < WSTAGES; ++i) {
      mbar_init(bar_wfull + 8 * i, 1);
      mbar_init(bar_wempty + 8 * i, 32 * NRW);
    }
    for (int i = 0; i < XSTAGES; ++i) {
      mbar_init(bar_xfull + 8 * i, 1);
      mbar_init(bar_xempty + 8 * i, 1);
    }
    for (int i = 0; i < ASTAGES; ++i) {
      mbar_init(bar_afull + 8 * i, 32 * NRW);
      mbar_init(bar_aempty + 8 * i, 1);
    }
    mbar_init(bar_accfull, 1);
    mbar_init(bar_accempty, 32 * NRW);
    mbar_init(bar_epi, 32 * NRW);
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    tmem_slot[3] = 0;                                   // a flag nobody sets (used by the drain waits)
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Weight producer state (thread 0 only).  The first ring of weight loads goes out before the rest of the
  // prologue: the packed weights depend on nothing that precedes this kernel in the stream.
  int issued = 0;
  int p_rt = cur.tile / a.token_tiles, p_tt = cur.tile - p_rt * a.token_tiles;
  auto produce_w = [&]() {
    const uint32_t st = smem_u32(smem_w) + (uint32_t)cur.ws * W_BYTES;
    const uint32_t bar = bar_wfull + 8 * cur.ws;
    mbar_expect_tx(bar, (uint32_t)W_BYTES);               // the box always spans CH chunks (zero-filled past the end of K)
    tma_load_3d(st, &tmap_w, 0, cur.step * CH, p_rt * TILE_STRIPS, bar);
    if (cur.step == spt - 1 && ++p_tt == a.token_tiles) { p_tt = 0; ++p_rt; }
    cur.next(spt);
  };
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_w) : "memory");
    grid_dep_launch();
    for (; issued < n_items && issued < WSTAGES; ++issued) produce_w();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_sf0 = tmem_base + C::ACC_COLS;

  auto fail = [&](uint32_t code) {
    *abort_flag = 1;
    grid_dep_wait();                                      // the status word lives in the (possibly shared) workspace
    atomicCAS(a.status, 0u, code);
  };

  if (warp == 0) {
    // ===================== weight producer =====================
    if (lane == 0) {
      for (; issued < n_items; ++issued) {
        if (!mbar_wait(bar_wempty + 8 * cur.ws, (uint32_t)cur.wph ^ 1u, abort_flag)) { fail(21); break; }
        produce_w();
      }
      // copies still in flight must land before this CTA's shared memory is released
      const int pending = issued < WSTAGES ? issued : WSTAGES;
      for (int f = issued - pending; f < issued; ++f)
        mbar_wait(bar_wfull + 8 * (f % WSTAGES), (uint32_t)((f / WSTAGES) & 1), tmem_slot + 3);
    }
  } else if (warp == X_WARP) {
    // ===================== activation producer (codes and scale factors written by the preparation kernel) =====================
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
      grid_dep_wait();
      int tt = cur.tile % a.token_tiles;
      int done = 0;
      for (; done < n_items; ++done) {
        if (done >= XSTAGES && !mbar_wait(bar_xempty + 8 * cur.xs, (uint32_t)cur.xph ^ 1u, abort_flag)) { fail(22); break; }
        const uint32_t st = smem_u32(smem_x) + (uint32_t)cur.xs * C::X_BYTES;
        const uint32_t bar = bar_xfull + 8 * cur.xs;
        mbar_expect_tx(bar, (uint32_t)C::X_BYTES);
        tma_load_2d(st, &tmap_x, cur.step * 128, tt * NT, bar);
#pragma unroll
        for (int h = 0; h < NT / 128; ++h)
          bulk_copy_g2s(st + C::X_CODE_BYTES + h * SF_BYTES,
                        a.sfb + ((size_t)(tt * (NT / 128) + h) * spt + cur.step) * SF_BYTES, SF_BYTES, bar);
        if (cur.step == spt - 1 && ++tt == a.token_tiles) tt = 0;
        cur.next(spt);
      }
      const int pending = done < XSTAGES ? done : XSTAGES;
      for (int f = done - pending; f < done; ++f)
        mbar_wait(bar_xfull + 8 * (f % XSTAGES), (uint32_t)((f / XSTAGES) & 1), tmem_slot + 3);
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (whole warp walks the items, one elected lane issues) =====================
    uint32_t seg = 0;
    auto wait_warp = [&](uint32_t bar, uint32_t parity, uint32_t code) -> bool {
      const bool got = mbar_wait(bar, parity, abort_flag);
      if (!got) fail(code);
      return __all_sync(0xFFFFFFFFu, got);
    };
    for (int i = 0; i < n_items; ++i) {
      const bool seg_first = (i == 0) || cur.step == 0;
      const bool seg_last = (i + 1 == n_items) || cur.step == spt - 1;
      const int nch = min(CH, a.g.k_chunks - cur.step * CH);
      if (!wait_warp(bar_afull + 8 * cur.as, (uint32_t)cur.aph, 23)) break;
      if (!wait_warp(bar_xfull + 8 * cur.xs, (uint32_t)cur.xph, 30)) break;
      if (seg_first && !wait_warp(bar_accempty, (seg & 1u) ^ 1u, 24)) break;
      tc_fence_after();
      const uint32_t xs = smem_u32(smem_x) + (uint32_t)cur.xs * C::X_BYTES;
      const uint32_t sfb_s = xs + C::X_CODE_BYTES;
      const uint32_t am = smem_u32(smem_a) + (uint32_t)cur.as * ASTAGE_BYTES;
      const uint32_t ac = am + A_TILE_BYTES;
      const uint32_t sfa_s = am + 2 * A_TILE_BYTES;
      const uint32_t sf_t = tmem_sf0 + cur.as * C::SF_COLS;
      if (elect_one()) {
        // the stage's scale factors first, then its MMAs back to back
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          if (c < nch) {
            copy_sf_to_tmem(sf_t + c * 4, sfa_s + c * SF_TILE_BYTES);
#pragma unroll
            for (int h = 0; h < NT / 128; ++h)
              copy_sf_to_tmem(sf_t + CH * 4 + c * 4 * (NT / 128) + h * 4, sfb_s + h * SF_BYTES + c * SF_TILE_BYTES);
          }
        }
        // With two accumulators the main and comp passes add into one each (summed in the epilogue), so that
        // consecutive MMAs never share an accumulator.
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          if (c < nch) {
            const uint32_t sfa_t = sf_t + c * 4, sfb_t = sf_t + CH * 4 + c * 4 * (NT / 128);
            // 64 codes further along k: +32 bytes inside the 128-byte rows
            const uint32_t b_lo = ((xs + c * 32) >> 4) | (1u << 16);
            const uint32_t first = (seg_first && c == 0) ? 0u : 1u;
            mma_fp4(tmem_base, ((am + c * 32) >> 4) | (1u << 16), b_lo, DESC_HI, C::IDESC, sfa_t, sfb_t, first);
            mma_fp4(tmem_base + (C::NACC - 1) * NT, ((ac + c * 32) >> 4) | (1u << 16), b_lo, DESC_HI, C::IDESC, sfa_t, sfb_t,
                    C::NACC == 2 ? first : 1u);
          }
        }
        tc_commit(bar_xempty + 8 * cur.xs);
        tc_commit(bar_aempty + 8 * cur.as);
        if (seg_last) tc_commit(bar_accfull);
      }
      __syncwarp();
      if (seg_last) ++seg;
      cur.next(spt);
    }
    // the MMAs issued so far read shared memory and TMEM until they complete: wait for them (bounded, not
    // watching the abort flag) before the CTA may release either
    __syncwarp();
    if (elect_one()) tc_commit(bar_drain);
    __syncwarp();
    mbar_wait(bar_drain, 0u, tmem_slot + 3);
  } else {
    // ===================== remap (thread = weight row) + epilogue =====================
    const int row = 32 * (warp & 3) + lane;              // weight row of the tile = TMEM lane of its outputs
    const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
    // All sixteen warps remap every item: warps w, w + 4, w + 8, w + 12 own the same 32 rows (a warp reaches only the
    // TMEM lanes 32 * (warp % 4) .. + 31, which the epilogue needs) and take one of the stage's four chunks each.
    // The item after it goes into the other operand slot, so its remap runs while this item's MMAs execute.
    const int chunk = (warp - 2) >> 2;
    static_assert(NRW == 4 * CH, "one set of four warps per chunk");
    constexpr int EPI_SETS = NRW / 4;                     // sets of four warps (all lane quarters) share the columns
    const int col_lo = 16 * ((((warp - 2) >> 2) * (NT / 16)) / EPI_SETS);
    const int col_hi = 16 * (((((warp - 2) >> 2) + 1) * (NT / 16)) / EPI_SETS);
    const bool leader = (threadIdx.x == 64);
    float ts = a.tensor_scale;
    bool dep_waited = false;
    uint32_t seg = 0, epi_phase = 0;
    auto wait_all = [&](uint32_t bar, uint32_t parity, uint32_t code) -> bool {
      const bool got = mbar_wait(bar, parity, abort_flag);
      if (!got) fail(code);
      return __all_sync(0xFFFFFFFFu, got);
    };
    auto epi_sync = [&]() -> bool {
      mbar_arrive(bar_epi);
      const bool got = wait_all(bar_epi, epi_phase & 1u, 28);
      ++epi_phase;
      return got;
    };
    const int r16 = row % STRIP_ROWS;
    const uint32_t strip_off = (uint32_t)(row / STRIP_ROWS) * (CH * PIECE_BYTES);
    const uint32_t scale_off = (uint32_t)PIECE_CODE_BYTES + (uint32_t)(r16 & 7) * 8;
    const uint32_t scale_sel = (r16 >> 3) ? 0x7531u : 0x6420u;
    uint32_t code_off[CHUNK_BLOCKS];
#pragma unroll
    for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) code_off[blk] = (uint32_t)piece_code_offset(blk, r16);
    const uint32_t row_off = (uint32_t)row * 128;        // this row inside an operand tile
    const uint32_t sw7 = (uint32_t)row & 7u;              // 128-byte swizzle: 16-byte unit u of row r sits at u ^ (r % 8)
    const uint32_t sf_word = (uint32_t)((row & 31) * 4 + (row >> 5)) * 4;
    for (int i = 0; i < n_items; ++i, cur.next(spt)) {
      const int tile = cur.tile, step = cur.step;
      const bool seg_last = (i + 1 == n_items) || step == spt - 1;
      const int nch = min(CH, a.g.k_chunks - step * CH);
      {
        // every remap thread sees every phase of the barriers it waits on, so the parity waits are sound
        if (!wait_all(bar_aempty + 8 * cur.as, (uint32_t)cur.aph ^ 1u, 26)) break;
        if (!wait_all(bar_wfull + 8 * cur.ws, (uint32_t)cur.wph, 25)) break;
        const uint32_t st = smem_addr(smem_w) + (uint32_t)cur.ws * W_BYTES + strip_off;
        const uint32_t am = smem_addr(smem_a) + (uint32_t)cur.as * ASTAGE_BYTES + row_off;
        const uint32_t ac = am + A_TILE_BYTES;
        const uint32_t sfa = smem_addr(smem_a) + (uint32_t)cur.as * ASTAGE_BYTES + 2 * A_TILE_BYTES + sf_word;
        {
          const int c = chunk;
          if (c < nch) {
            const uint32_t ck = st + c * PIECE_BYTES;
            const uint2 sq = lds64(ck + scale_off);
            const uint32_t sw = __byte_perm(sq.x, sq.y, scale_sel);   // this row's four scale bytes, in block order
            uint2 cw[CHUNK_BLOCKS];
#pragma unroll
            for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) cw[blk] = lds64(ck + code_off[blk]);
            uint32_t mw[8], pw[8];
#pragma unroll
            for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) {
              const uint32_t sb = (sw >> (8 * blk)) & 0xFFu;
              const uint32_t neg8 = (sb & PACKED_NEGATE) ? 0x88888888u : 0u;   // stored negated: flip every sign bit
              const uint32_t base = (sb & PACKED_SELECT) ? a.base1 : a.base0;
              const uint32_t rem = (sb & PACKED_SELECT) ? a.rem1 : a.rem0;
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const uint32_t w = h ? cw[blk].y : cw[blk].x;
                const uint32_t any = w | (w >> 1) | (w >> 2) | (w >> 3);
                const uint32_t z = ~any & 0x11111111u;                         // 1 in every nibble that is 0x0
                mw[2 * blk + h] = (w + z * base) ^ neg8;
                pw[2 * blk + h] = (z * rem) ^ neg8;
              }
            }
            const uint32_t u0 = ((uint32_t)(2 * c) ^ sw7) << 4, u1 = ((uint32_t)(2 * c + 1) ^ sw7) << 4;
            sts128(am + u0, mw[0], mw[1], mw[2], mw[3]);
            sts128(am + u1, mw[4], mw[5], mw[6], mw[7]);
            sts128(ac + u0, pw[0], pw[1], pw[2], pw[3]);
            sts128(ac + u1, pw[4], pw[5], pw[6], pw[7]);
            sts32(sfa + c * SF_TILE_BYTES, sw & 0x3F3F3F3Fu);
          }
        }
        mbar_arrive(bar_wempty + 8 * cur.ws);               // the packed bytes are in registers or written out
        fence_async_smem();
        mbar_arrive(bar_afull + 8 * cur.as);
      }

      if (!seg_last) continue;
      // ---------------- epilogue of the segment that ends with this item ----------------
      const int tile_begin = tile * spt;
      const int seg_begin = it_begin > tile_begin ? it_begin : tile_begin;
      const bool complete = (seg_begin == tile_begin) && (step == spt - 1);
      const int rt = tile / a.token_tiles, tt = tile - rt * a.token_tiles;
      const int n_out = rt * TILE_ROWS + row;
      const int m0 = tt * NT;
      if (!dep_waited) {
        grid_dep_wait();
        if (a.extra_scale) ts *= *a.extra_scale;
        dep_waited = true;
      }
      // A partial tile is finished by its owner, the CTA whose stripe holds the tile's FIRST items: for that CTA the
      // tile is the end of its stripe, for every other CTA of the tile it is the beginning, so their parts were
      // published (FP32 slot in the workspace, then a release-add on the tile's counter) long before the owner gets
      // here.  The owner adds its own accumulator (straight from TMEM) and the other parts in CTA order.
      const int c_first = cta_of_item(tile_begin, grid, a.total_items);
      const int c_last = cta_of_item(tile_begin + spt - 1, grid, a.total_items);
      const bool owner = !complete && cta == c_first;
      if (owner) {
        // acquire: every counted CTA's slot stores are visible to this thread's loads below
        const uint32_t others = (uint32_t)(c_last - c_first);
        uint32_t seen = 0;
        const uint64_t t0 = global_ns();
        for (;;) {
          asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.counters + tile) : "memory");
          if (seen >= others || *abort_flag || global_ns() - t0 > WAIT_LIMIT_NS) break;
          __nanosleep(200);
        }
        const bool ready = seen >= others;
        if (!ready) fail(29);
        if (!__all_sync(0xFFFFFFFFu, ready)) break;
      }
      if (!wait_all(bar_accfull, seg & 1u, 27)) break;
      tc_fence_after();
      float* my_slot = a.slots + (size_t)cta * 2 * (size_t)(NT * TILE_ROWS);   // a non-owner's part is its stripe's first segment
#pragma unroll 1
      for (int c0 = col_lo; c0 < col_hi; c0 += 16) {
        uint32_t v[16];
        tc_ld16(tmem_base + lane_off + c0, v);
        if (C::NACC == 2) {
          uint32_t v1[16];
          tc_ld16(tmem_base + lane_off + NT + c0, v1);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v1[j]));
        } else {
          tc_wait_ld();
        }
        if (complete || owner) {
          if (owner) {
            const int m_valid = a.M - (m0 + c0);                       // tokens of this column group that exist
            // ascending CTA order (a fixed summation order); the loads of two CTAs' slots are in flight together
            for (int cb = c_first + 1; cb <= c_last; cb += 2) {
              float part[2][16];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int c = cb + u <= c_last ? cb + u : c_last;
                const float* src = a.slots + (size_t)c * 2 * (size_t)(NT * TILE_ROWS);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                  part[u][j] = (cb + u <= c_last && j < m_valid) ? __ldcg(src + (c0 + j) * TILE_ROWS + row) : 0.0f;
              }
#pragma unroll
              for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + part[u][j]);
            }
          }
          if (n_out < a.g.N) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int m = m0 + c0 + j;
              if (m < a.M) a.y[(size_t)m * a.g.N + n_out] = __float2bfloat16_rn(ts * __uint_as_float(v[j]));
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (m0 + c0 + j < a.M) my_slot[(c0 + j) * TILE_ROWS + row] = __uint_as_float(v[j]);
        }
      }
      tc_fence_before();
      mbar_arrive(bar_accempty);
      ++seg;
      if (complete) continue;
      if (!epi_sync()) break;                                         // every thread has read the counter / stored its part
      if (leader) {
        if (owner) a.counters[tile] = 0;                              // leave the counter ready for the next call
        // release: the CTA's slot stores (ordered before this by the rendezvous) become visible with the count
        else asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.counters + tile) : "memory");
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS)
                 : "memory");
  }
}

// Activation operand for the kernel above.  codes_out: [M][KP / 8] 32-bit words (KP = K rounded up to whole
// stages, zero beyond K), each word's nibbles in the packed form's order (nibbles p and p + 4 = elements 2p and
// 2p + 1).  sfb: [128-token tile][stage][chunk] tiles of 128 words; word 4 * (t % 32) + t / 32 of a tile holds the
// four 7-bit scale bytes of token t of the tile for the chunk's four blocks (zero for tokens beyond M and
// blocks beyond K).
__global__ void fp4_act_prep_kernel(const uint32_t* __restrict__ codes, const uint8_t* __restrict__ scales, int M, int K,
                                    int KP, int tiles128, int spt, uint32_t* __restrict__ codes_out,
                                    uint32_t* __restrict__ sfb) {
  grid_dep_launch();
  grid_dep_wait();
  const long long row_quads = KP / 32, in_words = K / 8;               // a quad = four 32-bit words = 32 codes
  const long long n_code = (long long)M * row_quads;
  const long long n_sf = (long long)tiles128 * spt * CH * 128;
  const bool vec = (K % 32) == 0 && (reinterpret_cast<uintptr_t>(codes) % 16) == 0;   // rows of the input start on 16 bytes
  auto shuffle = [](uint32_t w) -> uint32_t {                          // element j of the word: nibble j -> nibble j / 2 + 4 (j % 2)
    uint32_t o = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) o |= ((w >> (4 * j)) & 0xFu) << (4 * ((j >> 1) + 4 * (j & 1)));
    return o;
  };
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_code + n_sf;
       i += (long long)gridDim.x * blockDim.x) {
    if (i < n_code) {
      const long long m = i / row_quads, q = i - m * row_quads;
      uint4 w = make_uint4(0u, 0u, 0u, 0u);
      const uint32_t* src = codes + m * in_words + 4 * q;
      if (vec && 4 * q + 3 < in_words) {
        w = *reinterpret_cast<const uint4*>(src);
      } else {
        if (4 * q + 0 < in_words) w.x = src[0];
        if (4 * q + 1 < in_words) w.y = src[1];
        if (4 * q + 2 < in_words) w.z = src[2];
        if (4 * q + 3 < in_words) w.w = src[3];
      }
      reinterpret_cast<uint4*>(codes_out)[i] = make_uint4(shuffle(w.x), shuffle(w.y), shuffle(w.z), shuffle(w.w));
    } else {
      const long long s = i - n_code;
      const int wi = (int)(s & 127);
      const long long tile = s >> 7;                                   // (token tile, stage, chunk)
      const int c = (int)(tile % CH);
      const int step = (int)((tile / CH) % spt);
      const int tt = (int)(tile / ((long long)CH * spt));
      const int token = tt * 128 + (wi >> 2) + 32 * (wi & 3);
      const int kb0 = (step * CH + c) * 4;
      uint32_t v = 0;
      if (token < M) {
#pragma unroll
        for (int kb = 0; kb < 4; ++kb)
          if ((kb0 + kb) * 16 < K) v |= (uint32_t)(scales[(size_t)token * (K / 16) + kb0 + kb] & 0x7Fu) << (8 * kb);
      }
      sfb[s] = v;
    }
  }
}

struct Plan {
  Fp4ActLayout act;
  int grid;
  long long tiles, total_items;
  size_t counters_bytes, slots_bytes;
};

static Plan make_plan(const razer_desc* d, int M) {
  Plan p;
  const Geometry g = make_geometry(d->N, d->K);
  p.act = make_fp4_act_layout(M, d->K);
  p.tiles = (long long)g.row_tiles * p.act.token_tiles;
  p.total_items = p.tiles * p.act.spt;
  const int sms = sm_count();
  p.grid = (int)(p.total_items < sms ? p.total_items : sms);
  p.counters_bytes = align256((size_t)p.tiles * sizeof(uint32_t));
  p.slots_bytes = (size_t)(p.grid > 148 ? p.grid : 148) * 2 * p.act.NT * TILE_ROWS * sizeof(float);
  return p;
}

// FP4 magnitude code (0 .5 1 1.5 2 3 4 6 -> 0..7) of v, or -1.
static int fp4_code_of(float v) {
  const float mags[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};
  for (int i = 1; i < 8; ++i)
    if (mags[i] == v) return i;
  return -1;
}

// Base / remainder pair of each special-value magnitude (App. D.3): the largest base that serves both
// magnitudes when there is one (4 for {5, 8}: 4 + 1 and 4 + 4), otherwise each magnitude's own largest base.
static bool split_special_values(const float sv[2], uint32_t base[2], uint32_t rem[2]) {
  const float mags[7] = {6.0f, 4.0f, 3.0f, 2.0f, 1.5f, 1.0f, 0.5f};   // descending
  for (int bi = 0; bi < 7; ++bi) {                                     // a base that serves both magnitudes
    const int r0 = fp4_code_of(sv[0] - mags[bi]), r1 = fp4_code_of(sv[1] - mags[bi]);
    if (r0 > 0 && r1 > 0) {
      base[0] = base[1] = (uint32_t)fp4_code_of(mags[bi]);
      rem[0] = (uint32_t)r0;
      rem[1] = (uint32_t)r1;
      return true;
    }
  }
  for (int s = 0; s < 2; ++s) {                                        // each magnitude on its own
    bool found = false;
    for (int bi = 0; bi < 7 && !found; ++bi) {
      const int r = fp4_code_of(sv[s] - mags[bi]);
      if (r > 0) {
        base[s] = (uint32_t)fp4_code_of(mags[bi]);
        rem[s] = (uint32_t)r;
        found = true;
      }
    }
    if (!found) return false;
  }
  return true;
}

}  // namespace fp4_path

Fp4ActLayout make_fp4_act_layout(int M, int K) {
  Fp4ActLayout L;
  L.NT = M > 128 ? 256 : 128;
  if (const char* e = getenv("RAZER_FP4_NT")) {                        // tuning and test aid: force the token tile
    const int v = atoi(e);
    if (v == 128 || v == 256) L.NT = v;
  }
  L.token_tiles = (M + L.NT - 1) / L.NT;
  L.tiles128 = L.token_tiles * (L.NT / 128);
  const int k_chunks = (K + CHUNK_K - 1) / CHUNK_K;
  L.spt = (k_chunks + fp4_path::CH - 1) / fp4_path::CH;
  L.KP = L.spt * fp4_path::CH * CHUNK_K;
  L.codes_bytes = align256((size_t)M * L.KP / 2);
  L.sfb_bytes = (size_t)L.tiles128 * L.spt * fp4_path::SF_BYTES;
  return L;
}

// workspace of the matmul proper: status word, tile counters, partial-tile slots
size_t gemm_fp4_core_workspace_bytes(const razer_desc* d, int M) {
  const fp4_path::Plan p = fp4_path::make_plan(d, M);
  return WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
}

// ... plus the re-laid-out activation operand when the caller brings the interchange format
size_t gemm_fp4_workspace_bytes(const razer_desc* d, int M) {
  const fp4_path::Plan p = fp4_path::make_plan(d, M);
  return WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes + p.act.codes_bytes + p.act.sfb_bytes;
}

// The matmul on a prepared activation operand (act_fp4: codes, then scale-factor tiles).
int launch_gemm_fp4_prepared(const razer_desc* d, const void* packed, const void* act_fp4, const float* act_tensor_scale_dev,
                             int M, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  using namespace fp4_path;
  const Geometry g = make_geometry(d->N, d->K);
  const Plan p = make_plan(d, M);
  const size_t need = WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
  if (!ws || ws_bytes < need)
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  Args a;
  {
    uint32_t base[2], rem[2];
    if (!split_special_values(d->sv_mag, base, rem))
      return set_error(RAZER_ERR_UNSUPPORTED, "special values %g / %g are not sums of two FP4 values", d->sv_mag[0],
                       d->sv_mag[1]);
    a.base0 = base[0];
    a.rem0 = rem[0];
    a.base1 = base[1];
    a.rem1 = rem[1];
  }
  EncodeTiledFn enc = encode_fn();
  if (!enc) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  char* base_ws = (char*)ws;
  a.status = (uint32_t*)base_ws;
  a.counters = (uint32_t*)(base_ws + WS_STATUS_BYTES);
  a.slots = (float*)(base_ws + WS_STATUS_BYTES + p.counters_bytes);
  uint8_t* codes_pad = (uint8_t*)const_cast<void*>(act_fp4);
  a.sfb = codes_pad + p.act.codes_bytes;
  a.y = (__nv_bfloat16*)y;
  a.extra_scale = act_tensor_scale_dev;
  a.g = g;
  a.tensor_scale = d->tensor_scale;
  a.M = M;
  a.token_tiles = p.act.token_tiles;
  a.steps_per_tile = p.act.spt;
  a.total_items = p.total_items;

  const cuuint32_t estr[3] = {1, 1, 1};
  CUtensorMap tmap_x, tmap_w;
  {
    // padded activation codes as bytes: [M][KP / 2]; box = 128 bytes (one stage of k) x NT tokens
    const cuuint64_t dims[2] = {(cuuint64_t)(p.act.KP / 2), (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)(p.act.KP / 2)};
    const cuuint32_t box[2] = {128, (cuuint32_t)p.act.NT};
    const CUresult r = enc(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, codes_pad, dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled (activation codes) failed with code %d", (int)r);
  }
  {
    const cuuint64_t dims[3] = {(cuuint64_t)(PIECE_BYTES / 8), (cuuint64_t)g.k_chunks, (cuuint64_t)g.strips()};
    const cuuint64_t strides[2] = {(cuuint64_t)PIECE_BYTES, (cuuint64_t)g.strip_bytes()};
    const cuuint32_t box[3] = {(cuuint32_t)(PIECE_BYTES / 8), (cuuint32_t)CH, (cuuint32_t)TILE_STRIPS};
    const CUresult r = enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_INT64, 3, const_cast<void*>(packed), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled (weights) failed with code %d", (int)r);
  }
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(THREADS);
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  cudaError_t e;
  if (p.act.NT == 128) {
    static bool attr_set = false;
    if (!attr_set) {
      RAZER_TRY(check_cuda(cudaFuncSetAttribute(razer_fp4_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)Cfg<128>::SMEM_BYTES), "cudaFuncSetAttribute(max dynamic shared memory)"));
      attr_set = true;
    }
    cfg.dynamicSmemBytes = Cfg<128>::SMEM_BYTES;
    e = cudaLaunchKernelEx(&cfg, razer_fp4_kernel<128>, tmap_x, tmap_w, a);
  } else {
    static bool attr_set = false;
    if (!attr_set) {
      RAZER_TRY(check_cuda(cudaFuncSetAttribute(razer_fp4_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)Cfg<256>::SMEM_BYTES), "cudaFuncSetAttribute(max dynamic shared memory)"));
      attr_set = true;
    }
    cfg.dynamicSmemBytes = Cfg<256>::SMEM_BYTES;
    e = cudaLaunchKernelEx(&cfg, razer_fp4_kernel<256>, tmap_x, tmap_w, a);
  }
  count_launches(1);
  return check_cuda(e, "razer_fp4_kernel launch");
}

// Interchange-format activations: re-lay them out into the workspace (one small kernel), then the matmul.
int launch_gemm_fp4(const razer_desc* d, const void* packed, const uint8_t* act_codes, const uint8_t* act_scales,
                    const float* act_tensor_scale_dev, int M, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  using namespace fp4_path;
  const Plan p = make_plan(d, M);
  const size_t core = WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
  const size_t need = core + p.act.codes_bytes + p.act.sfb_bytes;
  if (!ws || ws_bytes < need)
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  uint8_t* codes_pad = (uint8_t*)ws + core;
  uint8_t* sfb = codes_pad + p.act.codes_bytes;
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  {
    const long long work = (long long)M * (p.act.KP / 32) + (long long)p.act.tiles128 * p.act.spt * CH * 128;
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, fp4_act_prep_kernel, (const uint32_t*)act_codes, act_scales, M, d->K,
                                             p.act.KP, p.act.tiles128, p.act.spt, (uint32_t*)codes_pad, (uint32_t*)sfb);
    count_launches(1);
    RAZER_TRY(check_cuda(e, "fp4_act_prep_kernel launch"));
  }
  return launch_gemm_fp4_prepared(d, packed, codes_pad, act_tensor_scale_dev, M, y, ws, core, st);
}

}  // namespace razer
