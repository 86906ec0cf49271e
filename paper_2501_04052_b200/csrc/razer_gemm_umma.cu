// Tensor-core matmul against packed RaZeR weights for sm_100a (tcgen05 + TMEM + TMA).
//
//   y[m, n] = bf16( ts * sum_k x[m, k] * D1[n, k] ),   D1 = block_scale * element (exact bf16)
//
// Mapping onto the 5th-generation tensor core: the weight tile is the MMA's A operand
// (128 weight rows = 128 TMEM lanes), the activation tile is the B operand (NT tokens,
// K-major in shared memory, 128-byte swizzle, written by TMA), the accumulator D[128 x NT]
// lives in TMEM.  Weights never exist as bf16 in shared or global memory: TMA bulk copies (one
// per 16-row strip of the tile) bring the packed 4.5-bit chunks into shared memory, the "dequant" warps (thread = weight
// row) decode one 16-element block at a time in registers and write the bf16 pairs straight
// into TMEM with tcgen05.st, and the MMA reads A from TMEM.
//
// Warp roles (64 + 32 * NDW threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA
// issuer, warps 2.. = dequant.  A warp reaches only the TMEM lanes 32 * (warp % 4) .. + 31, so
// warps w and w + 4 own the same 32 weight rows and split the stage's blocks between them;
// the first four dequant warps also run the epilogue of the tile they just fed.
//
// The register-level decode is described in razer_decode.cuh.
//
// Work partition (Sec. 4.3 / App. E of the paper: stripes of about equal length that may span
// several output tiles, partial results reduced through global memory): the grid is
// persistent, work items are (output tile, k-stage) pairs in tile-major order and every CTA
// takes one contiguous stripe of items.  A stripe's first and last tile may be partial; those
// go to a per-CTA FP32 slot in the workspace.  The CTA that holds a tile's first items (its
// stripe ends inside the tile) owns the tile: it waits until the other CTAs of the tile have
// counted themselves in (one counter per tile; for them the tile came first, so they are
// long done), adds the slots in CTA order, scales and rounds once.  Tiles a stripe covers
// completely are written directly.
//
// Every wait (mbarrier, counter) is bounded: on expiry the thread records a code in the
// workspace status word and the kernel drains and exits instead of hanging the GPU.
#include <cuda.h>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_decode.cuh"
#include "razer_ptx.cuh"
#include "razer_tcgen05.cuh"

namespace razer {

// Shared-memory matrix descriptor of a K-major bf16 tile stored with the 128-byte swizzle:
// rows are 128 bytes (64 elements), groups of 8 rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_b_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;                 // stride byte offset: 8 rows x 128 B
  d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                            // swizzle mode: 128 B
  return d;
}

// Instruction descriptor: bf16 x bf16 -> f32, both operands K-major, M = 128, N = NT.
__host__ __device__ constexpr uint32_t make_idesc(int nt) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nt >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// ------------------------------------------------------------------ kernel
struct UmmaArgs {
  const uint8_t* packed;
  __nv_bfloat16* y;
  float* slots;              // [grid][2][NT][128] FP32 partial tiles
  uint32_t* counters;        // one per output tile, zero between calls
  uint32_t* status;          // device status word
  const float* extra_scale;  // optional device scalar multiplied into the tensor scale
  Geometry g;
  float sv0, sv1, tensor_scale;
  uint32_t mul_lo, mul_hi;   // 2^6 + 2^12 and 2^2 + 2^8, passed at run time so that they stay multiplies
  int M, token_tiles, steps_per_tile;
  int x_map_3d;              // the activation tensor map is the 3-D (64 k, tokens, k chunk) view: one load per stage
  long long total_items;
};

constexpr int MAX_ISSUERS = 5;          // the MMA warp, or one issuing warp per dequant group

template <int NT, int CH, int STAGES, int ASTAGES, int NACC>
struct UmmaCfg {
  static constexpr int W_BYTES = CH * CHUNK_BYTES;
  static constexpr int X_BOX_BYTES = NT * 128;                 // NT tokens x 64 k x 2 B
  static constexpr int X_BYTES = CH * X_BOX_BYTES;
  static constexpr int W_PAD = (W_BYTES + 1023) / 1024 * 1024; // keep the x boxes 1024-byte aligned
  static constexpr int STAGE_BYTES = W_PAD + X_BYTES;
  static constexpr int ACC_COLS = NACC * NT < 32 ? 32 : NACC * NT;   // NACC accumulators, used round robin
  static constexpr int A_STAGE_COLS = CH * 32;                 // 4 blocks x 8 columns per chunk
  static constexpr int TMEM_COLS_NEEDED = ACC_COLS + ASTAGES * A_STAGE_COLS;
  static constexpr int TMEM_COLS = TMEM_COLS_NEEDED <= 64 ? 64 : TMEM_COLS_NEEDED <= 128 ? 128
                                   : TMEM_COLS_NEEDED <= 256 ? 256 : 512;
  static constexpr int NUM_BARS = 2 * STAGES + 2 * ASTAGES + 3 + MAX_ISSUERS;
  static constexpr int TABLE_BYTES = DECODE_TABLE_BYTES;        // scale table + special-value constants
  static constexpr size_t SMEM_BYTES =
      1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + NUM_BARS * 8 + 16 + 64 + TABLE_BYTES;
  static_assert(TMEM_COLS_NEEDED <= 512, "TMEM budget exceeded");
  static_assert(NT % 16 == 0 && NT >= 16 && NT <= 256, "UMMA N for M = 128");
};

// GI ("group issue"): each dequant group issues the MMAs of the items it decoded itself, into accumulators
// of its own, instead of handing them to the MMA warp.  Used for the narrowest token tile (16), where an
// item's MMAs are short; from 32 tokens up the MMA warp keeps up and issues (measured level at 16, the MMA
// warp ahead at 32 and 64).
template <int NT, int CH, int STAGES, int ASTAGES, int NDW, int NACC, bool GI>
__global__ void __launch_bounds__(64 + 32 * NDW, 1)
razer_umma_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const UmmaArgs a) {
  using Cfg = UmmaCfg<NT, CH, STAGES, ASTAGES, NACC>;
  constexpr int THREADS = 64 + 32 * NDW;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * Cfg::STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(        // 16-byte aligned: the tables behind it are read as uint4
      (reinterpret_cast<uintptr_t>(bars + Cfg::NUM_BARS) + 15) & ~(uintptr_t)15);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  uint8_t* tables = reinterpret_cast<uint8_t*>(tmem_slot + 16);   // decode tables (razer_decode.cuh)

  const uint32_t bar_full = smem_u32(bars);             // [STAGES]  TMA -> dequant, MMA
  const uint32_t bar_empty = bar_full + 8 * STAGES;     // [STAGES]  MMA commit -> TMA
  const uint32_t bar_afull = bar_empty + 8 * STAGES;    // [ASTAGES] dequant -> MMA
  const uint32_t bar_aempty = bar_afull + 8 * ASTAGES;  // [ASTAGES] MMA commit -> dequant
  const uint32_t bar_accfull = bar_aempty + 8 * ASTAGES;
  const uint32_t bar_accempty = bar_accfull + 8;
  const uint32_t bar_epi = bar_accempty + 8;            // rendezvous of the 128 epilogue threads
  const uint32_t bar_drain = bar_epi + 8;               // [MAX_ISSUERS] an issuing warp's own MMAs have all completed

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grid = gridDim.x, cta = blockIdx.x;
  const int it_begin = (int)((a.total_items * cta) / grid);
  const int it_end = (int)((a.total_items * (cta + 1)) / grid);
  const int n_items = it_end - it_begin;
  const int spt = a.steps_per_tile;
  ItemCursor cur;
  cur.tile = it_begin / spt;
  cur.step = it_begin - cur.tile * spt;
  cur.stage = cur.phase = cur.astage = cur.aphase = 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    for (int i = 0; i < ASTAGES; ++i) {
      mbar_init(bar_afull + 8 * i, 128);
      mbar_init(bar_aempty + 8 * i, 1);
    }
    mbar_init(bar_accfull, GI ? NDW / 4 : 1);
    mbar_init(bar_accempty, GI ? 128 : 32 * NDW);         // threads that read the accumulator in the epilogue
    mbar_init(bar_epi, GI ? 128 : 32 * NDW);
    for (int i = 0; i < MAX_ISSUERS; ++i) mbar_init(bar_drain + 8 * i, 1);
    *abort_flag = 0;
    tmem_slot[3] = 0;                                   // a flag nobody sets (used by the drain waits)
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Producer state (thread 0 only).  The first ring of loads goes out before the rest of the prologue
  // (tables, TMEM allocation) so that the first HBM round trip overlaps it.
  int issued = 0;
  int p_rt = cur.tile / a.token_tiles, p_tt = cur.tile - p_rt * a.token_tiles;
  auto produce_x = [&](int stage, int step, int tt) {       // activation box(es) of one stage
    const int c0 = step * CH;
    const int nch = min(CH, a.g.k_chunks - c0);
    const uint32_t st = smem_u32(smem) + (uint32_t)stage * Cfg::STAGE_BYTES;
    const uint32_t bar = bar_full + 8 * stage;
    if (a.x_map_3d) {
      tma_load_3d(st + Cfg::W_PAD, &tmap_x, 0, tt * NT, c0, bar);
    } else {
      for (int c = 0; c < nch; ++c)
        tma_load_2d(st + Cfg::W_PAD + c * Cfg::X_BOX_BYTES, &tmap_x, (c0 + c) * CHUNK_K, tt * NT, bar);
    }
  };
  auto produce = [&](bool with_x) {
    const int c0 = cur.step * CH;
    const int nch = min(CH, a.g.k_chunks - c0);
    const uint32_t st = smem_u32(smem) + (uint32_t)cur.stage * Cfg::STAGE_BYTES;
    const uint32_t bar = bar_full + 8 * cur.stage;
    const uint32_t n_x = a.x_map_3d ? CH : nch;           // the 3-D box always spans CH chunks (zero-filled past K)
    // The packed buffer as a (piece bytes, k chunk, strip) tensor: one box brings chunks c0 .. c0 + CH - 1 of the
    // row tile's eight strips, [strip][chunk][piece] in shared memory (chunks past the end of K arrive as zeros).
    mbar_expect_tx(bar, (uint32_t)(CH * CHUNK_BYTES) + n_x * Cfg::X_BOX_BYTES);
    tma_load_3d(st, &tmap_w, 0, c0, p_rt * TILE_STRIPS, bar);
    if (with_x) produce_x(cur.stage, cur.step, p_tt);
    if (cur.step == spt - 1 && ++p_tt == a.token_tiles) { p_tt = 0; ++p_rt; }
    cur.template next<STAGES, ASTAGES>(spt);
  };
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_w) : "memory");
    grid_dep_launch();                                    // the next kernel may start its own prologue
    // first ring: packed weights now, their activation boxes once the preceding kernel has finished
    const ItemCursor first = cur;
    const int first_tt = p_tt;
    for (; issued < n_items && issued < STAGES; ++issued) produce(false);
    grid_dep_wait();
    ItemCursor c2 = first;
    int tt2 = first_tt;
    for (int i = 0; i < issued; ++i) {
      produce_x(c2.stage, c2.step, tt2);
      if (c2.step == spt - 1 && ++tt2 == a.token_tiles) tt2 = 0;
      c2.template next<STAGES, ASTAGES>(spt);
    }
  }
  if (warp != 0) decode_tables_fill(tables, a.sv0, a.sv1, threadIdx.x - 32, THREADS - 32);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_a0 = tmem_base + Cfg::ACC_COLS;

  auto fail = [&](uint32_t code) {
    *abort_flag = 1;
    grid_dep_wait();                                      // the status word lives in the (possibly shared) workspace
    atomicCAS(a.status, 0u, code);
  };

  // Whole warp, on leaving an issue loop (at its end or after a wait gave up): the MMAs this warp has issued
  // read shared memory and TMEM and write TMEM until they complete, so the warp commits them to a barrier of
  // its own and waits for it (bounded, not watching the abort flag) before the CTA may release either.
  auto drain_mmas = [&](int issuer_idx) {
    __syncwarp();
    const uint32_t bar = bar_drain + 8 * issuer_idx;
    if (elect_one()) tc_commit(bar);
    __syncwarp();
    mbar_wait(bar, 0u, tmem_slot + 3);
  };

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      for (; issued < n_items; ++issued) {
        if (!mbar_wait(bar_empty + 8 * cur.stage, (uint32_t)cur.phase ^ 1u, abort_flag)) { fail(1); break; }
        produce(true);
      }
      // Drain: copies still in flight must land before this CTA's shared memory is released.
      const int pending = issued < STAGES ? issued : STAGES;
      for (int f = issued - pending; f < issued; ++f)
        mbar_wait(bar_full + 8 * (f % STAGES), (uint32_t)((f / STAGES) & 1), tmem_slot + 3);
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (whole warp walks the items, one elected lane issues) =====================
    if (!GI) {
      constexpr uint32_t idesc = make_idesc(NT);
      // upper half of the shared-memory descriptor: 1024-byte group stride, descriptor version, 128-byte swizzle
      constexpr uint32_t bd_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
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
        // the group that filled this A stage waited for the shared-memory stage (weights and activations)
        // before it decoded, so its arrival also covers the activation tile
        if (!wait_warp(bar_afull + 8 * cur.astage, (uint32_t)cur.aphase, 3)) break;
        if (seg_first && !wait_warp(bar_accempty, (seg & 1u) ^ 1u, 4)) break;
        tc_fence_after();
        const uint32_t xs = smem_u32(smem) + (uint32_t)cur.stage * Cfg::STAGE_BYTES + Cfg::W_PAD;
        const uint32_t a_t = tmem_a0 + cur.astage * Cfg::A_STAGE_COLS;
        const uint32_t bd_lo = (xs >> 4) | (1u << 16);    // start address and (unused) leading offset fields
        if (elect_one()) {
          // Consecutive MMAs go to NACC different accumulators (summed in the epilogue): MMAs on one
          // accumulator execute one after the other, and a narrow MMA is far shorter than its latency.
#pragma unroll
          for (int j = 0; j < CH * 4; ++j) {
            // 16 k further along: +32 bytes inside a chunk's 128-byte rows, next chunk's box after four
            if (j < nch * 4) {
              const uint32_t bd = bd_lo + (uint32_t)(((j >> 2) * Cfg::X_BOX_BYTES + (j & 3) * 32) >> 4);
              const uint32_t d_t = tmem_base + (j % NACC) * NT;
              if (j < NACC && seg_first) tc_mma_ts2<false>(d_t, a_t + j * 8, bd, bd_hi, idesc);
              else tc_mma_ts2<true>(d_t, a_t + j * 8, bd, bd_hi, idesc);
            }
          }
          tc_commit(bar_empty + 8 * cur.stage);
          tc_commit(bar_aempty + 8 * cur.astage);
          if (seg_last) tc_commit(bar_accfull);
        }
        __syncwarp();
        if (seg_last) ++seg;
        cur.template next<STAGES, ASTAGES>(spt);
      }
      drain_mmas(0);
    }
  } else {
    // ===================== dequant (32 * NDW threads, thread = weight row) + epilogue =====================
    const int row = 32 * (warp & 3) + lane;              // TMEM lane this thread owns
    const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
    const int group = (warp - 2) >> 2;                   // four warps (all TMEM lane quarters) decode one item together
    constexpr int GROUPS = NDW / 4;
    static_assert(NDW % 4 == 0 && GROUPS <= ASTAGES, "every dequant group needs an A stage of its own");
    static_assert(GROUPS + 1 <= MAX_ISSUERS, "a drain barrier per issuing warp");
    static_assert(!GI || (NACC % GROUPS == 0 && ASTAGES == GROUPS), "group issue: A stage and accumulators per group");
    static_assert(GI ? STAGES % GROUPS == 0 : (GROUPS == ASTAGES && STAGES >= ASTAGES),
                  "every fill of a stage must be known complete to the group that waits for the next one");
    constexpr int APG = GI ? NACC / GROUPS : NACC;       // accumulators per group
    // one warp of each group issues the group's MMAs; the groups pick different ones so that the issuing
    // warps sit on different schedulers (a warp's scheduler is warp % 4)
    const bool issuer = GI && ((warp - 2) & 3) == (group & 3);
    uint32_t own_phase = 0, gseg = 0;                    // GI: parity of the group's A stage; segments seen
    bool fresh = true;                                   // GI: the group's accumulators hold nothing of this segment yet
    // Epilogue: with group issue only group 0 drains the (narrow) accumulators while the other groups
    // keep decoding; otherwise every group drains its share of the columns of its TMEM lane quarter.
    const bool epi_warp = !GI || (group == 0);
    // shares in units of 16 columns: group g takes units [g U / GROUPS, (g + 1) U / GROUPS), U = NT / 16
    const int col_lo = GI ? 0 : 16 * ((group * (NT / 16)) / GROUPS);
    const int col_hi = GI ? NT : 16 * (((group + 1) * (NT / 16)) / GROUPS);
    const bool leader = (threadIdx.x == 64);
    float ts = a.tensor_scale;                           // (x extra scale: read after the grid dependency)
    bool dep_waited = false;
    uint32_t seg = 0, epi_phase = 0;
    // all 32 lanes take the same branch after a wait, so the .aligned tcgen05 instructions stay convergent
    auto wait_all = [&](uint32_t bar, uint32_t parity, uint32_t code) -> bool {
      const bool got = mbar_wait(bar, parity, abort_flag);
      if (!got) fail(code);
      return __all_sync(0xFFFFFFFFu, got);
    };
    auto epi_sync = [&]() -> bool {                     // bounded rendezvous of the epilogue threads
      mbar_arrive(bar_epi);
      const bool got = wait_all(bar_epi, epi_phase & 1u, 8);
      ++epi_phase;
      return got;
    };
    const DecodeTables dt = decode_tables_view(tables, lane);
    const uint32_t mul_lo = a.mul_lo, mul_hi = a.mul_hi;
    // where this thread's weight row sits inside a stage: strip row / 16, row r = row % 16 of it
    const int r16 = row % STRIP_ROWS;
    const uint32_t strip_off = (uint32_t)(row / STRIP_ROWS) * (CH * PIECE_BYTES);
    const uint32_t scale_off = (uint32_t)PIECE_CODE_BYTES + (uint32_t)(r16 & 7) * 8;
    const uint32_t scale_sel = (r16 >> 3) ? 0x7531u : 0x6420u;
    uint32_t code_off[CHUNK_BLOCKS];
#pragma unroll
    for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) code_off[blk] = (uint32_t)piece_code_offset(blk, r16);
    int turn = 0;                                        // item i is decoded by group i % GROUPS
    for (int i = 0; i < n_items; ++i, cur.template next<STAGES, ASTAGES>(spt), turn = (turn + 1 == GROUPS ? 0 : turn + 1)) {
      const int tile = cur.tile, step = cur.step;
      const bool seg_last = (i + 1 == n_items) || step == spt - 1;
      const int nch = min(CH, a.g.k_chunks - step * CH);
      const bool seg_first = (i == 0) || step == 0;
      if (GI && seg_first) {
        fresh = true;
        // the epilogue of the previous segment must have read the accumulators before any group moves on
        if (issuer && gseg > 0 && !wait_all(bar_accempty, (gseg & 1u) ^ 1u, 4)) break;
      }
      if (turn == group) {
      const int astage = GI ? group : cur.astage;
      const uint32_t aph = GI ? own_phase : (uint32_t)cur.aphase;
      // Order matters.  A parity wait is only sound for a waiter that knows the barrier's previous phase to be
      // complete, and a group does not see every fill of a shared-memory stage (the loads of a ring complete in
      // any order: a group could come back to a stage one ring later while the fill it skipped is still in
      // flight, take that for its own and decode the stage's old bytes).  Group issue: STAGES is a multiple of
      // GROUPS, so a stage always serves the same group, which sees all its fills (making every group wait for
      // the fills it skips is no way out: the groups free the stages themselves and end up waiting for one
      // another).  Otherwise the A stage is
      // this group's own (GROUPS == ASTAGES) and its release by the MMA warp, which takes the items in order,
      // means that every item up to i - ASTAGES was issued, hence decoded, hence landed, the stage's previous
      // fill (item i - STAGES, STAGES >= ASTAGES) among them.
      if (!wait_all(bar_aempty + 8 * astage, aph ^ 1u, 6)) break;
      if (!wait_all(bar_full + 8 * cur.stage, (uint32_t)cur.phase, 5)) break;
      tc_fence_after();
      // this thread's strip of the stage: [strip 0..7][chunk 0..CH-1] pieces
      const uint32_t st = smem_addr(smem) + (uint32_t)cur.stage * Cfg::STAGE_BYTES + strip_off;
      const uint32_t a_t = tmem_a0 + astage * Cfg::A_STAGE_COLS + lane_off;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        if (c < nch) {
          const uint32_t ck = st + c * PIECE_BYTES;
          // all of the chunk's loads first, then the arithmetic
          const uint2 sq = lds64(ck + scale_off);           // the eight scale bytes of rows r % 8 and r % 8 + 8
          const uint32_t sw = __byte_perm(sq.x, sq.y, scale_sel);   // this row's four, in block order
          uint2 cw[CHUNK_BLOCKS];
#pragma unroll
          for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) cw[blk] = lds64(ck + code_off[blk]);
          uint32_t ss2[CHUNK_BLOCKS];
          SvConsts svc[CHUNK_BLOCKS];
#pragma unroll
          for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) decode_block_consts(dt, sw, blk, ss2[blk], svc[blk]);
#pragma unroll
          for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) {
            uint32_t v[8];
            decode_word(cw[blk].x, ss2[blk], svc[blk], mul_lo, mul_hi, v);
            decode_word(cw[blk].y, ss2[blk], svc[blk], mul_lo, mul_hi, v + 4);
            tc_st8(a_t + (c * 4 + blk) * 8, v);
          }
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_afull + 8 * astage);
      if (GI) {
        if (issuer) {
          // the group's 128 threads have stored their rows: issue this item's MMAs from here
          if (!wait_all(bar_afull + 8 * astage, aph, 3)) break;
          tc_fence_after();
          constexpr uint32_t idesc = make_idesc(NT);
          constexpr uint32_t bd_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
          const uint32_t xs = smem_u32(smem) + (uint32_t)cur.stage * Cfg::STAGE_BYTES + Cfg::W_PAD;
          const uint32_t bd_lo = (xs >> 4) | (1u << 16);
          const uint32_t a_s = tmem_a0 + astage * Cfg::A_STAGE_COLS;
          if (elect_one()) {
#pragma unroll
            for (int j = 0; j < CH * 4; ++j) {
              if (j < nch * 4) {
                const uint32_t bd = bd_lo + (uint32_t)(((j >> 2) * Cfg::X_BOX_BYTES + (j & 3) * 32) >> 4);
                const uint32_t d_t = tmem_base + (group * APG + j % APG) * NT;
                if (j < APG && fresh) tc_mma_ts2<false>(d_t, a_s + j * 8, bd, bd_hi, idesc);
                else tc_mma_ts2<true>(d_t, a_s + j * 8, bd, bd_hi, idesc);
              }
            }
            tc_commit(bar_empty + 8 * cur.stage);
            tc_commit(bar_aempty + 8 * astage);
          }
          __syncwarp();
        }
        fresh = false;
        own_phase ^= 1u;
      }
      }
      if (GI && seg_last) {
        // every group reports its share of the segment (a group without an item in it reports at once)
        if (issuer) {
          if (elect_one()) tc_commit(bar_accfull);
          __syncwarp();
        }
        ++gseg;
      }

      if (!seg_last || !epi_warp) continue;
      // ---------------- epilogue of the segment that ends with this item ----------------
      const int it = it_begin + i;
      const int tile_begin = tile * spt;
      const int seg_begin = it_begin > tile_begin ? it_begin : tile_begin;
      const bool complete = (seg_begin == tile_begin) && (step == spt - 1);
      const int rt = tile / a.token_tiles, tt = tile - rt * a.token_tiles;
      const int n_out = rt * TILE_ROWS + row;
      const int m0 = tt * NT;
      if (!dep_waited) {                                   // outputs, workspace and the scale scalar may belong to the preceding kernel
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
        if (!ready) fail(9);
        if (!__all_sync(0xFFFFFFFFu, ready)) break;
      }
      if (!wait_all(bar_accfull, seg & 1u, 7)) break;
      tc_fence_after();
      float* my_slot = a.slots + (size_t)cta * 2 * (size_t)(NT * TILE_ROWS);   // a non-owner's part is its stripe's first segment
      bool acc_valid[GROUPS];                                         // GI: which groups had an item in this segment
      {
        const int i0 = seg_begin - it_begin, len = i - i0 + 1;
#pragma unroll
        for (int q = 0; q < GROUPS; ++q) acc_valid[q] = (len >= GROUPS) || (((q - i0 % GROUPS + GROUPS) % GROUPS) < len);
      }
#pragma unroll 1
      for (int c0 = col_lo; c0 < col_hi; c0 += 16) {
        uint32_t v[16];
        tc_ld16(tmem_base + lane_off + c0, v);
        tc_wait_ld();
        if (GI && !acc_valid[0]) {                                    // group 0 had no item in this segment
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0;
        }
#pragma unroll
        for (int q = 1; q < NACC; ++q) {
          uint32_t w[16];
          tc_ld16(tmem_base + lane_off + q * NT + c0, w);
          tc_wait_ld();
          if (!GI || acc_valid[q / APG]) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
          }
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
      (void)it;
    }
    if (GI && issuer) drain_mmas(1 + group);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();                                       // lane 0 ran the issue loop alone; dealloc is warp-wide
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
  }
}

// ------------------------------------------------------------------ host side
struct UmmaPlan {
  int NT, CH;
  int token_tiles, steps_per_tile, grid;
  long long tiles, total_items;
  size_t counters_bytes, slots_bytes;
};

static UmmaPlan make_plan(const razer_desc* d, int M) {
  UmmaPlan p;
  const Geometry g = make_geometry(d->N, d->K);
  p.NT = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : 256;
  p.CH = p.NT <= 64 ? 4 : p.NT == 128 ? 2 : 1;
  p.token_tiles = (M + p.NT - 1) / p.NT;
  p.steps_per_tile = (g.k_chunks + p.CH - 1) / p.CH;
  p.tiles = (long long)g.row_tiles * p.token_tiles;
  p.total_items = p.tiles * p.steps_per_tile;
  const int sms = sm_count();
  p.grid = (int)(p.total_items < sms ? p.total_items : sms);
  p.counters_bytes = align256((size_t)p.tiles * sizeof(uint32_t));
  p.slots_bytes = (size_t)p.grid * 2 * p.NT * TILE_ROWS * sizeof(float);
  return p;
}

bool umma_supported(const razer_desc* d, int M) {
  (void)d;
  (void)M;
  // RAZER_KERNEL=simt routes every matmul to the CUDA-core kernel (debugging aid)
  const char* e = getenv("RAZER_KERNEL");
  return !(e && e[0] == 's' && e[1] == 'i');
}

size_t umma_workspace_bytes(const razer_desc* d, int M) {
  // sized for the largest grid (all SMs); the status word comes first
  UmmaPlan p = make_plan(d, M);
  const size_t slots = (size_t)(p.grid > 148 ? p.grid : 148) * 2 * p.NT * TILE_ROWS * sizeof(float);
  return WS_STATUS_BYTES + p.counters_bytes + slots;
}

// Leading part of the workspace that has to be zero before a launch (status word + counters).
size_t umma_workspace_zero_bytes(const razer_desc* d, int M) {
  return WS_STATUS_BYTES + make_plan(d, M).counters_bytes;
}

template <int NT, int CH, int STAGES, int ASTAGES, int NDW, int NACC, bool GI>
static int launch_cfg(const CUtensorMap& tmap, const CUtensorMap& tmap_w, const UmmaArgs& args, int grid, cudaStream_t st) {
  using Cfg = UmmaCfg<NT, CH, STAGES, ASTAGES, NACC>;
  auto kern = razer_umma_kernel<NT, CH, STAGES, ASTAGES, NDW, NACC, GI>;
  static bool attr_set = false;
  if (!attr_set) {
    RAZER_TRY(check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM_BYTES),
                         "cudaFuncSetAttribute(max dynamic shared memory)"));
    attr_set = true;
  }
  // Programmatic dependent launch (RAZER_PDL=0 turns it off): the kernel may begin while the preceding
  // kernel of the stream drains; it touches nothing that kernel may own before its grid_dep_wait().
  static const bool pdl = [] { const char* e = getenv("RAZER_PDL"); return !(e && e[0] == '0'); }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(64 + 32 * NDW);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmap, tmap_w, args);
  count_launches(1);
  return check_cuda(e, "razer_umma_kernel launch");
}

int launch_gemm_umma(const razer_desc* d, const void* packed, const void* x, int M, int ldx_K, float extra_scale,
                     const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  const Geometry g = make_geometry(d->N, d->K);
  const UmmaPlan p = make_plan(d, M);
  const size_t need = WS_STATUS_BYTES + p.counters_bytes + p.slots_bytes;
  if (!ws || ws_bytes < need)
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  EncodeTiledFn enc = encode_fn();
  if (!enc) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  CUtensorMap tmap;
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = CUDA_ERROR_UNKNOWN;
  int map_3d = 0;
  if (d->K % CHUNK_K == 0 && ldx_K == d->K) {
    // (64 k, tokens, k chunk) view of x: one box brings the activations of all CH chunks of a stage
    const cuuint64_t dims[3] = {(cuuint64_t)CHUNK_K, (cuuint64_t)M, (cuuint64_t)(d->K / CHUNK_K)};
    const cuuint64_t strides[2] = {(cuuint64_t)ldx_K * 2, (cuuint64_t)CHUNK_K * 2};
    const cuuint32_t box[3] = {(cuuint32_t)CHUNK_K, (cuuint32_t)p.NT, (cuuint32_t)p.CH};
    r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    map_3d = (r == CUDA_SUCCESS);
  }
  if (!map_3d) {
    const cuuint64_t dims[2] = {(cuuint64_t)d->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx_K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)CHUNK_K, (cuuint32_t)p.NT};
    r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  // packed weights: (72 x 8 bytes of a piece, k chunk, strip), box = (whole piece, CH chunks, the tile's 8 strips)
  CUtensorMap tmap_w;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)(PIECE_BYTES / 8), (cuuint64_t)g.k_chunks, (cuuint64_t)g.strips()};
    const cuuint64_t strides[2] = {(cuuint64_t)PIECE_BYTES, (cuuint64_t)g.strip_bytes()};
    const cuuint32_t box[3] = {(cuuint32_t)(PIECE_BYTES / 8), (cuuint32_t)p.CH, (cuuint32_t)TILE_STRIPS};
    r = enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_INT64, 3, const_cast<void*>(packed), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(RAZER_ERR_CUDA, "cuTensorMapEncodeTiled (weights) failed with code %d", (int)r);
  }

  UmmaArgs a;
  a.packed = (const uint8_t*)packed;
  a.y = (__nv_bfloat16*)y;
  a.status = (uint32_t*)ws;
  a.counters = (uint32_t*)((char*)ws + WS_STATUS_BYTES);
  a.slots = (float*)((char*)ws + WS_STATUS_BYTES + p.counters_bytes);
  a.extra_scale = extra_scale_dev;
  a.g = g;
  a.sv0 = d->sv_mag[0];
  a.sv1 = d->sv_mag[1];
  a.mul_lo = (1u << 6) + (1u << 12);
  a.mul_hi = (1u << 2) + (1u << 8);
  a.tensor_scale = d->tensor_scale * extra_scale;
  a.M = M;
  a.token_tiles = p.token_tiles;
  a.steps_per_tile = p.steps_per_tile;
  a.total_items = p.total_items;
  a.x_map_3d = map_3d;
  switch (p.NT) {
    case 16:
      return launch_cfg<16, 4, 6, 3, 12, 6, true>(tmap, tmap_w, a, p.grid, st);
    case 32: return launch_cfg<32, 4, 6, 3, 12, 2, false>(tmap, tmap_w, a, p.grid, st);
    case 64: return launch_cfg<64, 4, 4, 3, 12, 2, false>(tmap, tmap_w, a, p.grid, st);
    case 128: return launch_cfg<128, 2, 4, 4, 16, 1, false>(tmap, tmap_w, a, p.grid, st);
    default: return launch_cfg<256, 1, 5, 4, 16, 1, false>(tmap, tmap_w, a, p.grid, st);
  }
}

}  // namespace razer
