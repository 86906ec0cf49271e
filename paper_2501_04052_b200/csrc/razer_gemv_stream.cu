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
#include "razer_stream_common.cuh"

namespace razer {

namespace stream_path {

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
    epilogue_loop<C::ROWS>(a, work, b, lane, red, bar_red_full, bar_red_free, abort_flag, ts, fail);
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
