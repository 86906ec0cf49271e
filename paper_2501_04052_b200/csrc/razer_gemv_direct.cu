// Decode GEMV (M <= 8) against packed RaZeR weights for sm_100a: register-only weight path, no split-K
// through global memory.
//
//   y[m, n] = bf16( ts * sum_k x[m, k] * D1[n, k] ),   D1 = block_scale * element (exact bf16)
//
// Every weight byte is used exactly once, so this kernel does not stage weights anywhere: each
// lane loads the 8-byte code words of "its" blocks straight from global memory into registers
// (streaming loads, several chunks ahead), decodes them there (razer_decode.cuh) and feeds them
// as the A fragment of a warp-level m16n8k16 tensor-core MMA whose B fragment is the activation
// slice (tokens along n), accumulated in FP32 registers.  Sec. 4.3 of the paper describes this style
// for its weight-only kernel (weights pre-shuffled so that each thread's loads match its MMA fragment).
//
// Work unit: R = 16 * MT weight rows over the whole of K.  A CTA (16 warps) takes a contiguous range of
// units; inside a unit warp w takes the chunks (64 columns) w, w + 16, ...  In a chunk, lane
// (g = lane / 4, t = lane % 4) decodes block t of rows g and g + 8 of each 16-row MMA tile; MMA q (0..3)
// takes elements 4q .. 4q + 3 of every lane's block, i.e. the MMA's k slots are columns
// 16 t + 4 q + {0, 1, 2, 3}, for A and B alike.  At the end of a unit the 16 warps leave their partial sums
// in shared memory, and R * 8 threads add them in warp order, scale, round and store.  Nothing is exchanged
// between CTAs, so there is no workspace, no counter and no wait on another CTA; the price is that the
// rows have to divide evenly enough over the SMs, which the host checks before it picks this kernel.
#include <cuda.h>
#include <cstdlib>

#include "razer_common.cuh"
#include "razer_decode.cuh"

namespace razer {

namespace direct_path {

constexpr int WARPS = 16;
constexpr int THREADS = 32 * WARPS;
constexpr int TOKENS = 8;
constexpr int DEPTH_MT1 = 5;    // chunks in flight per warp (register sets)
constexpr int DEPTH_MT2 = 3;

template <int MT>
struct Cfg {
  static constexpr int R = 16 * MT;                               // rows of a unit
  static constexpr int RED_FLOATS = R * TOKENS;                   // one warp's partial sums
  static constexpr int RED_BYTES = 2 * WARPS * RED_FLOATS * 4;    // two buffers
  static constexpr size_t SMEM_BYTES = RED_BYTES + DECODE_TABLE_BYTES;
};

__device__ __forceinline__ uint2 ldg_stream64(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ldg_stream32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ldg128(const void* p) {   // activations: cached, re-read for every unit
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
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
  int M, units;              // units of R rows
};

// One chunk's registers of a lane: code words and scale words of rows (g, g + 8) of each MMA tile,
// and the lane's 16 activation columns (token g).
template <int MT>
struct ChunkRegs {
  uint2 cw[MT][2];
  uint32_t sw[MT][2];
  uint4 xa, xb;
};

template <int MT, int DEPTH>
__global__ void __launch_bounds__(THREADS, 1) razer_direct_kernel(const Args a) {
  using C = Cfg<MT>;
  extern __shared__ __align__(16) uint8_t smem[];
  float* red = reinterpret_cast<float*>(smem);
  uint8_t* tables = smem + C::RED_BYTES;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int kc = a.g.k_chunks;                               // >= WARPS (host check): every warp has chunks
  const int u_begin = (int)(((long long)a.units * blockIdx.x) / gridDim.x);
  const int u_end = (int)(((long long)a.units * (blockIdx.x + 1)) / gridDim.x);

  grid_dep_launch();
  decode_tables_fill(tables, a.sv0, a.sv1, threadIdx.x, THREADS);

  // this lane's byte offsets inside a chunk, relative to the unit's first row
  int code_off[MT][2], scale_off[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int r = 16 * mt + 8 * h + g;                     // units start on multiples of 16 rows: the slot swizzle stays inside
      code_off[mt][h] = packed_code_offset(t, r);
      scale_off[mt][h] = CHUNK_CODE_BYTES + r * 4;
    }
  const bool has_token = g < a.M;
  const __nv_bfloat16* x_lane = a.x + (size_t)(has_token ? g : 0) * a.g.K + 16 * t;

  auto load_w = [&](ChunkRegs<MT>& r, int u, int c) {       // weights: no dependency on earlier kernels
    const int n0 = u * C::R, tile = n0 / TILE_ROWS, r0 = n0 % TILE_ROWS;
    const uint8_t* ck = a.packed + ((size_t)tile * kc + c) * CHUNK_BYTES;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        r.cw[mt][h] = ldg_stream64(ck + r0 * 8 + code_off[mt][h]);
        r.sw[mt][h] = ldg_stream32(ck + r0 * 4 + scale_off[mt][h]);
      }
  };
  auto load_x = [&](ChunkRegs<MT>& r, int c) {
    if (has_token && c * CHUNK_K + 16 * t < a.g.K) {         // K is a multiple of 16: a 16-column group is whole
      r.xa = ldg128(x_lane + (size_t)c * CHUNK_K);
      r.xb = ldg128(x_lane + (size_t)c * CHUNK_K + 8);
    } else {
      r.xa = make_uint4(0, 0, 0, 0);
      r.xb = make_uint4(0, 0, 0, 0);
    }
  };
  auto advance = [&](int& u, int& c) {
    c += WARPS;
    if (c >= kc) {
      c = warp;
      ++u;
    }
  };

  // ---------------- prologue: the first DEPTH chunks' weights, then (after the dependency) their activations ----------------
  ChunkRegs<MT> regs[DEPTH];
  int pu = u_begin, pc = warp;                               // prefetch cursor
  {
    int u = pu, c = pc;
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) {
      if (u < u_end) load_w(regs[d], u, c);
      advance(u, c);
    }
  }
  __syncthreads();                                           // tables are ready
  const DecodeTables dt = decode_tables_view(tables, lane);
  const uint32_t mul_lo = a.mul_lo, mul_hi = a.mul_hi;
  grid_dep_wait();                                           // activations and outputs may belong to the preceding kernel
  float ts = a.tensor_scale;
  if (a.extra_scale) ts *= *a.extra_scale;
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    if (pu < u_end) load_x(regs[d], pc);
    advance(pu, pc);
  }

  float acc[MT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[mt][j] = 0.0f;

  auto compute = [&](const ChunkRegs<MT>& r) {
    const uint32_t xq[4][2] = {{r.xa.x, r.xa.y}, {r.xa.z, r.xa.w}, {r.xb.x, r.xb.y}, {r.xb.z, r.xb.w}};
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint32_t e[2][8];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t ss2;
        SvConsts svc;
        decode_block_consts_byte(dt, r.sw[mt][h] >> (8 * t), ss2, svc);
        decode_word(r.cw[mt][h].x, ss2, svc, mul_lo, mul_hi, e[h]);
        decode_word(r.cw[mt][h].y, ss2, svc, mul_lo, mul_hi, e[h] + 4);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        mma_16816(acc[mt], e[0][2 * q], e[1][2 * q], e[0][2 * q + 1], e[1][2 * q + 1], xq[q][0], xq[q][1]);
    }
  };

  // End of a unit: leave this warp's partial sums, meet, and let R * 8 threads finish the rows.
  // Element (row, token) of the unit sits at row * 8 + token, so a warp's 32 stores hit 32 banks.
  int buf = 0;
  auto unit_end = [&](int u) {
    float* mine = red + (buf * WARPS + warp) * C::RED_FLOATS;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mine[(16 * mt + 8 * (j >> 1) + g) * TOKENS + 2 * t + (j & 1)] = acc[mt][j];
        acc[mt][j] = 0.0f;
      }
    __syncthreads();                                         // the buffer written two units ago was read before the previous meeting
    if ((int)threadIdx.x < C::RED_FLOATS) {
      const float* src = red + buf * WARPS * C::RED_FLOATS + threadIdx.x;
      float s = 0.0f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) s += src[w * C::RED_FLOATS];   // warp order: a fixed summation order
      const int n = u * C::R + ((int)threadIdx.x >> 3), m = (int)threadIdx.x & 7;
      if (m < a.M && n < a.g.N) a.y[(size_t)m * a.g.N + n] = __float2bfloat16_rn(ts * s);
    }
    buf ^= 1;
  };

  // ---------------- main loop: consume the oldest register set, refill it DEPTH chunks ahead ----------------
  int cu = u_begin, cc = warp;                               // compute cursor
  while (cu < u_end) {
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) {
      if (cu < u_end) {
        compute(regs[d]);
        if (pu < u_end) {
          load_w(regs[d], pu, pc);
          load_x(regs[d], pc);
        }
        advance(pu, pc);
        const int u_done = cu;
        advance(cu, cc);
        if (cu != u_done) unit_end(u_done);
      }
    }
  }
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
  int mt, units, grid;
  double balance;            // useful share of the SMs' time: rows are not split over K
};

static DirectPlan direct_plan(const razer_desc* d) {
  const Geometry g = make_geometry(d->N, d->K);
  const int sms = direct_sm_count();
  DirectPlan best = {};
  for (int mt = 2; mt >= 1; --mt) {
    DirectPlan p;
    p.mt = mt;
    p.units = (g.row_tiles * TILE_ROWS) / (16 * mt);
    p.grid = p.units < sms ? p.units : sms;
    const int per_cta = (p.units + p.grid - 1) / p.grid;
    p.balance = (double)p.units / ((double)per_cta * sms);
    if (mt == 2 || p.balance > best.balance + 0.20) best = p;   // wider units amortise the activation loads
  }
  return best;
}

bool gemv_direct_supported(const razer_desc* d, int M) {
  const Geometry g = make_geometry(d->N, d->K);
  return M >= 1 && M <= direct_path::TOKENS && g.k_chunks >= direct_path::WARPS &&
         (long long)g.row_tiles * g.k_chunks < (1ll << 30);
}

double gemv_direct_balance(const razer_desc* d) { return direct_plan(d).balance; }

template <int MT, int DEPTH>
static int launch_direct_cfg(const direct_path::Args& a, int grid, cudaStream_t st) {
  using C = direct_path::Cfg<MT>;
  auto kern = direct_path::razer_direct_kernel<MT, DEPTH>;
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
  a.units = p.units;
  if (p.mt == 2) return launch_direct_cfg<2, direct_path::DEPTH_MT2>(a, p.grid, st);
  return launch_direct_cfg<1, direct_path::DEPTH_MT1>(a, p.grid, st);
}

}  // namespace razer
