// razer_quant_act: online RaZeR quantization of bf16 activations (Sec. 4.2, Eq. 1-3, 6-7).
//
// Every FP32 operation below is a single correctly rounded IEEE operation issued through
// an intrinsic (__fdiv_rn, __fmul_rn, __fadd_rn, __fsub_rn), so the compiler can neither
// fuse nor reorder them: block scale, scaled values, the two candidate errors and the
// choice between +sv and -sv are reproducible bit for bit.
#include "razer_common.cuh"

namespace razer {

// Round a non-negative finite float to the nearest E4M3 code (ties to even mantissa),
// saturating at `max_code`.
__device__ __forceinline__ uint32_t round_to_e4m3(float t, uint32_t max_code) {
  uint32_t code;
  if (t < 0.015625f) {                       // below 2^-6: subnormal grid, quantum 2^-9
    code = (uint32_t)__float2int_rn(__fmul_rn(t, 512.0f));   // exact product, ties to even
  } else {
    const uint32_t b = __float_as_uint(t);
    const uint32_t e = (b >> 23) - 120u;     // biased E4M3 exponent (>= 1 here)
    const uint32_t man = b & 0x7FFFFFu;
    const uint32_t keep = man >> 20, rem = man & 0xFFFFFu;
    const uint32_t up = (rem > 0x80000u) || (rem == 0x80000u && (keep & 1u));
    code = (e >= 32u) ? max_code : ((e << 3) | keep) + up;   // a mantissa carry bumps the exponent
  }
  return min(code, max_code);
}

// Saturating round-to-nearest-even onto the FP4 magnitudes 0 .5 1 1.5 2 3 4 6 (Eq. 3).
__device__ __forceinline__ uint32_t round_to_fp4_idx(float a) {
  return (uint32_t)(a > 0.25f) + (uint32_t)(a >= 0.75f) + (uint32_t)(a > 1.25f) +
         (uint32_t)(a >= 1.75f) + (uint32_t)(a > 2.5f) + (uint32_t)(a >= 3.5f) + (uint32_t)(a > 5.0f);
}

// Quantize one 16-element block (Eq. 2-3, 6-7 with the candidates +sv and -sv): eight code bytes and the scale byte.
__device__ __forceinline__ void quant_act_block(const uint4 v0, const uint4 v1, float d32, float d32x6, float sv_mag,
                                                uint32_t& w0, uint32_t& w1, uint32_t& sbyte) {
  const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
  float xv[16];
  float bmax = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    xv[2 * j] = __uint_as_float(w[j] << 16);
    xv[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
    bmax = fmaxf(bmax, fmaxf(fabsf(xv[2 * j]), fabsf(xv[2 * j + 1])));
  }
  w0 = 0, w1 = 0, sbyte = 0;
  if (bmax > 0.0f) {
    const float tq = __fdiv_rn(bmax, d32x6);                         // Eq. 2 argument
    uint32_t scode = round_to_e4m3(tq, 126u);
    if (scode == 0) scode = 1;                                       // keep a non-empty block alive
    const float denom = __fmul_rn(d32, scale_value(scode));
    float e_pos = 0.0f, e_neg = 0.0f;
    uint32_t std_code[16];
    uint32_t take_pos = 0, take_neg = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float xs = __fdiv_rn(xv[j], denom);                      // the scaled block of Eq. 6
      const uint32_t idx = round_to_fp4_idx(fabsf(xs));
      const uint32_t neg = __float_as_uint(xs) >> 31;
      const float r = neg ? -fp4_mag(idx) : fp4_mag(idx);
      const float d_r = fabsf(__fsub_rn(xs, r));
      const float d_p = fabsf(__fsub_rn(xs, sv_mag));
      const float d_n = fabsf(__fsub_rn(xs, -sv_mag));
      const bool tp = d_p < d_r, tn = d_n < d_r;                     // strictly closer only
      const float qp = tp ? sv_mag : r, qn = tn ? -sv_mag : r;
      const float dp = __fsub_rn(qp, xs), dn = __fsub_rn(qn, xs);
      e_pos = __fadd_rn(e_pos, __fmul_rn(dp, dp));                   // ascending j, no fusion
      e_neg = __fadd_rn(e_neg, __fmul_rn(dn, dn));
      take_pos |= (uint32_t)tp << j;
      take_neg |= (uint32_t)tn << j;
      std_code[j] = idx ? (idx | (neg << 3)) : 0u;                   // a true zero is always code 0
    }
    const bool use_neg = e_neg < e_pos;                              // ties keep metadata 0 (+sv)
    const uint32_t take = use_neg ? take_neg : take_pos;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint32_t c = ((take >> j) & 1u) ? 8u : std_code[j];
      if (j < 8) w0 |= c << (4 * j); else w1 |= c << (4 * (j - 8));
    }
    sbyte = (use_neg ? 0x80u : 0u) | scode;
  }
}

// One launch for the whole of razer_quant_act, one thread per 16-element block.  When the tensor scale has to be
// computed (Eq. 1), the grid first takes the tensor maximum: every CTA folds its share into sync[0] and counts
// itself in sync[1], and all of them meet there (the launch is cooperative, so every CTA is resident; the wait is
// bounded all the same).  sync[] must be zero when the kernel starts; the last CTA to finish sets it back to zero.
// Where the quantizer writes: the interchange format (prepared == 0), or the FP4 activation operand of the
// block-scaled tensor-core kernel (Fp4ActLayout: codes padded to KP columns with each word's nibbles in the packed
// order, scale bytes in scale-factor tile order; the padding is written as zeros by this kernel too).
struct QuantActOut {
  int prepared;
  int M, k16, kp16, spt, m_pad;      // rows; 16-element blocks per row of the input / of the padded operand; stages; padded rows
};

__global__ void __launch_bounds__(256) quant_act_fused_kernel(const uint4* __restrict__ x, long long n_blocks, float sv_mag,
                                                             const float* __restrict__ scale_in, uint32_t* sync,
                                                             uint2* __restrict__ codes, uint8_t* __restrict__ scales,
                                                             float* __restrict__ scale_out, const QuantActOut o) {
  __shared__ uint32_t warp_max[8];
  __shared__ uint32_t amax_shared;
  float d32;
  if (scale_in) {
    d32 = *scale_in;
  } else {
    uint32_t m = 0;
    const long long n_vec = n_blocks * 2;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (long long)gridDim.x * blockDim.x) {
      const uint4 v = x[i];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t lo = w[j] & 0x7FFFu, hi = (w[j] >> 16) & 0x7FFFu;
        m = max(m, (lo > 0x7F80u) ? 0u : lo);                          // NaN patterns are skipped
        m = max(m, (hi > 0x7F80u) ? 0u : hi);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int i = 1; i < 8; ++i) m = max(m, warp_max[i]);
      if (m) atomicMax(&sync[0], m);
      __threadfence();
      atomicAdd(&sync[1], 1u);
      // all CTAs are resident (cooperative launch); the bound only guards against a dirty sync[]
      uint32_t seen = 0;
      for (uint32_t spins = 0; spins < (1u << 22); ++spins) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(sync + 1) : "memory");
        if (seen >= gridDim.x) break;
        __nanosleep(64);
      }
      uint32_t a;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(a) : "l"(sync) : "memory");
      amax_shared = seen >= gridDim.x ? a : 0xFFFFFFFFu;               // gave up: flagged below with a NaN scale
    }
    __syncthreads();
    const uint32_t bits = amax_shared;
    if (bits == 0xFFFFFFFFu) {
      if (blockIdx.x == 0 && threadIdx.x == 0) *scale_out = __uint_as_float(0x7FC00000u);
      return;
    }
    const float amax = __uint_as_float(bits << 16);
    d32 = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, __fmul_rn(448.0f, 6.0f));   // Eq. 1
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *scale_out = d32;
  const float d32x6 = __fmul_rn(d32, 6.0f);
  if (!o.prepared) {
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_blocks;
         t += (long long)gridDim.x * blockDim.x) {
      uint32_t w0, w1, sbyte;
      quant_act_block(x[2 * t], x[2 * t + 1], d32, d32x6, sv_mag, w0, w1, sbyte);
      codes[t] = make_uint2(w0, w1);
      scales[t] = (uint8_t)sbyte;
    }
  } else {
    // one thread per block of the PADDED operand: (row m, block kb); blocks beyond K and rows beyond M are zeros
    auto shuffle = [](uint32_t w) -> uint32_t {                        // element j of the word: nibble j -> nibble j / 2 + 4 (j % 2)
      uint32_t r = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) r |= ((w >> (4 * j)) & 0xFu) << (4 * ((j >> 1) + 4 * (j & 1)));
      return r;
    };
    const long long n_virtual = (long long)o.m_pad * o.kp16;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_virtual;
         t += (long long)gridDim.x * blockDim.x) {
      const int m = (int)(t / o.kp16), kb = (int)(t - (long long)m * o.kp16);
      uint32_t w0 = 0, w1 = 0, sbyte = 0;
      if (m < o.M && kb < o.k16) {
        const long long src = (long long)m * o.k16 + kb;
        quant_act_block(x[2 * src], x[2 * src + 1], d32, d32x6, sv_mag, w0, w1, sbyte);
      }
      if (m < o.M) codes[(long long)m * o.kp16 + kb] = make_uint2(shuffle(w0), shuffle(w1));
      // scale-factor tile of (128-token tile, stage, chunk); inside it word 4 * (t % 32) + t / 32, byte = block of the chunk
      const int tile = m >> 7, tm = m & 127, step = kb >> 4, c = (kb >> 2) & 3;
      const size_t at = (((size_t)tile * o.spt + step) * 4 + c) * 512 + (size_t)((tm & 31) * 4 + (tm >> 5)) * 4 + (kb & 3);
      scales[at] = (uint8_t)(sbyte & 0x7Fu);
    }
  }
  if (!scale_in) {
    __syncthreads();
    if (threadIdx.x == 0) {
      const uint32_t prev = atomicAdd(&sync[1], 1u);
      if (prev + 1 == 2 * gridDim.x) {                                 // everyone has read the maximum: leave sync[] clean
        sync[0] = 0;
        sync[1] = 0;
      }
    }
  }
}

// ------------------------------------------------------------------ offline weight quantizer (Sec. 4.2)
// The same procedure as the activation quantizer above with the weight format: FP32 input, the 6-bit E3M3
// block scale (codes 0..63 of the E4M3 grid, maximum 1.875) and four candidate special values
// +m0, +m1, -m0, -m1 in metadata order (meta = sign * 2 + select, bits 7:6 of the scale byte).

// Tensor maximum of |w| over FP32 input (Eq. 1 numerator); NaNs are skipped.
__global__ void weight_amax_kernel(const float4* __restrict__ w, long long n_vec, uint32_t* __restrict__ amax_bits) {
  uint32_t m = 0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 v = w[i];
    const uint32_t b[4] = {__float_as_uint(v.x) & 0x7FFFFFFFu, __float_as_uint(v.y) & 0x7FFFFFFFu,
                           __float_as_uint(v.z) & 0x7FFFFFFFu, __float_as_uint(v.w) & 0x7FFFFFFFu};
#pragma unroll
    for (int j = 0; j < 4; ++j) m = max(m, (b[j] > 0x7F800000u) ? 0u : b[j]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ uint32_t warp_max[32];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x + 31) / 32 ? warp_max[threadIdx.x] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (threadIdx.x == 0 && m) atomicMax(amax_bits, m);
  }
}

// One thread per scale block of `sub` groups of 16 elements (block size 16 * sub).  Three walks over the block:
// its maximum, the candidates' errors (FP32, ascending element order across the whole block), and the codes
// under the winning candidate.
//
// AWARE = false: the four special values share the scale of Eq. 2 (block maximum -> 6), Eq. 6-7 as printed.
// AWARE = true: a special value beyond 6 whose sign is that of the block's first largest element brings a
// second candidate with a scale of its own (block maximum -> |v|); slots 4 and 5 hold those for m0 and m1.
// Errors are then compared in the tensor's units, fl32(fl32(d * d) * e) with d the candidate's step.
template <bool AWARE>
__global__ void quant_weight_kernel(const float4* __restrict__ w, long long n_blocks, int sub, float m0, float m1,
                                    uint32_t remap_code, const float* __restrict__ scale_in,
                                    const uint32_t* __restrict__ amax_bits, uint2* __restrict__ codes,
                                    uint8_t* __restrict__ scales, float* __restrict__ scale_out) {
  constexpr int NC = AWARE ? 6 : 4;
  float d32;
  if (scale_in) {
    d32 = *scale_in;
  } else {
    const float amax = __uint_as_float(*amax_bits);
    d32 = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, __fmul_rn(1.875f, 6.0f));   // Eq. 1
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *scale_out = d32;
  const uint32_t other_zero = remap_code ^ 8u;
  const float mags[2] = {m0, m1};
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_blocks;
       t += (long long)gridDim.x * blockDim.x) {
    const float4* src = w + 4 * t * sub;
    float bmax = 0.0f;
    uint32_t top_neg = 0;                                              // sign of the first largest element
    for (int q = 0; q < 4 * sub; ++q) {
      const float4 v = src[q];
      const float xv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (fabsf(xv[j]) > bmax) { bmax = fabsf(xv[j]); top_neg = __float_as_uint(xv[j]) >> 31; }
    }
    uint32_t sbyte = 0;
    float denom = 1.0f, sv = m0;
    if (bmax > 0.0f) {
      float cv[NC], cd[NC];
      uint32_t cs[NC], cm[NC];
      bool ok[NC];
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const float qmax = c < 4 ? 6.0f : mags[c - 4];
        const float tq = __fdiv_rn(bmax, __fmul_rn(d32, qmax));        // Eq. 2 argument
        uint32_t scode = round_to_e4m3(tq, 63u);
        if (scode == 0) scode = 1;                                     // keep a non-empty block alive
        cs[c] = scode;
        cd[c] = __fmul_rn(d32, scale_value(scode));
        cm[c] = c < 4 ? (uint32_t)c : (top_neg * 2u + (uint32_t)(c - 4));
        cv[c] = (cm[c] & 2u) ? -mags[cm[c] & 1u] : mags[cm[c] & 1u];
        ok[c] = c < 4 || mags[c - 4] > 6.0f;
      }
      float err[NC];
#pragma unroll
      for (int c = 0; c < NC; ++c) err[c] = 0.0f;
#pragma unroll 1
      for (int q = 0; q < 4 * sub; ++q) {
        const float4 v = src[q];
        const float xv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          // the four standard candidates share the scale of Eq. 2, hence the scaled value and its FP4 rounding
          float xs = 0.0f, r = 0.0f, d_r = 0.0f;
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            if (c >= 4 && !ok[c]) continue;
            if (c == 0 || c >= 4) {
              xs = __fdiv_rn(xv[j], cd[c]);                            // the scaled block of Eq. 6
              const uint32_t idx = round_to_fp4_idx(fabsf(xs));
              r = (__float_as_uint(xs) >> 31) ? -fp4_mag(idx) : fp4_mag(idx);
              d_r = fabsf(__fsub_rn(xs, r));
            }
            const bool tk = fabsf(__fsub_rn(xs, cv[c])) < d_r;         // strictly closer only
            const float d = __fsub_rn(tk ? cv[c] : r, xs);
            err[c] = __fadd_rn(err[c], __fmul_rn(d, d));               // ascending element order, no fusion
          }
        }
      }
      if (AWARE) {
#pragma unroll
        for (int c = 0; c < NC; ++c) err[c] = __fmul_rn(__fmul_rn(cd[c], cd[c]), err[c]);
      }
      int pick = 0;                                                    // first minimum: ties keep the earlier candidate
      float best = err[0];
#pragma unroll
      for (int c = 1; c < NC; ++c)
        if (ok[c] && err[c] < best) { best = err[c]; pick = c; }
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (c == pick) { sbyte = (cm[c] << 6) | cs[c]; denom = cd[c]; sv = cv[c]; }
    }
#pragma unroll 1
    for (int g = 0; g < sub; ++g) {
      uint32_t wd[2] = {other_zero * 0x11111111u, other_zero * 0x11111111u};
      if (bmax > 0.0f) {
        wd[0] = wd[1] = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v = src[4 * g + q];
          const float xv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float xs = __fdiv_rn(xv[j], denom);
            const uint32_t idx = round_to_fp4_idx(fabsf(xs));
            const uint32_t neg = __float_as_uint(xs) >> 31;
            const float r = neg ? -fp4_mag(idx) : fp4_mag(idx);
            const bool tk = fabsf(__fsub_rn(xs, sv)) < fabsf(__fsub_rn(xs, r));
            const uint32_t c = tk ? remap_code : (idx ? (idx | (neg << 3)) : other_zero);   // a true zero is always the other zero code
            const int e = 4 * q + j;
            wd[e >> 3] |= c << (4 * (e & 7));
          }
        }
      }
      codes[t * sub + g] = make_uint2(wd[0], wd[1]);
    }
    scales[t] = (uint8_t)sbyte;
  }
}

int launch_quant_weight(const float* w, int N, int K, int block, int scale_aware, float m0, float m1, int remap_code,
                        const float* scale_in,
                        uint32_t* amax_scratch, uint8_t* codes, uint8_t* scales, float* scale_out, cudaStream_t st) {
  const int sub = block / 16;
  const long long n_blocks = (long long)N * (K / block);
  const long long n_vec = (long long)N * (K / 4);
  const int threads = 256;
  if (!scale_in) {
    RAZER_TRY(check_cuda(cudaMemsetAsync(amax_scratch, 0, sizeof(uint32_t), st), "amax memset"));
    long long b = (n_vec + threads * 4 - 1) / (threads * 4);
    const int g2 = (int)(b < 1 ? 1 : (b > 296 ? 296 : b));
    weight_amax_kernel<<<g2, threads, 0, st>>>((const float4*)w, n_vec, amax_scratch);
    count_launches(1);
    RAZER_TRY(check_cuda(cudaGetLastError(), "weight_amax_kernel launch"));
  }
  long long b = (n_blocks + threads - 1) / threads;
  const int g = (int)(b < 1 ? 1 : (b > 148LL * 16 ? 148LL * 16 : b));
  if (scale_aware)
    quant_weight_kernel<true><<<g, threads, 0, st>>>((const float4*)w, n_blocks, sub, m0, m1, (uint32_t)remap_code, scale_in,
                                                     amax_scratch, (uint2*)codes, scales, scale_out);
  else
    quant_weight_kernel<false><<<g, threads, 0, st>>>((const float4*)w, n_blocks, sub, m0, m1, (uint32_t)remap_code, scale_in,
                                                      amax_scratch, (uint2*)codes, scales, scale_out);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "quant_weight_kernel launch");
}

static int launch_quant_act_any(const void* x, int M, int K, float sv_mag, const float* scale_in, uint32_t* sync_scratch,
                                uint8_t* codes, uint8_t* scales, float* scale_out, const QuantActOut& o, cudaStream_t st) {
  const long long n_blocks = (long long)M * (K / 16);
  const long long n_work = o.prepared ? (long long)o.m_pad * o.kp16 : n_blocks;
  const int threads = 256;
  static int max_ctas = 0;                                             // CTAs that are resident together (cooperative launch)
  if (!max_ctas) {
    int dev = 0, sms = 0, per_sm = 0;
    RAZER_TRY(check_cuda(cudaGetDevice(&dev), "cudaGetDevice"));
    RAZER_TRY(check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "cudaDeviceGetAttribute"));
    RAZER_TRY(check_cuda(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quant_act_fused_kernel, threads, 0),
                         "cudaOccupancyMaxActiveBlocksPerMultiprocessor"));
    max_ctas = sms * (per_sm < 1 ? 1 : per_sm);
  }
  long long b = (n_work + threads - 1) / threads;
  const int grid = (int)(b < 1 ? 1 : (b > max_ctas ? max_ctas : b));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(threads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = scale_in ? 0 : 1;                                     // the grid only meets when it computes the scale
  const cudaError_t e = cudaLaunchKernelEx(&cfg, quant_act_fused_kernel, (const uint4*)x, n_blocks, sv_mag, scale_in,
                                           sync_scratch, (uint2*)codes, scales, scale_out, o);
  count_launches(1);
  return check_cuda(e, "quant_act_fused_kernel launch");
}

int launch_quant_act(const void* x, int M, int K, float sv_mag, const float* scale_in,
                     uint32_t* sync_scratch, uint8_t* codes, uint8_t* scales, float* scale_out,
                     cudaStream_t st) {
  QuantActOut o = {};
  return launch_quant_act_any(x, M, K, sv_mag, scale_in, sync_scratch, codes, scales, scale_out, o, st);
}

// Plain NVFP4 quantization (no special value) straight into the FP4 activation operand of the block-scaled kernel.
int launch_quant_act_fp4(const void* x, int M, int K, const float* scale_in, uint32_t* sync_scratch, void* act_fp4,
                         float* scale_out, cudaStream_t st) {
  const Fp4ActLayout L = make_fp4_act_layout(M, K);
  QuantActOut o;
  o.prepared = 1;
  o.M = M;
  o.k16 = K / 16;
  o.kp16 = L.KP / 16;
  o.spt = L.spt;
  o.m_pad = L.tiles128 * 128;
  uint8_t* codes = (uint8_t*)act_fp4;
  return launch_quant_act_any(x, M, K, 0.0f, scale_in, sync_scratch, codes, codes + L.codes_bytes, scale_out, o, st);
}

}  // namespace razer
