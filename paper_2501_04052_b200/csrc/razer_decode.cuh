// Register-level decode of packed RaZeR blocks to bf16 pairs, shared by the matmul kernels.
//
// Per pair of elements, with no comparison and no conversion instruction: the stored nibble
// is isolated in both 16-bit halves of the word, one integer multiply-add drops two shifted
// copies of it, one logic op keeps sign -> bit 15 and E1 E0 M -> bits 8:6 (a bf16 pattern worth
// value x 2^-126, subnormal for 0.5) and ORs in the special value, which one fused
// multiply-add with ReLU derives from the isolated nibble (the special value is the only
// nibble that is numerically zero); one packed bf16 multiply by +-scale x 2^126 finishes the
// exact product value x block scale (Sec. 3: dequantized element, without the tensor scale).
#pragma once

#include "razer_common.cuh"

namespace razer {

// Packed bf16 arithmetic on raw 32-bit patterns, through the compiler's own intrinsics (rather than
// inline PTX) so that it can place results directly in the consecutive registers the TMEM store or the
// MMA wants.
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t v) { return *reinterpret_cast<__nv_bfloat162*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ uint32_t fma_relu_bf16x2(uint32_t a, uint32_t b, uint32_t c) {
  return as_u32(__hfma2_relu(as_bf162(a), as_bf162(b), as_bf162(c)));
}
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) { return as_u32(__hmul2(as_bf162(a), as_bf162(b))); }
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) { return (a & b) | c; }

// Special-value constants of a block, selected by the scale byte's select bit.
struct SvConsts {
  uint32_t sv;               // (sv, sv) x 2^-126 as bf16x2
  uint32_t nsv_lo;           // -(sv x 2^7):  sv - nsv_lo * (nibble in bits 3:0 read as bf16) = 0 for nibble 1
  uint32_t nsv_hi;           // -(sv x 2^3):  the same for a nibble in bits 7:4
  uint32_t pad;
};

// Decode tables in shared memory.
//   ss[(negate << 6 | scale code)][lane] : (+-scale x 2^126) as bf16x2; one copy per lane so that a
//                                          warp's 32 lookups never collide on a bank
//   sv[select]                           : SvConsts
constexpr int DECODE_SS_ENTRIES = 128;
constexpr int DECODE_TABLE_BYTES = DECODE_SS_ENTRIES * 32 * 4 + 2 * 16;

struct DecodeTables {         // 32-bit shared-window addresses
  uint32_t ss_lane;          // &ss[0][lane]
  uint32_t sv;
};

// Fill the tables (all threads of the CTA call this; a __syncthreads() must follow).
__device__ __forceinline__ void decode_tables_fill(uint8_t* base, float sv0, float sv1, int tid, int nthreads) {
  // every entry is computed once per quarter (four threads per entry) and written as eight of its 32 lane copies
  for (int i = tid; i < DECODE_SS_ENTRIES * 4; i += nthreads) {
    const uint32_t idx = (uint32_t)i >> 2;
    // scale x 2^126 has four significant bits: the upper half of the FP32 pattern is the exact bf16
    const float sc = scale_value(idx & 0x3Fu) * 8.50705917e37f;   // 2^126
    const uint32_t b = (__float_as_uint(sc) >> 16) | ((idx & 0x40u) << 9);
    const uint32_t v = b | (b << 16);
    uint4* dst = reinterpret_cast<uint4*>(base + idx * 128 + (i & 3) * 32);
    dst[0] = make_uint4(v, v, v, v);
    dst[1] = make_uint4(v, v, v, v);
  }
  if (tid < 2) {
    const float sv = tid ? sv1 : sv0;                          // at most four significant bits
    const uint32_t p0 = __float_as_uint(sv * 1.17549435e-38f) >> 16;     // sv x 2^-126
    const uint32_t p1 = __float_as_uint(-sv * 128.0f) >> 16;
    const uint32_t p2 = __float_as_uint(-sv * 8.0f) >> 16;
    SvConsts c;
    c.sv = p0 | (p0 << 16);
    c.nsv_lo = p1 | (p1 << 16);
    c.nsv_hi = p2 | (p2 << 16);
    c.pad = 0;
    reinterpret_cast<SvConsts*>(base + DECODE_SS_ENTRIES * 32 * 4)[tid] = c;
  }
}

__device__ __forceinline__ DecodeTables decode_tables_view(const uint8_t* base, int lane) {
  DecodeTables t;
  t.ss_lane = smem_addr(base) + lane * 4;
  t.sv = smem_addr(base) + DECODE_SS_ENTRIES * 32 * 4;
  return t;
}

// Constants of block `blk` (0..3, compile-time) of a chunk, from the row's scale word
// (four packed scale bytes [select | negate | 6-bit scale code]).
__device__ __forceinline__ void decode_block_consts(const DecodeTables& t, uint32_t sw, int blk, uint32_t& ss2,
                                                    SvConsts& svc) {
  const uint32_t off_ss = (blk == 0 ? sw << 7 : sw >> (8 * blk - 7)) & 0x3F80u;   // (byte & 0x7F) * 128
  const uint32_t off_sv = (sw >> (8 * blk + 3)) & 0x10u;                          // (byte >> 7) * 16
  ss2 = lds32(t.ss_lane + off_ss);
  const uint4 c = lds128(t.sv + off_sv);
  svc.sv = c.x;
  svc.nsv_lo = c.y;
  svc.nsv_hi = c.z;
  svc.pad = 0;
}

// The same for a scale byte already shifted down to bits 7:0 (higher bits may hold anything).
__device__ __forceinline__ void decode_block_consts_byte(const DecodeTables& t, uint32_t sb, uint32_t& ss2, SvConsts& svc) {
  ss2 = lds32(t.ss_lane + ((sb << 7) & 0x3F80u));
  const uint4 c = lds128(t.sv + ((sb >> 3) & 0x10u));
  svc.sv = c.x;
  svc.nsv_lo = c.y;
  svc.nsv_hi = c.z;
  svc.pad = 0;
}

// The same for a scale word rotated so that the block's byte sits on bits 14:7 (higher and lower bits may hold
// anything), for tables that start on a 16 KB boundary of the shared window: the table offsets are then
// merged into the addresses by the same logic op that isolates them.
__device__ __forceinline__ void decode_block_consts_rot(const DecodeTables& t, uint32_t r, uint32_t& ss2, SvConsts& svc) {
  ss2 = lds32(and_or(r, 0x3F80u, t.ss_lane));
  const uint4 c = lds128(and_or(r >> 10, 0x10u, t.sv));
  svc.sv = c.x;
  svc.nsv_lo = c.y;
  svc.nsv_hi = c.z;
  svc.pad = 0;
}

// Four stored nibbles of each 16-bit half of `w` -> four bf16x2 registers (elements 2p, 2p+1
// of the word in register p), each the exact product value x scale with the block's sign.
// mul_lo = 2^6 + 2^12, mul_hi = 2^2 + 2^8 (run-time values so that they stay multiplies).
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t ss2, const SvConsts& c, uint32_t mul_lo,
                                            uint32_t mul_hi, uint32_t* out) {
  const uint32_t w8 = w >> 8;
  const uint32_t n0 = w & 0x000F000Fu, n1 = w & 0x00F000F0u;
  const uint32_t n2 = w8 & 0x000F000Fu, n3 = w8 & 0x00F000F0u;
  // nibble * (2^6 + 2^12) [bits 3:0] or * (2^2 + 2^8) [bits 7:4]: one copy lands with E1 E0 M on
  // bits 8:6, the other with S on bit 15; the mask keeps exactly those
  const uint32_t u0 = and_or(n0 * mul_lo, 0x81C081C0u, fma_relu_bf16x2(n0, c.nsv_lo, c.sv));
  const uint32_t u1 = and_or(n1 * mul_hi, 0x81C081C0u, fma_relu_bf16x2(n1, c.nsv_hi, c.sv));
  const uint32_t u2 = and_or(n2 * mul_lo, 0x81C081C0u, fma_relu_bf16x2(n2, c.nsv_lo, c.sv));
  const uint32_t u3 = and_or(n3 * mul_hi, 0x81C081C0u, fma_relu_bf16x2(n3, c.nsv_hi, c.sv));
  out[0] = mul_bf16x2(u0, ss2);
  out[1] = mul_bf16x2(u1, ss2);
  out[2] = mul_bf16x2(u2, ss2);
  out[3] = mul_bf16x2(u3, ss2);
}

}  // namespace razer
