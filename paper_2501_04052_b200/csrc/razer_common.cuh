// Shared declarations of the RaZeR CUDA library: packed-layout geometry, error plumbing,
// small device helpers.  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/razer.h"

namespace razer {

// ---------------------------------------------------------------------------------
// Packed layout (GPU-internal form written by razer_pack_layout)
//
// The tensor is cut into strips of STRIP_ROWS = 16 rows (one tensor-core row tile of the decode kernel) and
// chunks of CHUNK_K = 64 columns (4 blocks of 16).  One strip-chunk ("piece") is PIECE_BYTES = 576 contiguous
// bytes, and the pieces are ordered [strip][k chunk]: the whole K run of a strip is one contiguous byte range,
// so any k range of any group of strips reaches shared memory with one bulk copy per strip.
//   piece = [blk 0..3][slot 0..15] 8 bytes : the block's 16 nibbles as two 32-bit words; row r of the strip sits
//                                            in slot r ^ (4 * blk), so that thread = row reads (16 consecutive
//                                            slots) stay contiguous while the fragment-style read of the
//                                            decode kernel (lane (g, t) reads rows g and g + 8 of block t)
//                                            covers all banks; element j of the block sits in word j / 8,
//                                            nibble (j % 8) / 2 + 4 * (j % 2), so that nibbles p and p + 4 of
//                                            a word (the same position in its two 16-bit halves) are
//                                            elements 2p and 2p + 1
//           [g 0..7][blk 0..3][h 0..1] 1 byte : scale byte of row g + 8 h, block blk (the two bytes a lane
//                                            of the decode kernel needs are adjacent; a row's four bytes
//                                            sit in one 8-byte group)
// Rows are padded to whole 128-row tiles (8 strips, what the tcgen05 kernel takes as one MMA tile) and columns
// to whole chunks; rows beyond N and columns beyond K are zero blocks (scale byte 0).
//
// Inside the packed form:
//   * the special value is always nibble 0x0, a true zero always nibble 0x8, every other
//     nibble is S E1 E0 M as in Eq. 5;
//   * a block whose special value is negative is stored negated (sign bits of all non-zero
//     codes flipped) so that nibble 0x0 always means "+sv_mag[select]";
//   * scale byte = [select | negate | 6-bit scale code]; negate = 1 means the block's
//     values are the negatives of the stored codes' values.
// With these conventions the decoder needs no comparison: the nibble's bits drop into a
// bf16 bit pattern (sign to bit 15, E1 E0 M to bits 8:6, value x 2^-126), the special value
// is the one nibble that is numerically zero, and the block sign rides on the scale.
// ---------------------------------------------------------------------------------
constexpr int TILE_ROWS = 128;
constexpr int STRIP_ROWS = 16;
constexpr int TILE_STRIPS = TILE_ROWS / STRIP_ROWS;              // 8
constexpr int CHUNK_K = 64;
constexpr int CHUNK_BLOCKS = CHUNK_K / 16;
constexpr int PIECE_CODE_BYTES = CHUNK_BLOCKS * STRIP_ROWS * 8;  // 512
constexpr int PIECE_SCALE_BYTES = STRIP_ROWS * CHUNK_BLOCKS;     // 64
constexpr int PIECE_BYTES = PIECE_CODE_BYTES + PIECE_SCALE_BYTES;   // 576
constexpr int CHUNK_BYTES = TILE_STRIPS * PIECE_BYTES;           // 4608: one 128-row tile x 64 columns

struct Geometry {
  int N, K;
  int row_tiles;   // ceil(N / 128)
  int k_chunks;    // ceil(K / 64)
  __host__ __device__ int strips() const { return row_tiles * TILE_STRIPS; }
  __host__ __device__ size_t strip_bytes() const { return (size_t)k_chunks * PIECE_BYTES; }   // one strip's K run
  __host__ __device__ size_t packed_bytes() const {
    return (size_t)row_tiles * (size_t)k_chunks * CHUNK_BYTES;
  }
};

__host__ __device__ inline Geometry make_geometry(int N, int K) {
  Geometry g;
  g.N = N;
  g.K = K;
  g.row_tiles = (N + TILE_ROWS - 1) / TILE_ROWS;
  g.k_chunks = (K + CHUNK_K - 1) / CHUNK_K;
  return g;
}

// Every matmul workspace starts with the device status word (0 = ok), on a block of its own.
constexpr size_t WS_STATUS_BYTES = 256;

// Layout of the FP4 activation operand as the block-scaled tensor-core kernel reads it (written by the activation
// re-layout kernel or directly by the quantizer): codes [M][KP / 2] bytes (KP = K rounded up to whole 256-column
// stages, zero beyond K, the nibbles of every 32-bit word in the packed form's order), then scale-factor tiles
// [128-token tile][stage][chunk][512 bytes] (word 4 * (t % 32) + t / 32 of a tile = the four 7-bit scale bytes of
// token t of the tile for the chunk's four blocks; zero for tokens beyond M and blocks beyond K).
struct Fp4ActLayout {
  int NT;            // tokens per tile of the matmul kernel: 128, or 256 above 128 tokens
  int token_tiles, tiles128, spt, KP;
  size_t codes_bytes, sfb_bytes;
};
Fp4ActLayout make_fp4_act_layout(int M, int K);   // host (razer_gemm_fp4.cu)

// Decode parameters derived from a razer_desc on the host, passed to kernels by value.
struct DecodeParams {
  float sv_mag[2];
  float tensor_scale;
  int remap_code;
};

// ---------------------------------------------------------------------------------
// Error plumbing (host)
// ---------------------------------------------------------------------------------
int set_error(int code, const char* fmt, ...);
int check_desc(const razer_desc* d);
int check_cuda(cudaError_t e, const char* what);
void count_launches(int n);   // bookkeeping behind razer_kernel_launches()
bool sv_allowed(float m);

#define RAZER_TRY(expr)            \
  do {                             \
    int _rc = (expr);              \
    if (_rc != RAZER_OK) return _rc; \
  } while (0)

// ---------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------

// FP4-E2M1 magnitude of the low three bits (Eq. 5): 0 .5 1 1.5 2 3 4 6.
__device__ __forceinline__ float fp4_mag(uint32_t idx) {
  const uint32_t e = (idx >> 1) & 3u;
  const uint32_t m = idx & 1u;
  // e != 0: 2^(e-1) * (1 + m/2); e == 0: m/2.  Build the float from its fields.
  const float normal = __uint_as_float(((126u + e) << 23) | (m << 22));
  return e ? normal : 0.5f * (float)m;
}

// Value of a 6/7-bit E4M3-coded block scale (Eq. 4, sign ignored).
__device__ __forceinline__ float scale_value(uint32_t code) {
  const uint32_t e = (code >> 3) & 0xFu;
  const uint32_t m = code & 7u;
  const float normal = __uint_as_float(((120u + e) << 23) | (m << 20));
  return e ? normal : (float)m * 0.001953125f;   // m * 2^-9
}

// Byte offsets inside a piece: the code words of row r (0..15) of block blk, and that block's scale byte.
__host__ __device__ __forceinline__ int piece_code_offset(int blk, int r) { return (blk * STRIP_ROWS + (r ^ (4 * blk))) * 8; }
__host__ __device__ __forceinline__ int piece_scale_offset(int blk, int r) {
  return PIECE_CODE_BYTES + (r & 7) * 8 + blk * 2 + (r >> 3);
}
// Byte offset of the piece of (row n, k chunk c) in the packed buffer.
__host__ __device__ __forceinline__ size_t piece_offset(const Geometry& g, int n, int c) {
  return ((size_t)(n / STRIP_ROWS) * g.k_chunks + c) * PIECE_BYTES;
}
constexpr uint32_t PACKED_NEGATE = 0x40u, PACKED_SELECT = 0x80u;   // bits of a packed scale byte

// Position (in bits) of element j's nibble inside the block's 64-bit code word.
__host__ __device__ __forceinline__ int packed_nibble_shift(int j) {
  return 32 * (j >> 3) + 4 * (((j & 7) >> 1) + 4 * (j & 1));
}

// Stored nibble of element j of a packed block.
__device__ __forceinline__ uint32_t packed_nibble(uint2 cw, int j) {
  const int sh = packed_nibble_shift(j);
  return ((sh < 32 ? cw.x >> sh : cw.y >> (sh - 32))) & 0xFu;
}

// Element value of a packed-form nibble: 0x0 is +sv, 0x8 is zero, everything else Eq. 5.
__device__ __forceinline__ float packed_elem(uint32_t nib, float sv) {
  const float mag = fp4_mag(nib & 7u);
  const float v = (nib & 8u) ? -mag : mag;
  return (nib == 0u) ? sv : v;
}

// Shared-memory loads by 32-bit shared-window address.  Pointers into dynamic shared memory that
// went through integer alignment arithmetic are generic to the compiler; these keep the loads
// in the shared address space (no 64-bit address math, no generic-address resolution).
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) {
  return __uint_as_float(b << 16);
}

}  // namespace razer
