// razer_pack_layout, razer_dequant, razer_decode_act: layout shuffle and exact decode kernels.
#include "razer_common.cuh"

namespace razer {

// One thread per (row tile, k chunk, block, row): reads the interchange-format block
// (8 code bytes + 1 scale byte), canonicalises it and writes it at its packed position.
// `sub` = 16-element groups per scale block (block size / 16): the packed form always carries one scale byte per 16
// elements, so a larger block's byte is repeated for each of its groups and the kernels need not know the block size.
__global__ void pack_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                            uint8_t* __restrict__ packed, Geometry g, int remap_code, int sub) {
  const long long total = (long long)g.row_tiles * g.k_chunks * CHUNK_BLOCKS * TILE_ROWS;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int row_in = (int)(t % TILE_ROWS);
    const int blk = (int)((t / TILE_ROWS) % CHUNK_BLOCKS);
    const long long chunk = t / (TILE_ROWS * CHUNK_BLOCKS);
    const int kc = (int)(chunk % g.k_chunks);
    const int rt = (int)(chunk / g.k_chunks);
    const int n = rt * TILE_ROWS + row_in;
    const int kb = kc * CHUNK_BLOCKS + blk;            // block index along K
    uint32_t w0 = 0, w1 = 0, sb = 0;
    if (n < g.N && kb * 16 < g.K) {
      const uint2 c = *reinterpret_cast<const uint2*>(codes + (size_t)n * (g.K / 2) + (size_t)kb * 8);
      w0 = c.x;
      w1 = c.y;
      sb = scales[(size_t)n * (g.K / 16 / sub) + kb / sub];
    }
    // bit 3 of each nibble of nz is set iff the nibble's magnitude (low three bits) is non-zero
    auto canon = [&](uint32_t w, bool negate) -> uint32_t {
      const uint32_t m = w & 0x77777777u;
      const uint32_t nz = ((m + 0x77777777u) & 0x88888888u);
      if (remap_code == 0x8) w ^= (~nz) & 0x88888888u;  // packed form: special value 0x0, true zero 0x8
      if (negate) w ^= nz;                              // flip the sign of non-zero codes
      return w;
    };
    // interchange nibble order (element j in nibble j) -> packed order (nibbles p and p+4 = elements 2p, 2p+1)
    auto shuffle = [](uint32_t w) -> uint32_t {
      uint32_t o = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) o |= ((w >> (4 * j)) & 0xFu) << (4 * ((j >> 1) + 4 * (j & 1)));
      return o;
    };
    const uint32_t scode = sb & 0x3Fu;
    const bool negate = (sb & 0x80u) != 0;              // negative special value: store the block negated
    uint32_t out_sb = 0;
    if (scode != 0) {
      out_sb = (negate ? PACKED_NEGATE : 0u) | ((sb & 0x40u) ? PACKED_SELECT : 0u) | scode;
      w0 = shuffle(canon(w0, negate));
      w1 = shuffle(canon(w1, negate));
    } else {
      w0 = w1 = 0x88888888u;                            // zero block: sixteen true zeros
    }
    uint8_t* base = packed + piece_offset(g, n, kc);
    *reinterpret_cast<uint2*>(base + piece_code_offset(blk, row_in % STRIP_ROWS)) = make_uint2(w0, w1);
    base[piece_scale_offset(blk, row_in % STRIP_ROWS)] = (uint8_t)out_sb;
  }
}

// One thread per packed block: 16 outputs.  D1 = block_scale * element is exact in bf16;
// zeros are written as +0 whatever the stored sign.
template <bool FP32_OUT>
__global__ void dequant_kernel(const uint8_t* __restrict__ packed, void* __restrict__ out, Geometry g,
                               DecodeParams p) {
  const long long total = (long long)g.row_tiles * g.k_chunks * CHUNK_BLOCKS * TILE_ROWS;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int row_in = (int)(t % TILE_ROWS);
    const int blk = (int)((t / TILE_ROWS) % CHUNK_BLOCKS);
    const long long chunk = t / (TILE_ROWS * CHUNK_BLOCKS);
    const int kc = (int)(chunk % g.k_chunks);
    const int rt = (int)(chunk / g.k_chunks);
    const int n = rt * TILE_ROWS + row_in;
    const int k0 = (kc * CHUNK_BLOCKS + blk) * 16;
    if (n >= g.N || k0 >= g.K) continue;
    const uint8_t* base = packed + piece_offset(g, n, kc);
    const uint2 c = *reinterpret_cast<const uint2*>(base + piece_code_offset(blk, row_in % STRIP_ROWS));
    const uint32_t sb = base[piece_scale_offset(blk, row_in % STRIP_ROWS)];
    float s = scale_value(sb & 0x3Fu);
    if (sb & PACKED_NEGATE) s = -s;
    const float sv = p.sv_mag[(sb & PACKED_SELECT) ? 1 : 0];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float d1 = packed_elem(packed_nibble(c, j), sv) * s;   // exact: <= 8 significant bits
      d1 = __fadd_rn(d1, 0.0f);                       // canonical +0 (-0 + 0 = +0)
      const size_t o = (size_t)n * g.K + k0 + j;
      if (FP32_OUT) {
        reinterpret_cast<float*>(out)[o] = __fmul_rn(p.tensor_scale, d1);
      } else {
        reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(d1);
      }
    }
  }
}

// Activations in the interchange format (E4M3 scale, metadata bit 7 = sign of the special
// value, remapped code 0x8) -> bf16 block_scale * element.  One thread per block.
__global__ void decode_act_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                  __nv_bfloat16* __restrict__ out, long long n_blocks, float sv_mag) {
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_blocks;
       t += (long long)gridDim.x * blockDim.x) {
    const uint2 c = *reinterpret_cast<const uint2*>(codes + t * 8);
    const uint32_t sb = scales[t];
    const float s = scale_value(sb & 0x7Fu);
    const float sv = (sb & 0x80u) ? -sv_mag : sv_mag;
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
      const uint32_t w = (j < 8) ? c.x : c.y;
      const uint32_t n0 = (w >> (4 * (j & 7))) & 0xFu;
      const uint32_t n1 = (w >> (4 * (j & 7) + 4)) & 0xFu;
      float a = (n0 == 8u) ? sv : ((n0 & 8u) ? -fp4_mag(n0 & 7u) : fp4_mag(n0 & 7u));
      float b = (n1 == 8u) ? sv : ((n1 & 8u) ? -fp4_mag(n1 & 7u) : fp4_mag(n1 & 7u));
      a *= s;
      b *= s;
      a = __fadd_rn(a, 0.0f);                           // canonical +0
      b = __fadd_rn(b, 0.0f);
      const uint32_t lo = __float_as_uint(a) >> 16;     // exact: the product fits bf16
      const uint32_t hi = __float_as_uint(b) >> 16;
      o[j / 2] = lo | (hi << 16);
    }
    uint4* dst = reinterpret_cast<uint4*>(out + t * 16);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

static int grid_for(long long total, int threads) {
  long long b = (total + threads - 1) / threads;
  const long long cap = 148LL * 32;
  return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

// The matmul kernels are launched with programmatic stream serialization and begin to fetch packed weights
// before the kernel ahead of them in the stream is known to have finished (only activations, workspace and
// outputs wait for it).  An empty, ordinarily launched kernel behind the pack kernel makes that kernel, not
// the one that writes the weights, the matmul's predecessor: it cannot start before the weights are written
// and visible.
__global__ void pack_done_kernel() {}

int launch_pack(const razer_desc* d, const uint8_t* codes, const uint8_t* scales, void* packed,
                cudaStream_t st) {
  const Geometry g = make_geometry(d->N, d->K);
  const long long total = (long long)g.row_tiles * g.k_chunks * CHUNK_BLOCKS * TILE_ROWS;
  pack_kernel<<<grid_for(total, 256), 256, 0, st>>>(codes, scales, (uint8_t*)packed, g, d->remap_code, d->block / 16);
  count_launches(1);
  RAZER_TRY(check_cuda(cudaGetLastError(), "pack_kernel launch"));
  pack_done_kernel<<<1, 32, 0, st>>>();
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pack_done_kernel launch");
}

int launch_dequant(const razer_desc* d, const void* packed, void* out, int fp32, cudaStream_t st) {
  const Geometry g = make_geometry(d->N, d->K);
  DecodeParams p{{d->sv_mag[0], d->sv_mag[1]}, d->tensor_scale, d->remap_code};
  const long long total = (long long)g.row_tiles * g.k_chunks * CHUNK_BLOCKS * TILE_ROWS;
  if (fp32)
    dequant_kernel<true><<<grid_for(total, 256), 256, 0, st>>>((const uint8_t*)packed, out, g, p);
  else
    dequant_kernel<false><<<grid_for(total, 256), 256, 0, st>>>((const uint8_t*)packed, out, g, p);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "dequant_kernel launch");
}

int launch_decode_act(const uint8_t* codes, const uint8_t* scales, int M, int K, float sv_mag,
                      void* out, cudaStream_t st) {
  const long long nb = (long long)M * (K / 16);
  decode_act_kernel<<<grid_for(nb, 256), 256, 0, st>>>(codes, scales, (__nv_bfloat16*)out, nb, sv_mag);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "decode_act_kernel launch");
}

}  // namespace razer
