// CUDA-core matmul against packed RaZeR weights (Sec. 4.3: the paper's "CUDA-core variant"
// for GEMV workloads).  thread = weight row: each thread walks its row's blocks along K,
// decodes 16 elements, multiplies by the activations staged in shared memory as FP32 and
// keeps one FP32 accumulator per token.  No cross-lane reduction is needed; K can be split
// across CTAs, whose partial sums a second kernel adds in a fixed order.
#include "razer_common.cuh"

namespace razer {

constexpr int SIMT_GROUP_CHUNKS = 4;                       // 256 columns of x staged at a time
constexpr int SIMT_GROUP_K = SIMT_GROUP_CHUNKS * CHUNK_K;

template <int MT>
__global__ void __launch_bounds__(TILE_ROWS)
gemv_simt_kernel(const uint8_t* __restrict__ packed, const __nv_bfloat16* __restrict__ x,
                 __nv_bfloat16* __restrict__ y, float* __restrict__ partial, Geometry g,
                 DecodeParams p, const float* __restrict__ extra_scale, int M, int chunks_per_split,
                 int n_splits) {
  __shared__ float xs[MT][SIMT_GROUP_K];
  const int rt = blockIdx.x, split = blockIdx.y, m0 = blockIdx.z * MT;
  const int row_in = threadIdx.x;
  const int c_begin = split * chunks_per_split;
  const int c_end = min(g.k_chunks, c_begin + chunks_per_split);
  const float sv0 = p.sv_mag[0], sv1 = p.sv_mag[1];
  float acc[MT];
#pragma unroll
  for (int m = 0; m < MT; ++m) acc[m] = 0.0f;

  for (int cg = c_begin; cg < c_end; cg += SIMT_GROUP_CHUNKS) {
    __syncthreads();
    for (int i = threadIdx.x; i < MT * SIMT_GROUP_K; i += TILE_ROWS) {
      const int m = i / SIMT_GROUP_K, kk = i % SIMT_GROUP_K;
      const int k = cg * CHUNK_K + kk;
      float v = 0.0f;
      if (m0 + m < M && k < g.K) v = __bfloat162float(x[(size_t)(m0 + m) * g.K + k]);
      xs[m][kk] = v;
    }
    __syncthreads();
    const int c_lim = min(c_end, cg + SIMT_GROUP_CHUNKS);
    for (int c = cg; c < c_lim; ++c) {
      const uint8_t* base = packed + piece_offset(g, rt * TILE_ROWS + row_in, c);
      const int r = row_in % STRIP_ROWS;
#pragma unroll
      for (int blk = 0; blk < CHUNK_BLOCKS; ++blk) {
        const uint2 cw = *reinterpret_cast<const uint2*>(base + piece_code_offset(blk, r));
        const uint32_t sb = base[piece_scale_offset(blk, r)];
        float s = scale_value(sb & 0x3Fu);
        if (sb & PACKED_NEGATE) s = -s;
        const float sv = (sb & PACKED_SELECT) ? sv1 : sv0;
        float part[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) part[m] = 0.0f;
        const int kk0 = (c - cg) * CHUNK_K + blk * 16;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float q = packed_elem(packed_nibble(cw, j), sv);
#pragma unroll
          for (int m = 0; m < MT; ++m) part[m] = fmaf(q, xs[m][kk0 + j], part[m]);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = fmaf(s, part[m], acc[m]);
      }
    }
  }
  const int n = rt * TILE_ROWS + row_in;
  if (n >= g.N) return;
#pragma unroll
  for (int m = 0; m < MT; ++m) {
    if (m0 + m >= M) break;
    if (n_splits == 1) {
      const float ts = extra_scale ? p.tensor_scale * *extra_scale : p.tensor_scale;
      y[(size_t)(m0 + m) * g.N + n] = __float2bfloat16_rn(ts * acc[m]);
    } else {
      partial[((size_t)split * M + (m0 + m)) * g.N + n] = acc[m];
    }
  }
}

// Sum the split-K partials in ascending split order, apply the tensor scale, round once.
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, __nv_bfloat16* __restrict__ y,
                                     long long mn, int n_splits, float tensor_scale,
                                     const float* __restrict__ extra_scale) {
  if (extra_scale) tensor_scale *= *extra_scale;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < mn;
       i += (long long)gridDim.x * blockDim.x) {
    float a = 0.0f;
    for (int s = 0; s < n_splits; ++s) a += partial[(size_t)s * mn + i];
    y[i] = __float2bfloat16_rn(tensor_scale * a);
  }
}

// Split-K choice for the CUDA-core kernel: enough CTAs for about two waves of the 148 SMs,
// each split at least one staged group long.
int simt_splits(const Geometry& g, int M, int MT) {
  const int mz = (M + MT - 1) / MT;
  const long long base = (long long)g.row_tiles * mz;
  int want = (int)((2 * 148 + base - 1) / base);
  const int max_splits = (g.k_chunks + SIMT_GROUP_CHUNKS - 1) / SIMT_GROUP_CHUNKS;
  if (want > max_splits) want = max_splits;
  if (want < 1) want = 1;
  return want;
}

size_t simt_workspace_bytes(const razer_desc* d, int M) {
  const Geometry g = make_geometry(d->N, d->K);
  const int MT = M >= 8 ? 8 : (M >= 4 ? 4 : (M >= 2 ? 2 : 1));
  const int s = simt_splits(g, M, MT);
  // the first 256 bytes of every workspace hold the device status word
  return 256 + (s > 1 ? (size_t)s * M * d->N * sizeof(float) : 0);
}

int launch_gemv_simt(const razer_desc* d, const void* packed, const void* x, int M,
                     const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t st) {
  const Geometry g = make_geometry(d->N, d->K);
  DecodeParams p{{d->sv_mag[0], d->sv_mag[1]}, d->tensor_scale, d->remap_code};
  const int MT = M >= 8 ? 8 : (M >= 4 ? 4 : (M >= 2 ? 2 : 1));
  const int splits = simt_splits(g, M, MT);
  int cps = (g.k_chunks + splits - 1) / splits;
  cps = (cps + SIMT_GROUP_CHUNKS - 1) / SIMT_GROUP_CHUNKS * SIMT_GROUP_CHUNKS;
  const int n_splits = (g.k_chunks + cps - 1) / cps;
  const size_t need = n_splits > 1 ? 256 + (size_t)n_splits * M * d->N * sizeof(float) : 0;
  float* partial = ws ? reinterpret_cast<float*>(static_cast<char*>(ws) + 256) : nullptr;
  if (need > ws_bytes || (need && !ws))
    return set_error(RAZER_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  dim3 grid(g.row_tiles, n_splits, (M + MT - 1) / MT);
  if (grid.z > 65535) return set_error(RAZER_ERR_UNSUPPORTED, "M too large for the CUDA-core kernel");
#define RAZER_LAUNCH_SIMT(MT_)                                                                      \
  gemv_simt_kernel<MT_><<<grid, TILE_ROWS, 0, st>>>((const uint8_t*)packed, (const __nv_bfloat16*)x, \
                                                    (__nv_bfloat16*)y, partial, g, p, extra_scale_dev, M, cps,  \
                                                    n_splits)
  switch (MT) {
    case 8: RAZER_LAUNCH_SIMT(8); break;
    case 4: RAZER_LAUNCH_SIMT(4); break;
    case 2: RAZER_LAUNCH_SIMT(2); break;
    default: RAZER_LAUNCH_SIMT(1); break;
  }
#undef RAZER_LAUNCH_SIMT
  count_launches(1);
  RAZER_TRY(check_cuda(cudaGetLastError(), "gemv_simt_kernel launch"));
  if (n_splits > 1) {
    const long long mn = (long long)M * d->N;
    long long b = (mn + 255) / 256;
    if (b > 148 * 8) b = 148 * 8;
    splitk_reduce_kernel<<<(int)b, 256, 0, st>>>(partial, (__nv_bfloat16*)y, mn, n_splits,
                                                  d->tensor_scale, extra_scale_dev);
    count_launches(1);
    RAZER_TRY(check_cuda(cudaGetLastError(), "splitk_reduce_kernel launch"));
  }
  return RAZER_OK;
}

}  // namespace razer
