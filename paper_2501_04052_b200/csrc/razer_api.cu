// extern "C" entry points of the RaZeR library: argument validation and dispatch only.
#include <cstdarg>
#include <cstdio>
#include <cmath>
#include <atomic>
#include <cstdlib>

#include "razer_common.cuh"

namespace razer {

static thread_local char g_err[512] = "";
static std::atomic<unsigned long long> g_launches{0};

void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

int set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return RAZER_OK;
  return set_error(RAZER_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool sv_allowed(float m) {
  // sums of two FP4 values that are not FP4 values themselves (App. D.3); all have at most
  // four significant bits, so special value x block scale stays exact in bf16
  static const float ok[] = {2.5f, 3.5f, 4.5f, 5.f, 5.5f, 6.5f, 7.f, 7.5f, 8.f, 9.f, 10.f, 12.f};
  for (float v : ok)
    if (m == v) return true;
  return false;
}

int check_desc(const razer_desc* d) {
  if (!d) return set_error(RAZER_ERR_INVALID_ARG, "descriptor is NULL");
  if (d->N < 1 || d->K < 16) return set_error(RAZER_ERR_INVALID_ARG, "N=%d K=%d out of range", d->N, d->K);
  if (d->K % 16) return set_error(RAZER_ERR_INVALID_ARG, "K=%d is not a multiple of 16", d->K);
  if (d->block != 16 && d->block != 32 && d->block != 64 && d->block != 128)
    return set_error(RAZER_ERR_UNSUPPORTED, "block size %d (16, 32, 64 and 128 are built)", d->block);
  if (d->K % d->block) return set_error(RAZER_ERR_INVALID_ARG, "K=%d is not a multiple of the block size %d", d->K, d->block);
  if (d->scale_fmt != RAZER_SCALE_E3M3_META2)
    return set_error(RAZER_ERR_UNSUPPORTED, "weight scale format %d (only E3M3 + 2 metadata bits)", d->scale_fmt);
  if (d->remap_code != 0x8 && d->remap_code != 0x0)
    return set_error(RAZER_ERR_INVALID_ARG, "remap_code 0x%x is not a zero code", d->remap_code);
  for (int i = 0; i < 2; ++i)
    if (!sv_allowed(d->sv_mag[i]))
      return set_error(RAZER_ERR_UNSUPPORTED, "special value magnitude %g is not allowed", d->sv_mag[i]);
  if (!(d->tensor_scale > 0.0f) || !std::isfinite(d->tensor_scale))
    return set_error(RAZER_ERR_INVALID_ARG, "tensor_scale must be positive and finite");
  return RAZER_OK;
}

static int check_ptr(const void* p, size_t align, const char* name) {
  if (!p) return set_error(RAZER_ERR_INVALID_ARG, "%s is NULL", name);
  if (reinterpret_cast<uintptr_t>(p) % align)
    return set_error(RAZER_ERR_INVALID_ARG, "%s is not %zu-byte aligned", name, align);
  return RAZER_OK;
}

// kernels' host launchers (defined next to the kernels)
int launch_pack(const razer_desc*, const uint8_t*, const uint8_t*, void*, cudaStream_t);
int launch_dequant(const razer_desc*, const void*, void*, int, cudaStream_t);
int launch_decode_act(const uint8_t*, const uint8_t*, int, int, float, void*, cudaStream_t);
int launch_quant_weight(const float*, int, int, int, int, float, float, int, const float*, uint32_t*, uint8_t*,
                        uint8_t*, float*, cudaStream_t);
int launch_quant_act(const void*, int, int, float, const float*, uint32_t*, uint8_t*, uint8_t*, float*,
                     cudaStream_t);
int launch_gemv_simt(const razer_desc*, const void*, const void*, int, const float*, void*, void*, size_t,
                     cudaStream_t);
size_t simt_workspace_bytes(const razer_desc*, int M);
int launch_gemm_fp4(const razer_desc*, const void*, const uint8_t*, const uint8_t*, const float*, int, void*, void*, size_t,
                    cudaStream_t);
size_t gemm_fp4_workspace_bytes(const razer_desc*, int M);
int launch_gemm_fp4_prepared(const razer_desc*, const void*, const void*, const float*, int, void*, void*, size_t, cudaStream_t);
int launch_quant_act_fp4(const void*, int, int, const float*, uint32_t*, void*, float*, cudaStream_t);
int launch_gemm_umma(const razer_desc*, const void* packed, const void* x, int M, int ldx_K, float extra_scale,
                     const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t);
size_t umma_workspace_bytes(const razer_desc*, int M);
bool umma_supported(const razer_desc*, int M);
int launch_gemv_stream(const razer_desc*, const void* packed, const void* x, int M, float extra_scale,
                       const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t);
size_t gemv_stream_workspace_bytes(const razer_desc*, int M);
bool gemv_stream_supported(const razer_desc*, int M);

// Kernel choice.  M <= 8 (one group of tokens along the MMA's n) goes to the TMA-fed register-fragment kernel
// (razer_gemv_stream.cu), whose fixed cost per launch is small and whose consumer warps do nothing but decode;
// everything else to the tcgen05 kernel.  RAZER_KERNEL (environment, read once) overrides: "umma" keeps
// everything on the tcgen05 kernel, "stream" is the default choice spelled out, "simt" routes everything to
// the CUDA-core kernel (debugging aid).
static char kernel_override() {
  static const char c = [] {
    const char* e = getenv("RAZER_KERNEL");
    if (!e || !e[0]) return '\0';
    if (e[0] == 's' && e[1] == 'i') return 's';         // simt
    if (e[0] == 's') return 't';                        // stream
    return e[0];                                        // umma
  }();
  return c;
}
static bool use_stream(const razer_desc* d, int M) {
  const char o = kernel_override();
  if (!gemv_stream_supported(d, M)) return false;
  return o == '\0' || o == 't';
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Workspace of a matmul against M tokens: enough for whichever kernel takes the shape.
static size_t matmul_workspace_need(const razer_desc* d, int M) {
  size_t b = simt_workspace_bytes(d, M);
  if (umma_supported(d, M)) b = b > umma_workspace_bytes(d, M) ? b : umma_workspace_bytes(d, M);
  if (gemv_stream_supported(d, M)) b = b > gemv_stream_workspace_bytes(d, M) ? b : gemv_stream_workspace_bytes(d, M);
  return b;
}

}  // namespace razer

using namespace razer;

extern "C" {

const char* razer_last_error(void) { return g_err; }

int razer_version(void) { return 100; }

unsigned long long razer_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int razer_packed_bytes(const razer_desc* d, size_t* bytes_out) {
  RAZER_TRY(check_desc(d));
  if (!bytes_out) return set_error(RAZER_ERR_INVALID_ARG, "bytes_out is NULL");
  *bytes_out = make_geometry(d->N, d->K).packed_bytes();
  return RAZER_OK;
}

int razer_pack_layout(const razer_desc* d, const uint8_t* codes_dev, const uint8_t* scales_dev,
                      void* packed_dev, void* stream) {
  RAZER_TRY(check_desc(d));
  RAZER_TRY(check_ptr(codes_dev, 8, "codes_dev"));
  RAZER_TRY(check_ptr(scales_dev, 1, "scales_dev"));
  RAZER_TRY(check_ptr(packed_dev, 16, "packed_dev"));
  return launch_pack(d, codes_dev, scales_dev, packed_dev, (cudaStream_t)stream);
}

int razer_dequant(const razer_desc* d, const void* packed_dev, void* out_dev, int out_is_fp32, void* stream) {
  RAZER_TRY(check_desc(d));
  RAZER_TRY(check_ptr(packed_dev, 16, "packed_dev"));
  RAZER_TRY(check_ptr(out_dev, out_is_fp32 ? 4 : 2, "out_dev"));
  return launch_dequant(d, packed_dev, out_dev, out_is_fp32 ? 1 : 0, (cudaStream_t)stream);
}

int razer_workspace_bytes(const razer_desc* d, int M, int op, size_t* bytes_out) {
  RAZER_TRY(check_desc(d));
  if (!bytes_out) return set_error(RAZER_ERR_INVALID_ARG, "bytes_out is NULL");
  if (M < 1) return set_error(RAZER_ERR_INVALID_ARG, "M=%d must be positive", M);
  size_t b = 0;
  switch (op) {
    case RAZER_OP_GEMV:
      if (M > 64) return set_error(RAZER_ERR_INVALID_ARG, "razer_gemv takes 1 <= M <= 64 (got %d)", M);
      /* fall through */
    case RAZER_OP_GEMM:
      b = matmul_workspace_need(d, M);
      break;
    case RAZER_OP_GEMM_W4A4: {
      const size_t g = matmul_workspace_need(d, M);
      b = align_up((size_t)M * d->K * 2, 256) + g;                     // decoded activations + the bf16 matmul's own
      const size_t f = gemm_fp4_workspace_bytes(d, M);                 // or the block-scaled FP4 path's
      b = b > f ? b : f;
      break;
    }
    default:
      return set_error(RAZER_ERR_INVALID_ARG, "unknown op %d", op);
  }
  *bytes_out = align_up(b, 256);
  return RAZER_OK;
}

int razer_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream) {
  RAZER_TRY(check_ptr(workspace_dev, 256, "workspace_dev"));
  if (workspace_bytes == 0) return RAZER_OK;
  return check_cuda(cudaMemsetAsync(workspace_dev, 0, workspace_bytes, (cudaStream_t)stream), "workspace memset");
}

int razer_workspace_status(const void* workspace_dev, void* stream) {
  RAZER_TRY(check_ptr(workspace_dev, 256, "workspace_dev"));
  uint32_t st = 0;
  RAZER_TRY(check_cuda(cudaMemcpyAsync(&st, workspace_dev, sizeof(st), cudaMemcpyDeviceToHost, (cudaStream_t)stream),
                       "status copy"));
  RAZER_TRY(check_cuda(cudaStreamSynchronize((cudaStream_t)stream), "stream synchronize"));
  if (st != 0) return set_error(RAZER_ERR_DEVICE_TIMEOUT, "a device-side wait gave up (wait id %u)", st);
  return RAZER_OK;
}

static int matmul_common(const razer_desc* d, const void* packed_dev, const void* x_dev, int M, void* y_dev,
                         void* ws, size_t ws_bytes, float extra_scale, const float* extra_scale_dev,
                         cudaStream_t st) {
  RAZER_TRY(check_ptr(packed_dev, 16, "packed_dev"));
  RAZER_TRY(check_ptr(x_dev, 16, "x_dev"));
  RAZER_TRY(check_ptr(y_dev, 2, "y_dev"));
  if (ws && reinterpret_cast<uintptr_t>(ws) % 256)
    return set_error(RAZER_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
  if (use_stream(d, M))
    return launch_gemv_stream(d, packed_dev, x_dev, M, extra_scale, extra_scale_dev, y_dev, ws, ws_bytes, st);
  if (umma_supported(d, M))
    return launch_gemm_umma(d, packed_dev, x_dev, M, d->K, extra_scale, extra_scale_dev, y_dev, ws, ws_bytes, st);
  razer_desc dd = *d;
  dd.tensor_scale = d->tensor_scale * extra_scale;
  return launch_gemv_simt(&dd, packed_dev, x_dev, M, extra_scale_dev, y_dev, ws, ws_bytes, st);
}

int razer_gemv(const razer_desc* d, const void* packed_dev, const void* x_dev, int M, void* y_dev,
               void* workspace_dev, size_t workspace_bytes, void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1 || M > 64) return set_error(RAZER_ERR_INVALID_ARG, "razer_gemv takes 1 <= M <= 64 (got %d)", M);
  return matmul_common(d, packed_dev, x_dev, M, y_dev, workspace_dev, workspace_bytes, 1.0f, nullptr,
                       (cudaStream_t)stream);
}

int razer_gemm(const razer_desc* d, const void* packed_dev, const void* x_dev, int M, void* y_dev,
               void* workspace_dev, size_t workspace_bytes, void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1) return set_error(RAZER_ERR_INVALID_ARG, "M=%d must be positive", M);
  return matmul_common(d, packed_dev, x_dev, M, y_dev, workspace_dev, workspace_bytes, 1.0f, nullptr,
                       (cudaStream_t)stream);
}

int razer_gemv_host(const razer_desc* d, const void* packed_dev, const void* x_host, int M, void* y_host,
                    void* x_stage_dev, void* y_stage_dev, void* workspace_dev, size_t workspace_bytes,
                    void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1 || M > 64) return set_error(RAZER_ERR_INVALID_ARG, "razer_gemv takes 1 <= M <= 64 (got %d)", M);
  if (!x_host || !y_host) return set_error(RAZER_ERR_INVALID_ARG, "host buffer is NULL");
  RAZER_TRY(check_ptr(x_stage_dev, 16, "x_stage_dev"));
  RAZER_TRY(check_ptr(y_stage_dev, 2, "y_stage_dev"));
  cudaStream_t st = (cudaStream_t)stream;
  // pinned host memory that the device can address takes the kernel's stores directly (no copy back)
  void* y_target = y_stage_dev;
  {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, y_host) == cudaSuccess) {
      if (at.type == cudaMemoryTypeHost && at.devicePointer) y_target = at.devicePointer;
    } else {
      cudaGetLastError();                                    // not a CUDA-known pointer: use the staging buffer
    }
  }
  RAZER_TRY(check_cuda(cudaMemcpyAsync(x_stage_dev, x_host, (size_t)M * d->K * 2, cudaMemcpyHostToDevice, st),
                       "copy of x to the device"));
  RAZER_TRY(matmul_common(d, packed_dev, x_stage_dev, M, y_target, workspace_dev, workspace_bytes, 1.0f,
                          nullptr, st));
  if (y_target == y_stage_dev)
    RAZER_TRY(check_cuda(cudaMemcpyAsync(y_host, y_stage_dev, (size_t)M * d->N * 2, cudaMemcpyDeviceToHost, st),
                         "copy of y to the host"));
  if (workspace_dev) return razer_workspace_status(workspace_dev, stream);   // synchronizes
  return check_cuda(cudaStreamSynchronize(st), "stream synchronize");
}

int razer_quant_act(const void* x_dev, int M, int K, float sv_mag, const float* tensor_scale_in_dev,
                    uint32_t* amax_scratch_dev, uint8_t* act_codes_dev, uint8_t* act_scales_dev,
                    float* tensor_scale_out_dev, void* stream) {
  if (M < 1 || K < 16 || K % 16) return set_error(RAZER_ERR_INVALID_ARG, "M=%d K=%d invalid (K %% 16 == 0)", M, K);
  if (sv_mag != 0.0f && !sv_allowed(sv_mag))                           // 0: no special value (plain NVFP4)
    return set_error(RAZER_ERR_UNSUPPORTED, "special value magnitude %g is not allowed", sv_mag);
  RAZER_TRY(check_ptr(x_dev, 16, "x_dev"));
  RAZER_TRY(check_ptr(act_codes_dev, 8, "act_codes_dev"));
  RAZER_TRY(check_ptr(act_scales_dev, 1, "act_scales_dev"));
  RAZER_TRY(check_ptr(tensor_scale_out_dev, 4, "tensor_scale_out_dev"));
  if (!tensor_scale_in_dev) RAZER_TRY(check_ptr(amax_scratch_dev, 8, "amax_scratch_dev"));
  return launch_quant_act(x_dev, M, K, sv_mag, tensor_scale_in_dev, amax_scratch_dev, act_codes_dev,
                          act_scales_dev, tensor_scale_out_dev, (cudaStream_t)stream);
}

int razer_fp4_act_bytes(int M, int K, size_t* bytes_out) {
  if (!bytes_out) return set_error(RAZER_ERR_INVALID_ARG, "bytes_out is NULL");
  if (M < 1 || K < 16 || K % 16) return set_error(RAZER_ERR_INVALID_ARG, "M=%d K=%d invalid (K %% 16 == 0)", M, K);
  const Fp4ActLayout L = make_fp4_act_layout(M, K);
  *bytes_out = L.codes_bytes + L.sfb_bytes;
  return RAZER_OK;
}

int razer_quant_act_fp4(const void* x_dev, int M, int K, const float* tensor_scale_in_dev, uint32_t* amax_scratch_dev,
                        void* act_fp4_dev, float* tensor_scale_out_dev, void* stream) {
  if (M < 1 || K < 16 || K % 16) return set_error(RAZER_ERR_INVALID_ARG, "M=%d K=%d invalid (K %% 16 == 0)", M, K);
  RAZER_TRY(check_ptr(x_dev, 16, "x_dev"));
  RAZER_TRY(check_ptr(act_fp4_dev, 256, "act_fp4_dev"));
  RAZER_TRY(check_ptr(tensor_scale_out_dev, 4, "tensor_scale_out_dev"));
  if (!tensor_scale_in_dev) RAZER_TRY(check_ptr(amax_scratch_dev, 8, "amax_scratch_dev"));
  return launch_quant_act_fp4(x_dev, M, K, tensor_scale_in_dev, amax_scratch_dev, act_fp4_dev, tensor_scale_out_dev,
                              (cudaStream_t)stream);
}

int razer_gemm_w4a4_fp4(const razer_desc* d, const void* packed_w_dev, const void* act_fp4_dev,
                        const float* act_tensor_scale_dev, int M, void* y_dev, void* workspace_dev, size_t workspace_bytes,
                        void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1) return set_error(RAZER_ERR_INVALID_ARG, "M=%d must be positive", M);
  RAZER_TRY(check_ptr(packed_w_dev, 16, "packed_w_dev"));
  RAZER_TRY(check_ptr(act_fp4_dev, 256, "act_fp4_dev"));
  RAZER_TRY(check_ptr(act_tensor_scale_dev, 4, "act_tensor_scale_dev"));
  RAZER_TRY(check_ptr(y_dev, 2, "y_dev"));
  RAZER_TRY(check_ptr(workspace_dev, 256, "workspace_dev"));
  return launch_gemm_fp4_prepared(d, packed_w_dev, act_fp4_dev, act_tensor_scale_dev, M, y_dev, workspace_dev,
                                  workspace_bytes, (cudaStream_t)stream);
}

int razer_quant_weight(const float* w_dev, int N, int K, int block, int scale_aware, const float sv_mag[2], int remap_code,
                       const float* tensor_scale_in_dev, uint32_t* amax_scratch_dev, uint8_t* codes_dev,
                       uint8_t* scales_dev, float* tensor_scale_out_dev, void* stream) {
  if (block != 16 && block != 32 && block != 64 && block != 128)
    return set_error(RAZER_ERR_UNSUPPORTED, "block size %d (16, 32, 64 and 128 are built)", block);
  if (N < 1 || K < block || K % block)
    return set_error(RAZER_ERR_INVALID_ARG, "N=%d K=%d invalid (K must be a multiple of the block size %d)", N, K, block);
  if (!sv_mag) return set_error(RAZER_ERR_INVALID_ARG, "sv_mag is NULL");
  if (remap_code != 0x8 && remap_code != 0x0)
    return set_error(RAZER_ERR_INVALID_ARG, "remap_code 0x%x is not a zero code", remap_code);
  for (int i = 0; i < 2; ++i)
    if (!sv_allowed(sv_mag[i]))
      return set_error(RAZER_ERR_UNSUPPORTED, "special value magnitude %g is not allowed", sv_mag[i]);
  RAZER_TRY(check_ptr(w_dev, 16, "w_dev"));
  RAZER_TRY(check_ptr(codes_dev, 8, "codes_dev"));
  RAZER_TRY(check_ptr(scales_dev, 1, "scales_dev"));
  RAZER_TRY(check_ptr(tensor_scale_out_dev, 4, "tensor_scale_out_dev"));
  if (!tensor_scale_in_dev) RAZER_TRY(check_ptr(amax_scratch_dev, 4, "amax_scratch_dev"));
  return launch_quant_weight(w_dev, N, K, block, scale_aware != 0, sv_mag[0], sv_mag[1], remap_code, tensor_scale_in_dev, amax_scratch_dev,
                             codes_dev, scales_dev, tensor_scale_out_dev, (cudaStream_t)stream);
}

int razer_decode_act(const uint8_t* act_codes_dev, const uint8_t* act_scales_dev, int M, int K, float sv_mag,
                     void* out_bf16_dev, void* stream) {
  if (M < 1 || K < 16 || K % 16) return set_error(RAZER_ERR_INVALID_ARG, "M=%d K=%d invalid (K %% 16 == 0)", M, K);
  if (!sv_allowed(sv_mag)) return set_error(RAZER_ERR_UNSUPPORTED, "special value magnitude %g is not allowed", sv_mag);
  RAZER_TRY(check_ptr(act_codes_dev, 8, "act_codes_dev"));
  RAZER_TRY(check_ptr(act_scales_dev, 1, "act_scales_dev"));
  RAZER_TRY(check_ptr(out_bf16_dev, 16, "out_bf16_dev"));
  return launch_decode_act(act_codes_dev, act_scales_dev, M, K, sv_mag, out_bf16_dev, (cudaStream_t)stream);
}

int razer_gemm_w4a4(const razer_desc* d, const void* packed_w_dev, const uint8_t* act_codes_dev,
                    const uint8_t* act_scales_dev, const float* act_tensor_scale_dev, float act_sv_mag, int M,
                    void* y_dev, void* workspace_dev, size_t workspace_bytes, int use_native_fp4, void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1) return set_error(RAZER_ERR_INVALID_ARG, "M=%d must be positive", M);
  RAZER_TRY(check_ptr(act_tensor_scale_dev, 4, "act_tensor_scale_dev"));
  RAZER_TRY(check_ptr(workspace_dev, 256, "workspace_dev"));
  if (use_native_fp4) {
    RAZER_TRY(check_ptr(packed_w_dev, 16, "packed_w_dev"));
    RAZER_TRY(check_ptr(act_codes_dev, 8, "act_codes_dev"));
    RAZER_TRY(check_ptr(act_scales_dev, 1, "act_scales_dev"));
    RAZER_TRY(check_ptr(y_dev, 2, "y_dev"));
    return launch_gemm_fp4(d, packed_w_dev, act_codes_dev, act_scales_dev, act_tensor_scale_dev, M, y_dev, workspace_dev,
                           workspace_bytes, (cudaStream_t)stream);
  }
  const size_t act_bytes = align_up((size_t)M * d->K * 2, 256);
  if (workspace_bytes < act_bytes) return set_error(RAZER_ERR_WORKSPACE, "workspace too small for the decoded activations");
  cudaStream_t st = (cudaStream_t)stream;
  RAZER_TRY(razer_decode_act(act_codes_dev, act_scales_dev, M, d->K, act_sv_mag, workspace_dev, stream));
  return matmul_common(d, packed_w_dev, workspace_dev, M, y_dev, (char*)workspace_dev + act_bytes,
                       workspace_bytes - act_bytes, 1.0f, act_tensor_scale_dev, st);
}

}  // extern "C"
