// razer_gemv_static: the decode GEMV for callers that cannot allocate device memory.
//
// The tensor-core matmul kernel needs scratch in global memory (a status word, per-tile
// arrival counters and per-CTA FP32 partial tiles for the stripe reduction).  The other
// entry points take that scratch from the caller.  This one keeps it in a fixed array that
// is part of the library image, so a caller that is not allowed to call cudaMalloc, or that
// runs where the allocator may not be entered, can still run the GEMV: it passes only
// inputs and outputs.
#include <mutex>

#include "razer_common.cuh"

namespace razer {

int launch_gemm_umma(const razer_desc*, const void* packed, const void* x, int M, int ldx_K, float extra_scale,
                     const float* extra_scale_dev, void* y, void* ws, size_t ws_bytes, cudaStream_t);
size_t umma_workspace_bytes(const razer_desc*, int M);
size_t umma_workspace_zero_bytes(const razer_desc*, int M);

// Every GPU that loads the library holds this array until the process exits.
constexpr size_t STATIC_SCRATCH_BYTES = 4u << 20;
constexpr int STATIC_MAX_M = 16;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address;
// the address a kernel can use comes from cudaGetSymbolAddress, once per device.
constexpr int MAX_DEVICES = 64;
static void* g_scratch_ptr[MAX_DEVICES] = {};
static std::mutex g_scratch_mutex;

static int static_scratch(void** out) {
  int dev = -1;
  RAZER_TRY(check_cuda(cudaGetDevice(&dev), "cudaGetDevice"));
  if (dev < 0 || dev >= MAX_DEVICES) return set_error(RAZER_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    RAZER_TRY(check_cuda(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)"));
    if (!p) return set_error(RAZER_ERR_CUDA, "the static scratch array has no device address");
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return RAZER_OK;
}

}  // namespace razer

using namespace razer;

extern "C" int razer_gemv_static(const razer_desc* d, const void* packed_dev, const void* x_dev, int M,
                                 void* y_dev, void* stream) {
  RAZER_TRY(check_desc(d));
  if (M < 1 || M > STATIC_MAX_M)
    return set_error(RAZER_ERR_INVALID_ARG, "razer_gemv_static takes 1 <= M <= %d (got %d)", STATIC_MAX_M, M);
  if (!packed_dev || !x_dev || !y_dev) return set_error(RAZER_ERR_INVALID_ARG, "a device pointer is NULL");
  if (reinterpret_cast<uintptr_t>(packed_dev) % 16 || reinterpret_cast<uintptr_t>(x_dev) % 16 ||
      reinterpret_cast<uintptr_t>(y_dev) % 2)
    return set_error(RAZER_ERR_INVALID_ARG, "packed_dev and x_dev must be 16-byte aligned, y_dev 2-byte aligned");
  const size_t need = umma_workspace_bytes(d, M);
  const size_t zeroed = umma_workspace_zero_bytes(d, M);   // status word + arrival counters
  if (need > STATIC_SCRATCH_BYTES || zeroed > need)
    return set_error(RAZER_ERR_UNSUPPORTED,
                     "this shape needs %zu bytes of scratch; the built-in array holds %zu (use razer_gemv with a "
                     "caller-owned workspace)", need, (size_t)STATIC_SCRATCH_BYTES);
  void* scratch = nullptr;
  RAZER_TRY(static_scratch(&scratch));
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the previous call left: the status word and the counters must start at zero.
  RAZER_TRY(check_cuda(cudaMemsetAsync(scratch, 0, zeroed, st), "static scratch clear"));
  return launch_gemm_umma(d, packed_dev, x_dev, M, d->K, 1.0f, nullptr, y_dev, scratch, STATIC_SCRATCH_BYTES, st);
}
