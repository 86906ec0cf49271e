// Tensor-core (tcgen05 / TMEM) matmul against packed RaZeR weights.  Placeholder until the
// kernel lands: reports every shape as unsupported so the CUDA-core kernel is used.
#include "razer_common.cuh"

namespace razer {

bool umma_supported(const razer_desc*, int) { return false; }
size_t umma_workspace_bytes(const razer_desc*, int) { return 0; }
int launch_gemm_umma(const razer_desc*, const void*, const void*, int, int, float, const float*, void*, void*,
                     size_t, cudaStream_t) {
  return set_error(RAZER_ERR_UNSUPPORTED, "tensor-core kernel not built");
}

}  // namespace razer
