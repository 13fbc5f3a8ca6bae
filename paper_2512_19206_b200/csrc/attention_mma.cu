// placeholder until the tensor-core kernel lands: routes to the plain-ALU kernel
#include "common.cuh"
namespace mixkvq {
cudaError_t attention_mma_setup() { return cudaSuccess; }
cudaError_t launch_attention_mma(const LayerView& lv, const void* q, float* out, float scale, float* ws, int n_sms,
                                 cudaStream_t stream, int* launches) {
  return launch_attention_simt(lv, q, out, scale, ws, n_sms, stream, launches);
}
}  // namespace mixkvq
