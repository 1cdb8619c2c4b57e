// placeholder while the layouts change: no tensor-core kernel
#include "xq_internal.h"
namespace xq {
bool decode_mma_supported(const Dims&, int, int) { return false; }
int decode_mma_ctas_per_sm(const Dims&, int, int) { return 0; }
cudaError_t launch_decode_mma(const DecodeParams&, cudaStream_t) { return cudaErrorInvalidValue; }
}  // namespace xq
