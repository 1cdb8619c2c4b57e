// Tensor-core decode kernel (placeholder until the kernel lands).
#include "xq_internal.h"
namespace xq {
bool decode_mma_supported(const Dims&, int, int) { return false; }
cudaError_t launch_decode_mma(const DecodeParams&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace xq
