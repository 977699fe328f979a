// Fused cluster path of the MetaSD verify round (one persistent kernel per call).
#include "metasd_device.cuh"

namespace metasd {

bool fused_supported(int, int, int) { return false; }
cudaError_t fused_prepare(int) { return cudaSuccess; }
cudaError_t launch_fused(const VerifyParams &, int, cudaStream_t, uint64_t *) { return cudaErrorNotSupported; }

}  // namespace metasd
