// Whole-chain persistent kernel for small float mixtures (placeholder until the kernel lands).
#include "sds_device.cuh"
#include "sds_internal.h"

namespace sds {

bool fused_small_supported(int, int, int) { return false; }
cudaError_t launch_fused_small(const WinArgs&, const GmmArgs&, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace sds
