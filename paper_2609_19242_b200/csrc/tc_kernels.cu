// tcgen05 kernels (placeholder until the tensor-memory path lands: reports "unsupported",
// so every call takes the portable kernels).
#include "tc_launch.h"

namespace bdlm {
bool tc_fwd_supported(const KArgs&) { return false; }
bool tc_bwd_supported(const KArgs&) { return false; }
size_t tc_bwd_extra_workspace(const bdlm_params*) { return 0; }
cudaError_t launch_tc_fwd(const KArgs&, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_tc_bwd(const KArgs&, void*, int, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace bdlm
