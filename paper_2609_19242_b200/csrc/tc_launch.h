// Host-side interface of the tcgen05 (5th-generation tensor core) kernels.
#pragma once
#include "bdlm_common.cuh"

namespace bdlm {

// Address of the device status word that bounded waits report to (nullptr on failure).
int* device_status_ptr();

bool tc_fwd_supported(const KArgs& a);
bool tc_bwd_supported(const KArgs& a);
size_t tc_bwd_extra_workspace(const bdlm_params* p);
cudaError_t launch_tc_fwd(const KArgs& a, cudaStream_t st);
cudaError_t launch_tc_bwd(const KArgs& a, void* extra_ws, int passes, cudaStream_t st);

}  // namespace bdlm
