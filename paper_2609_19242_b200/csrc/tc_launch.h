// Host-side interface of the tcgen05 (5th-generation tensor core) kernels.
#pragma once
#include <cuda.h>

#include "bdlm_common.cuh"

namespace bdlm {

// Address of the device status word that bounded waits report to (nullptr on failure).
int* device_status_ptr();

bool tc_encoder_available();
// Tensor map over a [batch, L, heads, d] bf16 tensor (d = 64 or 128), box = 64 columns x `rows` rows, 128-byte swizzle.
bool tc_make_map(CUtensorMap* m, const void* ptr, int heads, int L, int batch, int rows, int d);

// Tensor map over a row-major bf16 matrix [rows, cols] with leading dimension ld (elements): box = 64 columns x
// `box_rows` rows, 128-byte swizzle, zero fill outside the matrix.
bool tc_make_map_2d(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows);

bool tc_rows_ok(const KArgs& a);
bool tc_fwd_supported(const KArgs& a);
bool tc_bwd_supported(const KArgs& a);
// Bytes of the fused backward's fp32 dQ accumulators for these sizes (0 when the fused kernel cannot take them).
size_t tc_bwd_fused_workspace(const bdlm_params* p, const bdlm_packed_geometry* g);
cudaError_t launch_tc_fwd(const KArgs& a, cudaStream_t st);
cudaError_t launch_tc_bwd(const KArgs& a, void* extra_ws, int passes, cudaStream_t st);

}  // namespace bdlm
