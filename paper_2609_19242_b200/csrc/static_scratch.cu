// bdlm_attn_bwd_static_scratch: the backward pass for callers that may not allocate.
//
// The regular backward needs a caller-provided workspace for D_i = sum_d dO_i,d * O_i,d.  Some
// callers cannot supply one: a plug-in running inside a host framework whose pool already owns
// all device memory, or a latency-critical loop in which the device-wide synchronisation that
// cudaMalloc/cudaFree imply is not acceptable.  For them the scratch lives in a fixed device
// array that is part of the library image; this entry point hands its address to the same
// kernels the regular backward launches.  It never calls cudaMalloc, cudaFree or any other
// allocating routine.
#include <mutex>

#include "bdlm_common.cuh"

namespace {

// 2 streams x BDLM_STATIC_SCRATCH_ROWS floats.  Every GPU that loads the library holds these
// 8 MiB until the process exits.
static __device__ __align__(256) float g_static_dsum[2 * BDLM_STATIC_SCRATCH_ROWS];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_dsum, per device
std::mutex g_scratch_mutex;

// The array's name is only a host-side handle; kernels need the device address, which differs
// per device.  Looked up once per device, with that device current, and remembered per device
// ordinal: the address belongs to the device's primary context and goes stale if that context is
// torn down (cudaDeviceReset) -- the library has to be reloaded then.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BDLM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_dsum) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return BDLM_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return BDLM_OK;
}

}  // namespace

extern "C" int bdlm_attn_bwd_static_scratch(const bdlm_params* p,
                                            const void* q_clean, const void* k_clean, const void* v_clean,
                                            const void* q_noisy, const void* k_noisy, const void* v_noisy,
                                            const void* o_clean, const void* o_noisy,
                                            const float* lse_clean, const float* lse_noisy,
                                            const void* do_clean, const void* do_noisy,
                                            void* dq_clean, void* dk_clean, void* dv_clean,
                                            void* dq_noisy, void* dk_noisy, void* dv_noisy,
                                            void* cuda_stream) {
  if (p == nullptr) return BDLM_ERR_INVALID_ARG;
  // Always the two-pass kernels: they need only the D rows.  (The fused kernel's fp32 dQ accumulators take 512 bytes
  // per query row and head; no fixed array of a sensible size could hold them.)
  bdlm_params q = *p;
  q.bwd_single_pass = BDLM_BWD_TWO_PASS;
  const size_t need = bdlm_workspace_bytes(&q, BDLM_WS_BWD);
  if (need == 0)   // invalid or unsupported parameters: the regular entry point's checks say which, before they touch anything
    return bdlm_attn_bwd(&q, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy, lse_clean,
                         lse_noisy, do_clean, do_noisy, dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy,
                         nullptr, 0, cuda_stream);
  const size_t have = sizeof(float) * 2 * (size_t)BDLM_STATIC_SCRATCH_ROWS;
  if ((int64_t)q.batch * q.H * q.L > (int64_t)BDLM_STATIC_SCRATCH_ROWS || need > have)
    return BDLM_ERR_STATIC_SCRATCH_TOO_SMALL;
  float* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != BDLM_OK) return rc;
  // D is rewritten in full by every call before it is read, so nothing has to be cleared.
  return bdlm_attn_bwd(&q, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy,
                       lse_clean, lse_noisy, do_clean, do_noisy, dq_clean, dk_clean, dv_clean,
                       dq_noisy, dk_noisy, dv_noisy, scratch, have, cuda_stream);
}
