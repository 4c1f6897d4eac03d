// C-ABI entry points of the BDLM attention library: argument checks, parameter
// resolution and dispatch to the kernels.  No allocation, no synchronisation (except
// bdlm_get_device_status), no output on stdout/stderr.
#include <math.h>

#include <atomic>

#include "bdlm_common.cuh"
#include "tc_launch.h"

namespace bdlm {
namespace {

__device__ int g_device_status = 0;
constexpr int kMaxDevices = 64;
unsigned long long* g_trace[kMaxDevices] = {};   // trace buffer of each device ordinal (host-side copy of the pointer)
std::atomic<int> g_sm_count[kMaxDevices] = {};

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_params(const bdlm_params* p, const bdlm_packed_geometry* g = nullptr) {
  if (p == nullptr) return BDLM_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->L <= 0 || p->block_size <= 0 || p->H <= 0 || p->H_kv <= 0) return BDLM_ERR_INVALID_ARG;
  if (p->H % p->H_kv != 0) return BDLM_ERR_INVALID_ARG;
  if (g == nullptr) {
    if (p->L % p->block_size != 0) return BDLM_ERR_INVALID_ARG;
  } else {
    if (g->Lq_clean < 0 || g->clean_q_pos0 < 0 || g->n_blocks < 0) return BDLM_ERR_INVALID_ARG;
    if ((int64_t)g->clean_q_pos0 + g->Lq_clean > p->L) return BDLM_ERR_INVALID_ARG;
    if ((int64_t)g->n_blocks * p->block_size > (int64_t)1 << 30) return BDLM_ERR_INVALID_ARG;
    if (g->block_prefix != nullptr && (reinterpret_cast<uintptr_t>(g->block_prefix) & 3u)) return BDLM_ERR_INVALID_ARG;
    if (g->kv_chunk_len < 0) return BDLM_ERR_INVALID_ARG;
    if (g->kv_chunk_len > 0) {   // clean K/V in gathered order
      if (g->kv_chunk_len % 128 != 0 || p->L % g->kv_chunk_len != 0) return BDLM_ERR_INVALID_ARG;
      if (g->kv_chunk_pos == nullptr || g->kv_pos_chunk == nullptr) return BDLM_ERR_INVALID_ARG;
      if ((reinterpret_cast<uintptr_t>(g->kv_chunk_pos) & 3u) || (reinterpret_cast<uintptr_t>(g->kv_pos_chunk) & 3u)) return BDLM_ERR_INVALID_ARG;
      if (p->window > 0) return BDLM_ERR_UNSUPPORTED;
      if (p->kv_range_set && p->kv_begin % 128 != 0) return BDLM_ERR_UNSUPPORTED;
    }
  }
  if (p->clean_mask_mode != 0 && p->clean_mask_mode != 1) return BDLM_ERR_INVALID_ARG;
  if (p->impl < 0 || p->impl > 2) return BDLM_ERR_INVALID_ARG;
  if (p->bwd_passes < 0 || p->bwd_passes > 7) return BDLM_ERR_INVALID_ARG;
  if (p->bwd_single_pass < 0 || p->bwd_single_pass > 2) return BDLM_ERR_INVALID_ARG;
  if (p->window < 0) return BDLM_ERR_INVALID_ARG;
  if (!(p->scale >= 0.f) || isinf(p->scale)) return BDLM_ERR_INVALID_ARG;
  if (p->kv_range_set) {
    if (p->kv_begin < 0 || p->kv_end < p->kv_begin || p->kv_end > p->L) return BDLM_ERR_INVALID_ARG;
  }
  if ((int64_t)p->batch * 2 > 65535 || p->H > 65535) return BDLM_ERR_INVALID_ARG;
  if (p->d != 64 && p->d != 128) return BDLM_ERR_UNSUPPORTED;
  return BDLM_OK;
}

void fill(KArgs& a, const bdlm_params* p, const bdlm_packed_geometry* g) {
  a.batch = p->batch; a.L = p->L; a.M = p->block_size; a.H = p->H; a.Hkv = p->H_kv;
  a.G = p->H / p->H_kv; a.d = p->d;
  if (g == nullptr) {
    a.Lqc = p->L; a.cq_pos0 = 0; a.Ln = p->L; a.nb = p->L / p->block_size; a.prefix = nullptr;
    a.kv_chunk_len = 0; a.kv_chunk_pos = nullptr; a.kv_pos_chunk = nullptr;
  } else {
    a.kv_chunk_len = g->kv_chunk_len; a.kv_chunk_pos = g->kv_chunk_pos; a.kv_pos_chunk = g->kv_pos_chunk;
    a.Lqc = g->Lq_clean; a.cq_pos0 = g->clean_q_pos0; a.nb = g->n_blocks; a.Ln = g->n_blocks * p->block_size;
    a.prefix = g->block_prefix;
  }
  a.scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf((float)p->d);
  a.scale_log2 = a.scale * LOG2E;
  a.mode = p->clean_mask_mode;
  a.kv_begin = p->kv_range_set ? p->kv_begin : 0;
  a.kv_end = p->kv_range_set ? p->kv_end : p->L;
  a.diag = p->include_noisy_diag ? 1 : 0;
  a.window = p->window;
  for (int s = 0; s < 2; ++s) {
    a.q[s] = a.k[s] = a.v[s] = nullptr; a.o[s] = nullptr; a.lse[s] = nullptr;
    a.dout[s] = nullptr; a.dsum[s] = nullptr; a.dq[s] = a.dk[s] = a.dv[s] = nullptr;
  }
  {
    const int dev = current_device();
    a.trace = dev >= 0 ? g_trace[dev] : nullptr;
  }
  a.single_pass = 0; a.dq32[0] = a.dq32[1] = nullptr; a.dq32_rows[0] = a.dq32_rows[1] = 0;
}

bool is_sm100() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  return major == 10;
}

size_t dsum_bytes(const bdlm_params* p, const bdlm_packed_geometry* g = nullptr) {
  const size_t rows = g == nullptr ? (size_t)p->L
                                   : (size_t)(g->Lq_clean > g->n_blocks * p->block_size ? g->Lq_clean : g->n_blocks * p->block_size);
  size_t one = (size_t)p->batch * p->H * (rows > 0 ? rows : 1) * sizeof(float);
  return (one + 255) / 256 * 256;
}

}  // namespace

int device_sm_count() {
  const int dev = current_device();
  if (dev < 0) return 1;
  int n = g_sm_count[dev].load(std::memory_order_relaxed);
  if (n <= 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 1;
    g_sm_count[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

int* device_status_ptr() {
  int* ptr = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_device_status) != cudaSuccess) return nullptr;
  return ptr;
}

}  // namespace bdlm

using namespace bdlm;

extern "C" {

size_t bdlm_workspace_bytes(const bdlm_params* p, int32_t which) {
  if (check_params(p) != BDLM_OK) return 0;
  if (which == BDLM_WS_BWD)
    return 2 * dsum_bytes(p) + (p->bwd_single_pass != BDLM_BWD_TWO_PASS ? tc_bwd_fused_workspace(p, nullptr) : 0);
  return 0;
}

static int fwd_impl(const bdlm_params* p, const bdlm_packed_geometry* g,
                    const void* q_clean, const void* k_clean, const void* v_clean,
                    const void* q_noisy, const void* k_noisy, const void* v_noisy,
                    void* o_clean, void* o_noisy, float* lse_clean, float* lse_noisy, void* cuda_stream) {
  int rc = check_params(p, g);
  if (rc != BDLM_OK) return rc;
  if (g != nullptr && ((q_clean != nullptr && g->Lq_clean == 0) || (q_noisy != nullptr && g->n_blocks == 0))) return BDLM_ERR_INVALID_ARG;
  if (q_clean == nullptr && q_noisy == nullptr) return BDLM_ERR_INVALID_ARG;
  if (k_clean == nullptr || v_clean == nullptr) return BDLM_ERR_INVALID_ARG;
  if (q_clean != nullptr && (o_clean == nullptr || lse_clean == nullptr)) return BDLM_ERR_INVALID_ARG;
  if (q_noisy != nullptr && (o_noisy == nullptr || lse_noisy == nullptr)) return BDLM_ERR_INVALID_ARG;
  if (q_noisy != nullptr && p->include_noisy_diag && (k_noisy == nullptr || v_noisy == nullptr)) return BDLM_ERR_INVALID_ARG;
  const void* ptrs[] = {q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy, lse_clean, lse_noisy};
  for (const void* x : ptrs) if (!aligned16(x)) return BDLM_ERR_INVALID_ARG;
  if (!is_sm100()) return BDLM_ERR_UNSUPPORTED;

  KArgs a;
  fill(a, p, g);
  using bf = __nv_bfloat16;
  a.q[CLEAN] = (const bf*)q_clean; a.q[NOISY] = (const bf*)q_noisy;
  a.k[CLEAN] = (const bf*)k_clean; a.k[NOISY] = (const bf*)(k_noisy ? k_noisy : k_clean);
  a.v[CLEAN] = (const bf*)v_clean; a.v[NOISY] = (const bf*)(v_noisy ? v_noisy : v_clean);
  a.o[CLEAN] = (bf*)o_clean; a.o[NOISY] = (bf*)o_noisy;
  a.lse[CLEAN] = lse_clean; a.lse[NOISY] = lse_noisy;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  const bool tc_ok = tc_fwd_supported(a);
  if (p->impl == 2 && !tc_ok) return BDLM_ERR_UNSUPPORTED;
  cudaError_t e;
  if (tc_ok && p->impl != 1) e = launch_tc_fwd(a, st);
  else e = launch_portable_fwd(a, st);
  return e == cudaSuccess ? BDLM_OK : BDLM_ERR_CUDA;
}

static int bwd_impl(const bdlm_params* p, const bdlm_packed_geometry* g,
                    const void* q_clean, const void* k_clean, const void* v_clean,
                    const void* q_noisy, const void* k_noisy, const void* v_noisy,
                    const void* o_clean, const void* o_noisy,
                    const float* lse_clean, const float* lse_noisy,
                    const void* do_clean, const void* do_noisy,
                    void* dq_clean, void* dk_clean, void* dv_clean,
                    void* dq_noisy, void* dk_noisy, void* dv_noisy,
                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_params(p, g);
  if (rc != BDLM_OK) return rc;
  // the plain layer needs every tensor; a packed call may leave out one query stream with all that belongs to it
  const bool has_c = (g == nullptr) || q_clean != nullptr;
  const bool has_n = (g == nullptr) || q_noisy != nullptr;
  if (!has_c && !has_n) return BDLM_ERR_INVALID_ARG;
  if (g != nullptr && ((has_c && g->Lq_clean == 0) || (has_n && g->n_blocks == 0))) return BDLM_ERR_INVALID_ARG;
  const void* always[] = {k_clean, v_clean, dk_clean, dv_clean, workspace};
  for (const void* x : always) if (x == nullptr || !aligned16(x)) return BDLM_ERR_INVALID_ARG;
  if (has_c) {
    const void* need[] = {q_clean, o_clean, lse_clean, do_clean, dq_clean};
    for (const void* x : need) if (x == nullptr || !aligned16(x)) return BDLM_ERR_INVALID_ARG;
  }
  if (has_n) {
    const void* need[] = {q_noisy, k_noisy, v_noisy, o_noisy, lse_noisy, do_noisy, dq_noisy, dk_noisy, dv_noisy};
    for (const void* x : need) if (x == nullptr || !aligned16(x)) return BDLM_ERR_INVALID_ARG;
  }
  if (p->kv_range_set && (p->kv_begin != 0 || p->kv_end != p->L)) return BDLM_ERR_UNSUPPORTED;
  if (!p->include_noisy_diag) return BDLM_ERR_UNSUPPORTED;
  // the D rows are always needed; the fp32 dQ accumulators of the fused kernel only when that kernel runs
  const size_t need_min = 2 * dsum_bytes(p, g);
  const size_t need_fused = need_min + tc_bwd_fused_workspace(p, g);
  if (workspace_bytes < (p->bwd_single_pass == BDLM_BWD_FUSED ? need_fused : need_min)) return BDLM_ERR_WORKSPACE_TOO_SMALL;
  if (!is_sm100()) return BDLM_ERR_UNSUPPORTED;

  KArgs a;
  fill(a, p, g);
  using bf = __nv_bfloat16;
  a.q[CLEAN] = has_c ? (const bf*)q_clean : nullptr; a.q[NOISY] = has_n ? (const bf*)q_noisy : nullptr;
  a.k[CLEAN] = (const bf*)k_clean; a.k[NOISY] = has_n ? (const bf*)k_noisy : nullptr;
  a.v[CLEAN] = (const bf*)v_clean; a.v[NOISY] = has_n ? (const bf*)v_noisy : nullptr;
  a.o[CLEAN] = (bf*)const_cast<void*>(o_clean); a.o[NOISY] = (bf*)const_cast<void*>(o_noisy);
  a.lse[CLEAN] = const_cast<float*>(lse_clean); a.lse[NOISY] = const_cast<float*>(lse_noisy);
  a.dout[CLEAN] = (const bf*)do_clean; a.dout[NOISY] = (const bf*)do_noisy;
  float* ds_c = static_cast<float*>(workspace);
  float* ds_n = reinterpret_cast<float*>(static_cast<char*>(workspace) + dsum_bytes(p, g));
  a.dsum[CLEAN] = ds_c; a.dsum[NOISY] = ds_n;
  a.dq[CLEAN] = (bf*)dq_clean; a.dq[NOISY] = (bf*)dq_noisy;
  a.dk[CLEAN] = (bf*)dk_clean; a.dk[NOISY] = has_n ? (bf*)dk_noisy : nullptr;
  a.dv[CLEAN] = (bf*)dv_clean; a.dv[NOISY] = has_n ? (bf*)dv_noisy : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  const bool tc_ok = tc_bwd_supported(a);
  if (p->impl == 2 && !tc_ok) return BDLM_ERR_UNSUPPORTED;
  // automatic: the fused kernel whenever the tensor-core kernels take the shape and the workspace has room for its
  // fp32 dQ accumulators; the two-pass path otherwise (and always when it is asked for)
  a.single_pass = (p->bwd_single_pass != BDLM_BWD_TWO_PASS && tc_ok && p->impl != 1 && need_fused > need_min &&
                   workspace_bytes >= need_fused) ? 1 : 0;
  const int passes = p->bwd_passes ? p->bwd_passes : 7;
  cudaError_t e = cudaSuccess;
  if (passes & BDLM_BWD_PASS_DSUM) e = launch_dsum(a, ds_c, ds_n, st);
  if (e != cudaSuccess) return BDLM_ERR_CUDA;
  if (tc_ok && p->impl != 1) {
    void* extra = static_cast<char*>(workspace) + 2 * dsum_bytes(p, g);
    e = launch_tc_bwd(a, extra, passes, st);
  } else {
    e = launch_portable_bwd(a, passes, st);
  }
  return e == cudaSuccess ? BDLM_OK : BDLM_ERR_CUDA;
}

int bdlm_attn_fwd(const bdlm_params* p,
                  const void* q_clean, const void* k_clean, const void* v_clean,
                  const void* q_noisy, const void* k_noisy, const void* v_noisy,
                  void* o_clean, void* o_noisy, float* lse_clean, float* lse_noisy,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  (void)workspace; (void)workspace_bytes;
  return fwd_impl(p, nullptr, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy,
                  lse_clean, lse_noisy, cuda_stream);
}

int bdlm_attn_fwd_packed(const bdlm_params* p, const bdlm_packed_geometry* g,
                         const void* q_clean, const void* k_clean, const void* v_clean,
                         const void* q_noisy, const void* k_noisy, const void* v_noisy,
                         void* o_clean, void* o_noisy, float* lse_clean, float* lse_noisy,
                         void* cuda_stream) {
  if (g == nullptr) return BDLM_ERR_INVALID_ARG;
  return fwd_impl(p, g, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy,
                  lse_clean, lse_noisy, cuda_stream);
}

int bdlm_attn_bwd(const bdlm_params* p,
                  const void* q_clean, const void* k_clean, const void* v_clean,
                  const void* q_noisy, const void* k_noisy, const void* v_noisy,
                  const void* o_clean, const void* o_noisy,
                  const float* lse_clean, const float* lse_noisy,
                  const void* do_clean, const void* do_noisy,
                  void* dq_clean, void* dk_clean, void* dv_clean,
                  void* dq_noisy, void* dk_noisy, void* dv_noisy,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return bwd_impl(p, nullptr, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy, lse_clean,
                  lse_noisy, do_clean, do_noisy, dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy,
                  workspace, workspace_bytes, cuda_stream);
}

int bdlm_attn_bwd_packed(const bdlm_params* p, const bdlm_packed_geometry* g,
                         const void* q_clean, const void* k_clean, const void* v_clean,
                         const void* q_noisy, const void* k_noisy, const void* v_noisy,
                         const void* o_clean, const void* o_noisy,
                         const float* lse_clean, const float* lse_noisy,
                         const void* do_clean, const void* do_noisy,
                         void* dq_clean, void* dk_clean, void* dv_clean,
                         void* dq_noisy, void* dk_noisy, void* dv_noisy,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (g == nullptr) return BDLM_ERR_INVALID_ARG;
  return bwd_impl(p, g, q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, o_noisy, lse_clean,
                  lse_noisy, do_clean, do_noisy, dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy,
                  workspace, workspace_bytes, cuda_stream);
}

size_t bdlm_workspace_bytes_packed(const bdlm_params* p, const bdlm_packed_geometry* g, int32_t which) {
  if (g == nullptr || check_params(p, g) != BDLM_OK) return 0;
  if (which == BDLM_WS_BWD)
    return 2 * dsum_bytes(p, g) + (p->bwd_single_pass != BDLM_BWD_TWO_PASS ? tc_bwd_fused_workspace(p, g) : 0);
  return 0;
}

int bdlm_lse_merge(int32_t n_partials, int32_t batch, int32_t L, int32_t H, int32_t d,
                   const void* const* o_partials, const float* const* lse_partials,
                   int32_t partial_dtype, void* o_out, float* lse_out, void* cuda_stream) {
  if (n_partials < 1 || n_partials > 16 || batch <= 0 || L <= 0 || H <= 0 || d <= 0 || d % 8 != 0) return BDLM_ERR_INVALID_ARG;
  if (partial_dtype != 0 && partial_dtype != 1) return BDLM_ERR_INVALID_ARG;
  if (o_partials == nullptr || lse_partials == nullptr || o_out == nullptr || lse_out == nullptr) return BDLM_ERR_INVALID_ARG;
  if (!aligned16(o_out) || !aligned16(lse_out)) return BDLM_ERR_INVALID_ARG;
  for (int j = 0; j < n_partials; ++j) {
    if (o_partials[j] == nullptr || lse_partials[j] == nullptr) return BDLM_ERR_INVALID_ARG;
    if (!aligned16(o_partials[j]) || !aligned16(lse_partials[j])) return BDLM_ERR_INVALID_ARG;
    if (lse_partials[j] == lse_out) return BDLM_ERR_INVALID_ARG;   // threads of a row re-read the LSEs
  }
  cudaError_t e = launch_merge(n_partials, batch, L, H, d, o_partials, lse_partials, partial_dtype,
                               o_out, lse_out, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? BDLM_OK : BDLM_ERR_CUDA;
}

int bdlm_set_trace_buffer(void* device_counters, size_t bytes) {
  if (device_counters != nullptr && (bytes < BDLM_TRACE_SLOTS * sizeof(unsigned long long) || !aligned16(device_counters)))
    return BDLM_ERR_INVALID_ARG;
  const int dev = current_device();
  if (dev < 0) return BDLM_ERR_CUDA;
  g_trace[dev] = static_cast<unsigned long long*>(device_counters);
  return BDLM_OK;
}

const char* bdlm_status_string(int status) {
  switch (status) {
    case BDLM_OK: return "BDLM_OK";
    case BDLM_ERR_INVALID_ARG: return "BDLM_ERR_INVALID_ARG";
    case BDLM_ERR_UNSUPPORTED: return "BDLM_ERR_UNSUPPORTED";
    case BDLM_ERR_WORKSPACE_TOO_SMALL: return "BDLM_ERR_WORKSPACE_TOO_SMALL";
    case BDLM_ERR_CUDA: return "BDLM_ERR_CUDA";
    case BDLM_ERR_DEVICE_TIMEOUT: return "BDLM_ERR_DEVICE_TIMEOUT";
    case BDLM_ERR_STATIC_SCRATCH_TOO_SMALL: return "BDLM_ERR_STATIC_SCRATCH_TOO_SMALL";
    default: return "BDLM_ERR_UNKNOWN";
  }
}

int bdlm_get_device_status(void* cuda_stream) {
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return BDLM_ERR_CUDA;
  int* ptr = device_status_ptr();
  if (ptr == nullptr) return BDLM_ERR_CUDA;
  int host = 0;
  if (cudaMemcpy(&host, ptr, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return BDLM_ERR_CUDA;
  if (host != 0) {
    int zero = 0;
    if (cudaMemcpy(ptr, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return BDLM_ERR_CUDA;
    return BDLM_ERR_DEVICE_TIMEOUT;
  }
  return BDLM_OK;
}

}  // extern "C"
