// Shared device-side definitions for the BDLM attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bdlm_attn.h"

namespace bdlm {

constexpr int CLEAN = 0;
constexpr int NOISY = 1;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// Kernel-side copy of the call: sizes, the resolved clean-key range, pointers per stream.
struct KArgs {
  int batch, L, M, H, Hkv, G, d;
  float scale;        // q.k multiplier (1/sqrt(d) by default)
  float scale_log2;   // scale * log2(e): scores are exponentiated with exp2
  int mode;           // clean_mask_mode
  int kv_begin, kv_end;
  int diag;           // include_noisy_diag
  int window;         // sliding window over clean keys (0 = none)
  const __nv_bfloat16* q[2];
  const __nv_bfloat16* k[2];
  const __nv_bfloat16* v[2];
  __nv_bfloat16* o[2];
  float* lse[2];
  // backward only
  const __nv_bfloat16* dout[2];
  const float* dsum[2];   // D_i = sum_d dO*O, [batch, H, L]
  __nv_bfloat16* dq[2];
  __nv_bfloat16* dk[2];
  __nv_bfloat16* dv[2];
  unsigned long long* trace;   // optional cycle counters (bdlm_set_trace_buffer), else nullptr
  int single_pass;             // backward: dQ accumulated in the dK/dV kernel through fp32 atomics
  float* dq32[2];              // fp32 dQ accumulators [batch, L, H, d] (single-pass backward), else nullptr
};

// Visible key interval [lo, hi) of query row i (stream qs) inside key stream ks
// (section 3.2: clean row -> clean keys 0..i; noisy row -> clean keys of earlier blocks and
// the noisy keys of its own block).  Every row's visible set per key stream is one interval.
__device__ __forceinline__ void visible_interval(int qs, int ks, int i, int M, int mode,
                                                 int kv_begin, int kv_end, int diag,
                                                 int& lo, int& hi, int window) {
  // sliding-window layers: a clean key j is visible to position i only if i - j < window (0 = no window)
  if (ks == CLEAN && window > 0) kv_begin = max(kv_begin, i - window + 1);
  if (qs == CLEAN) {
    if (ks == CLEAN) {
      lo = kv_begin;
      int lim = (mode == 0) ? (i + 1) : ((i / M + 1) * M);
      hi = min(kv_end, lim);
    } else {
      lo = 0; hi = 0;
    }
  } else {
    if (ks == CLEAN) {
      lo = kv_begin;
      hi = min(kv_end, (i / M) * M);
    } else {
      lo = diag ? (i / M) * M : 0;
      hi = diag ? lo + M : 0;
    }
  }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Launchers (host).  Each enqueues on `st` and returns the launch's cudaError_t.
cudaError_t launch_portable_fwd(const KArgs& a, cudaStream_t st);
cudaError_t launch_portable_bwd(const KArgs& a, int passes, cudaStream_t st);
cudaError_t launch_dsum(const KArgs& a, float* dsum_clean, float* dsum_noisy, cudaStream_t st);
cudaError_t launch_merge(int n, int batch, int L, int H, int d, const void* const* o_parts,
                         const float* const* lse_parts, int dtype, void* o_out, float* lse_out,
                         cudaStream_t st);

}  // namespace bdlm
