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
//
// Row counts.  L is the number of clean K/V rows (= clean token positions).  The clean query tensors
// (q, o, dO, dQ, LSE, D) have Lqc rows standing at positions cq_pos0 .. cq_pos0 + Lqc - 1; every noisy
// tensor (queries and keys) has Ln = nb * M rows, nb packed blocks.  The plain layer is Lqc = Ln = L,
// cq_pos0 = 0, prefix = nullptr; one rank's launch of the CSBP schedule (Algorithms 1, 2) and
// DFlash2-style blocks (appendix E) set them otherwise.
struct KArgs {
  int batch, L, M, H, Hkv, G, d;
  int Lqc, cq_pos0;   // clean query rows and the position of the first one
  int Ln, nb;         // noisy rows (= nb * M) and packed blocks
  const int* prefix;  // device [nb], non-decreasing: clean keys j < prefix[b] are visible to block b; nullptr = b * M
  // Clean K/V in gathered order (Algorithm 1's all-gather output used without a reordering copy): memory is a
  // sequence of chunks of kv_chunk_len rows, chunk m holds positions kv_chunk_pos[m] .. + kv_chunk_len - 1, and
  // kv_pos_chunk is the inverse map (position chunk -> memory chunk).  kv_chunk_len = 0: stored by position.
  int kv_chunk_len;
  const int* kv_chunk_pos;
  const int* kv_pos_chunk;
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
  const float* dsum[2];   // D_i = sum_d dO*O, [batch, H, rows of the stream's queries]
  __nv_bfloat16* dq[2];
  __nv_bfloat16* dk[2];
  __nv_bfloat16* dv[2];
  unsigned long long* trace;   // optional cycle counters (bdlm_set_trace_buffer), else nullptr
  int single_pass;             // backward: the fused kernel forms dQ^T per step and adds it into dq32 by TMA bulk add-reductions
  float* dq32[2];              // fp32 dQ accumulators [batch, H, dq32_rows, 128] (fused backward), else nullptr
  int dq32_rows[2];            // their row counts: the stream's query rows rounded up to the 64-row step of the fused kernel
};

__host__ __device__ __forceinline__ int rows_q(const KArgs& a, int qs) { return qs == CLEAN ? a.Lqc : a.Ln; }
__host__ __device__ __forceinline__ int rows_k(const KArgs& a, int ks) { return ks == CLEAN ? a.L : a.Ln; }

// Memory row of the clean key at position `pos` (the first key of a tile; tiles never straddle a chunk).
__device__ __forceinline__ int clean_key_row(const KArgs& a, int pos) {
  if (a.kv_chunk_len == 0) return pos;
  const int c = pos / a.kv_chunk_len;
  return __ldg(a.kv_pos_chunk + c) * a.kv_chunk_len + (pos - c * a.kv_chunk_len);
}
// Position of the clean key stored at memory row `row`.
__device__ __forceinline__ int clean_key_pos(const KArgs& a, int row) {
  if (a.kv_chunk_len == 0) return row;
  const int m = row / a.kv_chunk_len;
  return __ldg(a.kv_chunk_pos + m) + (row - m * a.kv_chunk_len);
}

// Clean-prefix length of packed noisy block b.
__device__ __forceinline__ int block_prefix(const KArgs& a, int b) {
  return a.prefix != nullptr ? __ldg(a.prefix + b) : b * a.M;
}
// Smallest packed block index in [0, nb] whose prefix exceeds x (nb if none); the table is non-decreasing.
__device__ __forceinline__ int first_block_prefix_gt(const KArgs& a, int x) {
  if (a.prefix == nullptr) return min(a.nb, x < 0 ? 0 : x / a.M + 1);
  int lo = 0, hi = a.nb;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(a.prefix + mid) > x) hi = mid; else lo = mid + 1;
  }
  return lo;
}

// Visible key interval [lo, hi) of query row i (stream qs) inside key stream ks
// (section 3.2: clean row -> clean keys 0..position; noisy row -> the clean keys before its block's
// prefix and the noisy keys of its own block).  Every row's visible set per key stream is one interval.
// Sliding-window layers: a clean key j is visible to a token at position p only if p - j < window.
__device__ __forceinline__ void visible_interval(const KArgs& a, int qs, int ks, int i, int& lo, int& hi) {
  const int M = a.M;
  if (ks == NOISY) {
    if (qs == CLEAN || !a.diag) { lo = 0; hi = 0; }
    else { lo = (i / M) * M; hi = lo + M; }
    return;
  }
  int pos, lim;
  if (qs == CLEAN) {
    pos = a.cq_pos0 + i;
    lim = (a.mode == 0) ? (pos + 1) : ((pos / M + 1) * M);
  } else {
    const int bi = i / M;
    lim = block_prefix(a, bi);
    pos = lim + (i - bi * M);
  }
  lo = a.kv_begin;
  if (a.window > 0) lo = max(lo, pos - a.window + 1);
  hi = min(a.kv_end, lim);
}

// Query rows [lo, hi) of stream qs (row indices of that stream's tensors) that see clean key j.
// Needs token positions to be non-decreasing along the packed rows when a window is set.
__device__ __forceinline__ void visible_queries_of_clean_key(const KArgs& a, int qs, int j, int& lo, int& hi) {
  const int M = a.M, W = a.window;
  if (qs == CLEAN) {
    const int p_lo = (a.mode == 0) ? j : (j / M) * M;
    lo = max(0, p_lo - a.cq_pos0);
    hi = (W > 0) ? min(a.Lqc, j + W - a.cq_pos0) : a.Lqc;
    hi = max(hi, 0);
  } else {
    lo = first_block_prefix_gt(a, j) * M;
    hi = a.Ln;
    if (W > 0) {
      // first block that is not seen in full: prefix + M - 1 - j >= W
      const int b1 = first_block_prefix_gt(a, j + W - M);
      hi = (b1 >= a.nb) ? a.Ln : b1 * M + min(M, max(0, W + j - block_prefix(a, b1)));
    }
  }
}

// Number of SMs of the current device (cached per device ordinal; 1 if the query fails).
int device_sm_count();

// The tensor-core kernels run one CTA per (tile, head or head pair, batch element x stream) on a one-dimensional grid;
// CTAs start in the order of their index.  The work of a tile grows linearly with its position (appendix B, Eq.
// block-work-by-position), and x counts tiles from the heaviest down.  Two orders:
//   tile_major = 0   x fastest: the CTAs running at one time are neighbouring tiles of one head, so they walk the same
//                    Q / dO / K / V tiles (and, in the fused backward, the same dQ accumulator tiles) together;
//   tile_major = 1   x slowest: the heaviest tiles of every head, batch element and stream start first -- longest job
//                    first over the whole launch.  Chosen by the launchers when the heaviest tile is a sizeable part of
//                    the ideal duration of the launch (short sequences), where the first order would start the heavy
//                    tiles of the second and later batch elements too late.
struct TileGrid { int nx, ny, nz, tile_major; };
__device__ __forceinline__ void tile_grid_decode(const TileGrid& g, int& x, int& y, int& z) {
  int i = blockIdx.x;
  if (!g.tile_major) { x = i % g.nx; i /= g.nx; y = i % g.ny; z = i / g.ny; }
  else { const int c = g.ny * g.nz; x = i / c; i -= x * c; y = i % g.ny; z = i / g.ny; }
}
inline TileGrid make_tile_grid(int nx, int ny, int nz) {
  TileGrid g = {nx, ny, nz, 0};
  // heaviest tile ~ nx units, whole launch ~ ny nz nx (nx + 1) / 2 units over the device's SMs: tile-major when the
  // heaviest tile exceeds a fifth of the ideal duration
  g.tile_major = (10LL * device_sm_count() > (long long)ny * nz * (nx + 1)) ? 1 : 0;
  return g;
}
// Number of CTAs, or 0 if it does not fit a grid dimension.
inline unsigned tile_grid_blocks(const TileGrid& g) {
  const long long n = (long long)g.nx * g.ny * g.nz;
  return n > 0x7fffffffLL ? 0u : (unsigned)n;
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
