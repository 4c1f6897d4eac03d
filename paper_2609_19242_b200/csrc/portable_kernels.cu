// Portable BDLM attention kernels: warp-level mma.sync (m16n8k16, bf16 -> fp32), any
// block_size, any L that is a multiple of block_size, d in {64, 128}.  They are the general
// path (and the fallback for shapes the tcgen05 kernels do not take).  Forward follows
// Algorithm 1 with one running softmax per query row across the clean-prefix tiles and the
// noisy-diagonal tiles (Eq. correctness-online-softmax-merge); backward follows Algorithm 2
// as a dK/dV pass (per key tile, summing over the query heads of the KV group and over both
// query streams, Eq. correctness-clean-gradient) and a dQ pass (Eq. correctness-query-gradient).
#include "bdlm_common.cuh"

namespace bdlm {
namespace {

using bf16 = __nv_bfloat16;
constexpr int BQ = 64;    // query rows per CTA (forward, dQ pass); keys per CTA in the dK/dV pass
constexpr int BK = 64;    // keys per tile (forward, dQ pass)
constexpr int BQ2 = 32;   // query rows per inner step of the dK/dV pass
constexpr int PAD = 8;    // bf16 elements of row padding: 16-byte rows stay aligned, fragments conflict-free
constexpr int NTHREADS = 128;

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// B fragment (k16 x n8) from a tile stored [k][n] row-major: transposing 8x8 loads.
__device__ __forceinline__ void ldsm_x2_trans(uint32_t& r0, uint32_t& r1, const bf16* p) {
  uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];\n"
               : "=r"(r0), "=r"(r1) : "r"(addr));
}

__device__ __forceinline__ uint32_t ld32(const bf16* p) { return *reinterpret_cast<const uint32_t*>(p); }

// Copy ROWS x D bf16 (global row stride ld elements) into smem [ROWS][D+PAD]; rows >= nvalid are zero.
template <int D, int ROWS>
__device__ __forceinline__ void load_tile(bf16* dst, const bf16* src, int64_t ld, int nvalid) {
  constexpr int CH = D / 8;
  for (int idx = threadIdx.x; idx < ROWS * CH; idx += NTHREADS) {
    int r = idx / CH, c = idx % CH;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (r < nvalid) val = *reinterpret_cast<const uint4*>(src + (int64_t)r * ld + c * 8);
    *reinterpret_cast<uint4*>(dst + r * (D + PAD) + c * 8) = val;
  }
}

// A fragment (16 x 16) of a row-major smem tile at (row0, col0).
template <int LD>
__device__ __forceinline__ void a_frag(uint32_t (&a)[4], const bf16* tile, int row0, int col0, int g, int t) {
  a[0] = ld32(tile + (row0 + g) * LD + col0 + 2 * t);
  a[1] = ld32(tile + (row0 + g + 8) * LD + col0 + 2 * t);
  a[2] = ld32(tile + (row0 + g) * LD + col0 + 8 + 2 * t);
  a[3] = ld32(tile + (row0 + g + 8) * LD + col0 + 8 + 2 * t);
}

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(NTHREADS) portable_fwd_kernel(const KArgs a) {
  constexpr int LD = D + PAD;
  const int qs = blockIdx.z & 1;
  const int b = blockIdx.z >> 1;
  if (a.q[qs] == nullptr) return;
  const int h = blockIdx.y, hk = h / a.G;
  const int q0 = (gridDim.x - 1 - blockIdx.x) * BQ;   // longest rows first
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  bf16* Vs = Ks + BK * LD;

  const int L = rows_q(a, qs);   // rows of this stream's query tensors
  if (q0 >= L) return;
  const int r0 = q0 + warp * 16 + g, r1 = r0 + 8;
  const int64_t qld = (int64_t)a.H * D;
  const int64_t kld = (int64_t)a.Hkv * D;
  const bf16* qbase = a.q[qs] + ((int64_t)b * L * a.H + h) * D;

  uint32_t qf[D / 16][4];
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    qf[kk][0] = r0 < L ? ld32(qbase + r0 * qld + kk * 16 + 2 * t) : 0u;
    qf[kk][1] = r1 < L ? ld32(qbase + r1 * qld + kk * 16 + 2 * t) : 0u;
    qf[kk][2] = r0 < L ? ld32(qbase + r0 * qld + kk * 16 + 8 + 2 * t) : 0u;
    qf[kk][3] = r1 < L ? ld32(qbase + r1 * qld + kk * 16 + 8 + 2 * t) : 0u;
  }

  float oacc[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int last_row = min(q0 + BQ, L) - 1;

  for (int ks = 0; ks < 2; ++ks) {
    int seg_lo, seg_hi, tmp;
    visible_interval(a, qs, ks, q0, seg_lo, tmp);
    visible_interval(a, qs, ks, last_row, tmp, seg_hi);
    if (seg_hi <= seg_lo) continue;
    int rlo0 = 0, rhi0 = 0, rlo1 = 0, rhi1 = 0;
    if (r0 < L) visible_interval(a, qs, ks, r0, rlo0, rhi0);
    if (r1 < L) visible_interval(a, qs, ks, r1, rlo1, rhi1);
    const bf16* kbase = a.k[ks] + ((int64_t)b * rows_k(a, ks) * a.Hkv + hk) * D;
    const bf16* vbase = a.v[ks] + ((int64_t)b * rows_k(a, ks) * a.Hkv + hk) * D;

    for (int k0 = seg_lo; k0 < seg_hi; k0 += BK) {
      __syncthreads();
      const int krow = ks == CLEAN ? clean_key_row(a, k0) : k0;   // where the tile's first key is stored
      load_tile<D, BK>(Ks, kbase + (int64_t)krow * kld, kld, seg_hi - k0);
      load_tile<D, BK>(Vs, vbase + (int64_t)krow * kld, kld, seg_hi - k0);
      __syncthreads();

      float s[BK / 8][4];
#pragma unroll
      for (int nt = 0; nt < BK / 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
        for (int nt = 0; nt < BK / 8; ++nt) {
          uint32_t b0 = ld32(Ks + (nt * 8 + g) * LD + kk * 16 + 2 * t);
          uint32_t b1 = ld32(Ks + (nt * 8 + g) * LD + kk * 16 + 8 + 2 * t);
          mma16816(s[nt], qf[kk], b0, b1);
        }
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < BK / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          int j = k0 + nt * 8 + 2 * t + (e & 1);
          bool vis = (e < 2) ? (j >= rlo0 && j < rhi0) : (j >= rlo1 && j < rhi1);
          float val = vis ? s[nt][e] * a.scale_log2 : -INFINITY;
          s[nt][e] = val;
          if (e < 2) mx0 = fmaxf(mx0, val); else mx1 = fmaxf(mx1, val);
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float base0 = (mn0 == -INFINITY) ? 0.f : mn0;
      const float base1 = (mn1 == -INFINITY) ? 0.f : mn1;
      const float c0 = exp2f(m0 - base0), c1 = exp2f(m1 - base1);
      m0 = mn0; m1 = mn1;
      float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < BK / 8; ++nt) {
        s[nt][0] = exp2f(s[nt][0] - base0); s[nt][1] = exp2f(s[nt][1] - base0);
        s[nt][2] = exp2f(s[nt][2] - base1); s[nt][3] = exp2f(s[nt][3] - base1);
        ps0 += s[nt][0] + s[nt][1];
        ps1 += s[nt][2] + s[nt][3];
      }
      l0 = l0 * c0 + ps0;
      l1 = l1 * c1 + ps1;
#pragma unroll
      for (int nt = 0; nt < D / 8; ++nt) {
        oacc[nt][0] *= c0; oacc[nt][1] *= c0; oacc[nt][2] *= c1; oacc[nt][3] *= c1;
      }
#pragma unroll
      for (int kk2 = 0; kk2 < BK / 16; ++kk2) {
        uint32_t pa[4];
        pa[0] = pack_bf16(s[2 * kk2][0], s[2 * kk2][1]);
        pa[1] = pack_bf16(s[2 * kk2][2], s[2 * kk2][3]);
        pa[2] = pack_bf16(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1]);
        pa[3] = pack_bf16(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3]);
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
          uint32_t b0, b1;
          ldsm_x2_trans(b0, b1, Vs + (kk2 * 16 + (lane & 15)) * LD + nt * 8);
          mma16816(oacc[nt], pa, b0, b1);
        }
      }
    }
  }

  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
  bf16* obase = a.o[qs] + ((int64_t)b * L * a.H + h) * D;
#pragma unroll
  for (int nt = 0; nt < D / 8; ++nt) {
    if (r0 < L) *reinterpret_cast<uint32_t*>(obase + r0 * qld + nt * 8 + 2 * t) = pack_bf16(oacc[nt][0] * inv0, oacc[nt][1] * inv0);
    if (r1 < L) *reinterpret_cast<uint32_t*>(obase + r1 * qld + nt * 8 + 2 * t) = pack_bf16(oacc[nt][2] * inv1, oacc[nt][3] * inv1);
  }
  if (t == 0) {
    float* lse = a.lse[qs] + ((int64_t)b * a.H + h) * L;
    if (r0 < L) lse[r0] = l0 > 0.f ? (m0 + log2f(l0)) * LN2 : -INFINITY;
    if (r1 < L) lse[r1] = l1 > 0.f ? (m1 + log2f(l1)) * LN2 : -INFINITY;
  }
}

// ------------------------------------------------------------------------------------------
// backward, dQ pass: per query tile, loop over its visible key tiles
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(NTHREADS) portable_dq_kernel(const KArgs a) {
  constexpr int LD = D + PAD;
  const int qs = blockIdx.z & 1;
  const int b = blockIdx.z >> 1;
  const int h = blockIdx.y, hk = h / a.G;
  const int q0 = (gridDim.x - 1 - blockIdx.x) * BQ;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);
  bf16* dOs = Qs + BQ * LD;
  bf16* Ks = dOs + BQ * LD;
  bf16* Vs = Ks + BK * LD;

  if (a.q[qs] == nullptr) return;
  const int L = rows_q(a, qs);   // rows of this stream's query tensors
  if (q0 >= L) return;
  const int r0 = q0 + warp * 16 + g, r1 = r0 + 8;
  const int64_t qld = (int64_t)a.H * D;
  const int64_t kld = (int64_t)a.Hkv * D;
  const int64_t qoff = ((int64_t)b * L * a.H + h) * D;
  load_tile<D, BQ>(Qs, a.q[qs] + qoff + (int64_t)q0 * qld, qld, L - q0);
  load_tile<D, BQ>(dOs, a.dout[qs] + qoff + (int64_t)q0 * qld, qld, L - q0);

  const float* lsep = a.lse[qs] + ((int64_t)b * a.H + h) * L;
  const float* dsp = a.dsum[qs] + ((int64_t)b * a.H + h) * L;
  // +inf LSE makes P = exp2(s - inf) = 0 for rows past the end or with an empty key set
  float lse0 = INFINITY, lse1 = INFINITY, ds0 = 0.f, ds1 = 0.f;
  if (r0 < L) { float z = lsep[r0]; lse0 = isfinite(z) ? z * LOG2E : INFINITY; ds0 = dsp[r0]; }
  if (r1 < L) { float z = lsep[r1]; lse1 = isfinite(z) ? z * LOG2E : INFINITY; ds1 = dsp[r1]; }

  float dq[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }
  const int last_row = min(q0 + BQ, L) - 1;

  for (int ks = 0; ks < 2; ++ks) {
    int seg_lo, seg_hi, tmp;
    visible_interval(a, qs, ks, q0, seg_lo, tmp);
    visible_interval(a, qs, ks, last_row, tmp, seg_hi);
    if (seg_hi <= seg_lo) continue;
    int rlo0 = 0, rhi0 = 0, rlo1 = 0, rhi1 = 0;
    if (r0 < L) visible_interval(a, qs, ks, r0, rlo0, rhi0);
    if (r1 < L) visible_interval(a, qs, ks, r1, rlo1, rhi1);
    const bf16* kbase = a.k[ks] + ((int64_t)b * rows_k(a, ks) * a.Hkv + hk) * D;
    const bf16* vbase = a.v[ks] + ((int64_t)b * rows_k(a, ks) * a.Hkv + hk) * D;

    for (int k0 = seg_lo; k0 < seg_hi; k0 += BK) {
      __syncthreads();
      const int krow = ks == CLEAN ? clean_key_row(a, k0) : k0;   // where the tile's first key is stored
      load_tile<D, BK>(Ks, kbase + (int64_t)krow * kld, kld, seg_hi - k0);
      load_tile<D, BK>(Vs, vbase + (int64_t)krow * kld, kld, seg_hi - k0);
      __syncthreads();

      float s[BK / 8][4], dp[BK / 8][4];
#pragma unroll
      for (int nt = 0; nt < BK / 8; ++nt) {
        s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
        dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
      }
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        uint32_t qa[4], da[4];
        a_frag<LD>(qa, Qs, warp * 16, kk * 16, g, t);
        a_frag<LD>(da, dOs, warp * 16, kk * 16, g, t);
#pragma unroll
        for (int nt = 0; nt < BK / 8; ++nt) {
          uint32_t b0 = ld32(Ks + (nt * 8 + g) * LD + kk * 16 + 2 * t);
          uint32_t b1 = ld32(Ks + (nt * 8 + g) * LD + kk * 16 + 8 + 2 * t);
          mma16816(s[nt], qa, b0, b1);
          uint32_t v0 = ld32(Vs + (nt * 8 + g) * LD + kk * 16 + 2 * t);
          uint32_t v1 = ld32(Vs + (nt * 8 + g) * LD + kk * 16 + 8 + 2 * t);
          mma16816(dp[nt], da, v0, v1);
        }
      }
#pragma unroll
      for (int nt = 0; nt < BK / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          int j = k0 + nt * 8 + 2 * t + (e & 1);
          bool vis = (e < 2) ? (j >= rlo0 && j < rhi0) : (j >= rlo1 && j < rhi1);
          float p = vis ? exp2f(s[nt][e] * a.scale_log2 - (e < 2 ? lse0 : lse1)) : 0.f;
          s[nt][e] = p * (dp[nt][e] - (e < 2 ? ds0 : ds1));
        }
      }
#pragma unroll
      for (int kk2 = 0; kk2 < BK / 16; ++kk2) {
        uint32_t pa[4];
        pa[0] = pack_bf16(s[2 * kk2][0], s[2 * kk2][1]);
        pa[1] = pack_bf16(s[2 * kk2][2], s[2 * kk2][3]);
        pa[2] = pack_bf16(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1]);
        pa[3] = pack_bf16(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3]);
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
          uint32_t b0, b1;
          ldsm_x2_trans(b0, b1, Ks + (kk2 * 16 + (lane & 15)) * LD + nt * 8);
          mma16816(dq[nt], pa, b0, b1);
        }
      }
    }
  }
  bf16* dqbase = a.dq[qs] + qoff;
#pragma unroll
  for (int nt = 0; nt < D / 8; ++nt) {
    if (r0 < L) *reinterpret_cast<uint32_t*>(dqbase + r0 * qld + nt * 8 + 2 * t) = pack_bf16(dq[nt][0] * a.scale, dq[nt][1] * a.scale);
    if (r1 < L) *reinterpret_cast<uint32_t*>(dqbase + r1 * qld + nt * 8 + 2 * t) = pack_bf16(dq[nt][2] * a.scale, dq[nt][3] * a.scale);
  }
}

// ------------------------------------------------------------------------------------------
// backward, dK/dV pass: per key tile of one KV head, loop over every query tile that sees it,
// over both query streams and over the G query heads of the group (fixed order, no atomics)
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(NTHREADS) portable_dkdv_kernel(const KArgs a) {
  constexpr int LD = D + PAD;
  const int ks = blockIdx.z & 1;
  const int b = blockIdx.z >> 1;
  const int hk = blockIdx.y;
  const int k0_row = blockIdx.x * BQ;   // the tile's first key in memory; key tile 0 has the most queries: first
  const int k0 = ks == CLEAN ? clean_key_pos(a, k0_row) : k0_row;   // and its position
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  bf16* Vs = Ks + BQ * LD;
  bf16* Qs = Vs + BQ * LD;
  bf16* dOs = Qs + BQ2 * LD;
  float* lse_s = reinterpret_cast<float*>(dOs + BQ2 * LD);
  float* d_s = lse_s + BQ2;
  int* vlo_s = reinterpret_cast<int*>(d_s + BQ2);
  int* vhi_s = vlo_s + BQ2;

  const int L = rows_k(a, ks), M = a.M;   // rows of this stream's K/V tensors
  if (k0_row >= L || a.dk[ks] == nullptr) return;
  const int64_t qld = (int64_t)a.H * D;
  const int64_t kld = (int64_t)a.Hkv * D;
  const int64_t koff = ((int64_t)b * L * a.Hkv + hk) * D;
  load_tile<D, BQ>(Ks, a.k[ks] + koff + (int64_t)k0_row * kld, kld, L - k0_row);
  load_tile<D, BQ>(Vs, a.v[ks] + koff + (int64_t)k0_row * kld, kld, L - k0_row);
  const int j0 = k0 + warp * 16 + g, j1 = j0 + 8;
  const int k_last = k0 + min(BQ, L - k0_row) - 1;   // position of the tile's last key

  float dk[D / 8][4], dv[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
    dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
  }

  for (int qs = 0; qs < 2; ++qs) {
    // query rows of stream qs that can see some key of this tile
    int q_lo, q_hi;
    if (a.q[qs] == nullptr) continue;
    if (ks == CLEAN) {
      // the visible-query interval moves up with the key: first key's lower end, last key's upper end
      int tmp;
      visible_queries_of_clean_key(a, qs, k0, q_lo, tmp);
      visible_queries_of_clean_key(a, qs, k_last, tmp, q_hi);
    } else {
      if (qs == CLEAN) continue;
      q_lo = (k0 / M) * M;
      q_hi = min(L, (k_last / M + 1) * M);
    }
    const int Lq = rows_q(a, qs);
    for (int hh = 0; hh < a.G; ++hh) {
      const int h = hk * a.G + hh;
      const int64_t qoff = ((int64_t)b * Lq * a.H + h) * D;
      const float* lsep = a.lse[qs] + ((int64_t)b * a.H + h) * Lq;
      const float* dsp = a.dsum[qs] + ((int64_t)b * a.H + h) * Lq;
      for (int qq = q_lo; qq < q_hi; qq += BQ2) {
        __syncthreads();
        load_tile<D, BQ2>(Qs, a.q[qs] + qoff + (int64_t)qq * qld, qld, q_hi - qq);
        load_tile<D, BQ2>(dOs, a.dout[qs] + qoff + (int64_t)qq * qld, qld, q_hi - qq);
        if (threadIdx.x < BQ2) {
          int i = qq + threadIdx.x;
          float z = INFINITY, dd = 0.f;
          int lo = 0, hi = 0;
          if (i < q_hi) {
            float zz = lsep[i];
            z = isfinite(zz) ? zz * LOG2E : INFINITY;
            dd = dsp[i];
            visible_interval(a, qs, ks, i, lo, hi);
          }
          lse_s[threadIdx.x] = z; d_s[threadIdx.x] = dd;
          vlo_s[threadIdx.x] = lo; vhi_s[threadIdx.x] = hi;
        }
        __syncthreads();

        // S^T = K Q^T and dP^T = V dO^T : [16 keys of this warp] x [32 queries]
        float st[BQ2 / 8][4], dpt[BQ2 / 8][4];
#pragma unroll
        for (int nt = 0; nt < BQ2 / 8; ++nt) {
          st[nt][0] = st[nt][1] = st[nt][2] = st[nt][3] = 0.f;
          dpt[nt][0] = dpt[nt][1] = dpt[nt][2] = dpt[nt][3] = 0.f;
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          uint32_t ka[4], va[4];
          a_frag<LD>(ka, Ks, warp * 16, kk * 16, g, t);
          a_frag<LD>(va, Vs, warp * 16, kk * 16, g, t);
#pragma unroll
          for (int nt = 0; nt < BQ2 / 8; ++nt) {
            uint32_t b0 = ld32(Qs + (nt * 8 + g) * LD + kk * 16 + 2 * t);
            uint32_t b1 = ld32(Qs + (nt * 8 + g) * LD + kk * 16 + 8 + 2 * t);
            mma16816(st[nt], ka, b0, b1);
            uint32_t c0 = ld32(dOs + (nt * 8 + g) * LD + kk * 16 + 2 * t);
            uint32_t c1 = ld32(dOs + (nt * 8 + g) * LD + kk * 16 + 8 + 2 * t);
            mma16816(dpt[nt], va, c0, c1);
          }
        }
        // P^T = exp(S^T - LSE_i) on visible pairs, dS^T = P^T * (dP^T - D_i)
#pragma unroll
        for (int nt = 0; nt < BQ2 / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            int col = nt * 8 + 2 * t + (e & 1);
            int j = (e < 2) ? j0 : j1;
            bool vis = (j >= vlo_s[col]) && (j < vhi_s[col]);
            float p = vis ? exp2f(st[nt][e] * a.scale_log2 - lse_s[col]) : 0.f;
            st[nt][e] = p;
            dpt[nt][e] = p * (dpt[nt][e] - d_s[col]);
          }
        }
#pragma unroll
        for (int kk2 = 0; kk2 < BQ2 / 16; ++kk2) {
          uint32_t pa[4], da[4];
          pa[0] = pack_bf16(st[2 * kk2][0], st[2 * kk2][1]);
          pa[1] = pack_bf16(st[2 * kk2][2], st[2 * kk2][3]);
          pa[2] = pack_bf16(st[2 * kk2 + 1][0], st[2 * kk2 + 1][1]);
          pa[3] = pack_bf16(st[2 * kk2 + 1][2], st[2 * kk2 + 1][3]);
          da[0] = pack_bf16(dpt[2 * kk2][0], dpt[2 * kk2][1]);
          da[1] = pack_bf16(dpt[2 * kk2][2], dpt[2 * kk2][3]);
          da[2] = pack_bf16(dpt[2 * kk2 + 1][0], dpt[2 * kk2 + 1][1]);
          da[3] = pack_bf16(dpt[2 * kk2 + 1][2], dpt[2 * kk2 + 1][3]);
#pragma unroll
          for (int nt = 0; nt < D / 8; ++nt) {
            uint32_t b0, b1;
            ldsm_x2_trans(b0, b1, dOs + (kk2 * 16 + (lane & 15)) * LD + nt * 8);
            mma16816(dv[nt], pa, b0, b1);
            ldsm_x2_trans(b0, b1, Qs + (kk2 * 16 + (lane & 15)) * LD + nt * 8);
            mma16816(dk[nt], da, b0, b1);
          }
        }
      }
    }
  }
  bf16* dkb = a.dk[ks] + koff;
  bf16* dvb = a.dv[ks] + koff;
#pragma unroll
  for (int nt = 0; nt < D / 8; ++nt) {
    const int row0 = k0_row + (j0 - k0), row1 = row0 + 8;   // where the keys are stored
    if (row0 < L) {
      *reinterpret_cast<uint32_t*>(dkb + row0 * kld + nt * 8 + 2 * t) = pack_bf16(dk[nt][0] * a.scale, dk[nt][1] * a.scale);
      *reinterpret_cast<uint32_t*>(dvb + row0 * kld + nt * 8 + 2 * t) = pack_bf16(dv[nt][0], dv[nt][1]);
    }
    if (row1 < L) {
      *reinterpret_cast<uint32_t*>(dkb + row1 * kld + nt * 8 + 2 * t) = pack_bf16(dk[nt][2] * a.scale, dk[nt][3] * a.scale);
      *reinterpret_cast<uint32_t*>(dvb + row1 * kld + nt * 8 + 2 * t) = pack_bf16(dv[nt][2], dv[nt][3]);
    }
  }
}

int max_query_rows(const KArgs& a) {
  return max(a.q[CLEAN] != nullptr ? a.Lqc : 0, a.q[NOISY] != nullptr ? a.Ln : 0);
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

cudaError_t launch_portable_fwd(const KArgs& a, cudaStream_t st) {
  dim3 grid((max_query_rows(a) + BQ - 1) / BQ, a.H, a.batch * 2);
  size_t smem = (size_t)2 * BK * (a.d + PAD) * sizeof(bf16);
  cudaError_t e;
  if (a.d == 128) {
    if ((e = set_smem(portable_fwd_kernel<128>, smem)) != cudaSuccess) return e;
    portable_fwd_kernel<128><<<grid, NTHREADS, smem, st>>>(a);
  } else {
    if ((e = set_smem(portable_fwd_kernel<64>, smem)) != cudaSuccess) return e;
    portable_fwd_kernel<64><<<grid, NTHREADS, smem, st>>>(a);
  }
  return cudaGetLastError();
}

cudaError_t launch_portable_bwd(const KArgs& a, int passes, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  if (passes & BDLM_BWD_PASS_DKDV) {
    dim3 grid((max(a.L, a.Ln) + BQ - 1) / BQ, a.Hkv, a.batch * 2);
    size_t smem = (size_t)(2 * BQ + 2 * BQ2) * (a.d + PAD) * sizeof(bf16) + 4 * BQ2 * sizeof(float);
    if (a.d == 128) {
      if ((e = set_smem(portable_dkdv_kernel<128>, smem)) != cudaSuccess) return e;
      portable_dkdv_kernel<128><<<grid, NTHREADS, smem, st>>>(a);
    } else {
      if ((e = set_smem(portable_dkdv_kernel<64>, smem)) != cudaSuccess) return e;
      portable_dkdv_kernel<64><<<grid, NTHREADS, smem, st>>>(a);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (passes & BDLM_BWD_PASS_DQ) {
    dim3 grid((max_query_rows(a) + BQ - 1) / BQ, a.H, a.batch * 2);
    size_t smem = (size_t)(2 * BQ + 2 * BK) * (a.d + PAD) * sizeof(bf16);
    if (a.d == 128) {
      if ((e = set_smem(portable_dq_kernel<128>, smem)) != cudaSuccess) return e;
      portable_dq_kernel<128><<<grid, NTHREADS, smem, st>>>(a);
    } else {
      if ((e = set_smem(portable_dq_kernel<64>, smem)) != cudaSuccess) return e;
      portable_dq_kernel<64><<<grid, NTHREADS, smem, st>>>(a);
    }
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace bdlm
