// BDLM attention backward on tcgen05 tensor cores (Algorithm 2 on one device):
//
//   dK/dV pass  one CTA per 128-key tile of one KV head.  K and V stay in shared memory; the
//               CTA walks every 128-row query tile that sees the key tile -- clean and noisy
//               query streams, all G query heads of the group (Eq. correctness-clean-gradient;
//               a noisy key tile is seen only by its own block's queries, Eq.
//               correctness-corrupted-gradient) -- and accumulates dV += P^T dO and
//               dK += dS^T Q in tensor memory, in a fixed order, without atomics.
//   dQ pass     one CTA per 128-row query tile of one head; Q and dO stay in shared memory,
//               the CTA walks its visible key tiles and accumulates dQ += dS K
//               (Eq. correctness-query-gradient).
//
// Both are warp-specialised: warp 8 issues TMA loads, warp 9 issues tcgen05.mma, warps 0-7
// (two warpgroups, each owning half of the 128 score columns of every TMEM lane) recompute
// P = exp(S - LSE) and dS = P * (dP - D) and hand them back to the tensor core as TMEM-resident
// A operands.  Every wait is bounded and abortable.
#include "tc_common.cuh"
#include "tc_launch.h"

namespace bdlm {
namespace {

using namespace tc;
using bf16 = __nv_bfloat16;

struct BwdMaps {
  CUtensorMap q[2], dout[2], k[2], v[2];
};

constexpr int BWD_THREADS = 320;
constexpr int TILE_BYTES = 2 * PANEL_BYTES;
constexpr uint32_t IDESC_KK = make_idesc(128, 128, false, false);   // A, B both K-major
constexpr uint32_t IDESC_KM = make_idesc(128, 128, false, true);    // B MN-major (a [k][n] tile as loaded)

// K-major operand tile (two 64-column panels): descriptor of the kk-th 16-wide slice of the contraction dim
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile, int kk) {
  return smem_desc(tile + (kk >> 2) * PANEL_BYTES + (kk & 3) * 32, 16, 1024);
}
// MN-major operand: the tile is stored [contraction row][128 columns]; slice kk = rows 16kk..16kk+15
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t tile, int kk) {
  return smem_desc(tile + kk * 2048, PANEL_BYTES, 1024);
}

__device__ __forceinline__ void tma_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int col0, int row0, int b) {
  tma_load_3d(dst, map, bar, col0, row0, b);
  tma_load_3d(dst + PANEL_BYTES, map, bar, col0 + 64, row0, b);
}

// Write a thread's 128 accumulator columns (4 x 32) as bf16 to a global row, scaled.
__device__ __forceinline__ void store_row_chunk(bf16* dst, const uint32_t (&v)[32], float scale) {
#pragma unroll
  for (int e8 = 0; e8 < 4; ++e8) {
    uint4 o;
    uint32_t* po = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int e = 0; e < 4; ++e)
      po[e] = pack_bf16(__uint_as_float(v[e8 * 8 + 2 * e]) * scale, __uint_as_float(v[e8 * 8 + 2 * e + 1]) * scale);
    *reinterpret_cast<uint4*>(dst + e8 * 8) = o;
  }
}

// =============================================================================================
// dK/dV pass
// =============================================================================================
constexpr int DKDV_ARR = 6 * TILE_BYTES;            // after K, V and two (Q, dO) stages
constexpr int DKDV_BARS = DKDV_ARR + 4096 + 64;
constexpr int DKDV_SMEM = DKDV_BARS + 256 + 1024;

struct QStep { int qs, h, q0; };

__global__ void __launch_bounds__(BWD_THREADS, 1)
tc_dkdv_kernel(const __grid_constant__ BwdMaps maps, const KArgs a, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sK = base, sV = base + TILE_BYTES, sQ0 = base + 2 * TILE_BYTES;   // stage s: Q at sQ0 + s*2*TILE, dO after it
  float* lse_s = reinterpret_cast<float*>(sm + DKDV_ARR);          // [2][128], log2 units
  float* d_s = lse_s + 256;                                        // [2][128]
  int* vlo_s = reinterpret_cast<int*>(d_s + 256);                  // [2][128] visible key interval of each query column
  int* vhi_s = vlo_s + 256;
  int* flag_s = reinterpret_cast<int*>(sm + DKDV_ARR + 4096);      // [2] tile needs masking
  const uint32_t bars = base + DKDV_BARS;
  const uint32_t bar_kv = bars, bar_qdo_full = bars + 8 /*[2]*/, bar_qdo_empty = bars + 24 /*[2]*/,
                 bar_st = bars + 40, bar_dpt = bars + 48, bar_pt = bars + 56, bar_dst = bars + 64, bar_done = bars + 72;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + DKDV_BARS + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + DKDV_BARS + 136);

  const int ks = blockIdx.z & 1, b = blockIdx.z >> 1, hk = blockIdx.y;
  const int k0 = blockIdx.x * TILE;   // key tile 0 has the most query tiles: scheduled first
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int L = a.L, M = a.M, NT = L / TILE;

  // query tiles that see this key tile: segment A then segment B, for each head of the group
  int tA0, nA, tB0 = 0, nB = 0;
  if (ks == CLEAN) {
    const int qa_lo = (a.mode == 0) ? k0 : (k0 / M) * M;
    tA0 = qa_lo / TILE; nA = NT - tA0;
    const int qb_lo = (k0 / M + 1) * M;
    if (qb_lo < L) { tB0 = qb_lo / TILE; nB = NT - tB0; }
  } else {
    const int lo = (k0 / M) * M, hi = min(L, ((k0 + TILE - 1) / M + 1) * M);
    tA0 = lo / TILE; nA = (hi + TILE - 1) / TILE - tA0;
  }
  const int per_head = nA + nB;
  const int nsteps = per_head * a.G;
  auto step_of = [&](int i) {
    QStep s;
    const int hh = i / per_head, r = i - hh * per_head;
    s.h = hk * a.G + hh;
    if (r < nA) { s.qs = (ks == NOISY) ? NOISY : CLEAN; s.q0 = (tA0 + r) * TILE; }
    else { s.qs = NOISY; s.q0 = (tB0 + r - nA) * TILE; }
    return s;
  };

  if (threadIdx.x == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_qdo_full, 1); mbar_init(bar_qdo_full + 8, 1);
    mbar_init(bar_qdo_empty, 1); mbar_init(bar_qdo_empty + 8, 1);
    mbar_init(bar_st, 1); mbar_init(bar_dpt, 1);
    mbar_init(bar_pt, 256); mbar_init(bar_dst, 256);
    mbar_init(bar_done, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: [0,128) S^T / P^T   [128,256) dP^T / dS^T   [256,384) dV   [384,512) dK

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      mbar_expect_tx(bar_kv, 2 * TILE_BYTES);
      tma_tile(sK, &maps.k[ks], bar_kv, hk * 128, k0, b);
      tma_tile(sV, &maps.v[ks], bar_kv, hk * 128, k0, b);
    }
    bool ok = true;
    for (int i = 0; i < nsteps && ok; ++i) {
      const int s = i & 1;
      if (i >= 2) ok = mbar_wait_abortable(bar_qdo_empty + 8 * s, ((i >> 1) - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const QStep st = step_of(i);
      const float* lsep = a.lse[st.qs] + ((int64_t)b * a.H + st.h) * L + st.q0;
      const float* dsp = a.dsum[st.qs] + ((int64_t)b * a.H + st.h) * L + st.q0;
      bool need = false;
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        const int c = lane + 32 * c4;
        const float z = lsep[c];
        int lo, hi;
        visible_interval(st.qs, ks, st.q0 + c, M, a.mode, a.kv_begin, a.kv_end, a.diag, lo, hi);
        lse_s[s * 128 + c] = isfinite(z) ? z * LOG2E : INFINITY;
        d_s[s * 128 + c] = dsp[c];
        vlo_s[s * 128 + c] = lo;
        vhi_s[s * 128 + c] = hi;
        need |= (lo > k0) || (hi < k0 + TILE);
      }
      need = __any_sync(0xffffffffu, need);
      if (lane == 0) flag_s[s] = need ? 1 : 0;
      __syncwarp();
      if (lane == 0) {
        const uint32_t bar = bar_qdo_full + 8 * s;
        const uint32_t dQ = sQ0 + s * 2 * TILE_BYTES;
        mbar_expect_tx(bar, 2 * TILE_BYTES);
        tma_tile(dQ, &maps.q[st.qs], bar, st.h * 128, st.q0, b);
        tma_tile(dQ + TILE_BYTES, &maps.dout[st.qs], bar, st.h * 128, st.q0, b);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer (one thread)
    if (lane == 0 && nsteps > 0) {
      bool ok = mbar_wait_abortable(bar_kv, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_qdo_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tmem, kmajor_desc(sK, kk), kmajor_desc(sQ0, kk), IDESC_KK, kk > 0);
        mma_commit(bar_st);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tmem + 128, kmajor_desc(sV, kk), kmajor_desc(sQ0 + TILE_BYTES, kk), IDESC_KK, kk > 0);
        mma_commit(bar_dpt);
      }
      for (int i = 0; i < nsteps && ok; ++i) {
        const int s = i & 1;
        const uint32_t cQ = sQ0 + s * 2 * TILE_BYTES, cdO = cQ + TILE_BYTES;
        const uint32_t nQ = sQ0 + (s ^ 1) * 2 * TILE_BYTES, ndO = nQ + TILE_BYTES;
        // dV += P^T dO_i   (P^T: this lane's 64+64 bf16 pairs at columns [0,32) and [64,96))
        ok = mbar_wait_abortable(bar_pt, i & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tmem + 256, tmem + (kk < 4 ? kk * 8 : 64 + (kk - 4) * 8), mnmajor_desc(cdO, kk), IDESC_KM, (i > 0 || kk > 0) ? 1u : 0u);
        // S^T of the next step may start as soon as its Q is in shared memory
        if (i + 1 < nsteps) {
          ok = mbar_wait_abortable(bar_qdo_full + 8 * (s ^ 1), ((i + 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) mma_ss(tmem, kmajor_desc(sK, kk), kmajor_desc(nQ, kk), IDESC_KK, kk > 0);
          mma_commit(bar_st);
        }
        // dK += dS^T Q_i
        ok = mbar_wait_abortable(bar_dst, i & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tmem + 384, tmem + 128 + (kk < 4 ? kk * 8 : 64 + (kk - 4) * 8), mnmajor_desc(cQ, kk), IDESC_KM, (i > 0 || kk > 0) ? 1u : 0u);
        mma_commit(bar_qdo_empty + 8 * s);
        if (i + 1 < nsteps) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) mma_ss(tmem + 128, kmajor_desc(sV, kk), kmajor_desc(ndO, kk), IDESC_KK, kk > 0);
          mma_commit(bar_dpt);
        }
      }
      mma_commit(bar_done);
    }
  } else {
    // ------------------------------------------------------------------ compute warpgroups
    const int w = warp >> 2;                                   // column half: query columns [64w, 64w+64)
    const int r = (warp & 3) * 32 + lane;                      // TMEM lane = key row of the tile
    const int j = k0 + r;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = w * 64;
    bool ok = true;
    for (int i = 0; i < nsteps; ++i) {
      const int s = i & 1;
      ok = mbar_wait_abortable(bar_qdo_full + 8 * s, (i >> 1) & 1, abort_flag);
      ok = ok && mbar_wait_abortable(bar_st, i & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t x[64];
      {
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(x);
        tmem_ld32(tl + c0, c[0]); tmem_ld32(tl + c0 + 32, c[1]);
        tmem_wait_ld();
      }
      const bool need_mask = flag_s[s] != 0;
      const float* lz = lse_s + s * 128 + c0;
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        float p = exp2f(__uint_as_float(x[c]) * a.scale_log2 - lz[c]);
        if (need_mask) p = (j >= vlo_s[s * 128 + c0 + c] && j < vhi_s[s * 128 + c0 + c]) ? p : 0.f;
        x[c] = __float_as_uint(p);
      }
      {
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) pk[e] = pack_bf16(__uint_as_float(x[2 * e]), __uint_as_float(x[2 * e + 1]));
        tmem_st32(tl + c0, pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_pt);

      ok = mbar_wait_abortable(bar_dpt, i & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      {
        uint32_t y[64];
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(y);
        tmem_ld32(tl + 128 + c0, c[0]); tmem_ld32(tl + 128 + c0 + 32, c[1]);
        tmem_wait_ld();
        const float* dz = d_s + s * 128 + c0;
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float d0 = __uint_as_float(x[2 * e]) * (__uint_as_float(y[2 * e]) - dz[2 * e]);
          const float d1 = __uint_as_float(x[2 * e + 1]) * (__uint_as_float(y[2 * e + 1]) - dz[2 * e + 1]);
          pk[e] = pack_bf16(d0, d1);
        }
        tmem_st32(tl + 128 + c0, pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_dst);
    }
    // epilogue: warpgroup 0 writes dV, warpgroup 1 writes dK (scaled)
    if (ok && nsteps > 0) {
      ok = mbar_wait_abortable(bar_done, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      bf16* dst = (w == 0 ? a.dv[ks] : a.dk[ks]) + (((int64_t)b * L + j) * a.Hkv + hk) * 128;
      const float sc = (w == 0) ? 1.f : a.scale;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t v[32];
        if (nsteps > 0) { tmem_ld32(tl + 256 + w * 128 + c * 32, v); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        store_row_chunk(dst + c * 32, v, sc);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tmem, 512);
}

// =============================================================================================
// dQ pass
// =============================================================================================
constexpr int DQ_BARS = 6 * TILE_BYTES;             // Q, dO, two (K, V) stages
constexpr int DQ_SMEM = DQ_BARS + 256 + 1024;

__global__ void __launch_bounds__(BWD_THREADS, 1)
tc_dq_kernel(const __grid_constant__ BwdMaps maps, const KArgs a, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base, sdO = base + TILE_BYTES, sK0 = base + 2 * TILE_BYTES;   // stage s: K at sK0 + s*2*TILE, V after it
  const uint32_t bars = base + DQ_BARS;
  const uint32_t bar_qdo = bars, bar_kv_full = bars + 8 /*[2]*/, bar_kv_empty = bars + 24 /*[2]*/,
                 bar_s = bars + 40 /*[2]*/, bar_dp = bars + 56, bar_ds = bars + 64, bar_done = bars + 72;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + DQ_BARS + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + DQ_BARS + 136);

  const int qs = blockIdx.z & 1, b = blockIdx.z >> 1, h = blockIdx.y, hk = h / a.G;
  const int q0 = (gridDim.x - 1 - blockIdx.x) * TILE;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int L = a.L;

  // key tiles visible from this query tile: clean segment, then noisy segment
  int seg_lo[2], ntile[2], lo_last[2], hi_first[2];
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    int lo_f, hi_f, lo_l, hi_l;
    visible_interval(qs, ks, q0, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, lo_f, hi_f);
    visible_interval(qs, ks, q0 + TILE - 1, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, lo_l, hi_l);
    seg_lo[ks] = lo_f; lo_last[ks] = lo_l; hi_first[ks] = hi_f;
    ntile[ks] = hi_l > lo_f ? (hi_l - lo_f + TILE - 1) / TILE : 0;
  }
  const int nsteps = ntile[0] + ntile[1];
  auto tile_ks = [&](int i) { return i < ntile[0] ? 0 : 1; };
  auto tile_k0 = [&](int i) { return i < ntile[0] ? seg_lo[0] + i * TILE : seg_lo[1] + (i - ntile[0]) * TILE; };

  if (threadIdx.x == 0) {
    mbar_init(bar_qdo, 1);
    mbar_init(bar_kv_full, 1); mbar_init(bar_kv_full + 8, 1);
    mbar_init(bar_kv_empty, 1); mbar_init(bar_kv_empty + 8, 1);
    mbar_init(bar_s, 1); mbar_init(bar_s + 8, 1);
    mbar_init(bar_dp, 1); mbar_init(bar_ds, 256); mbar_init(bar_done, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: [0,128) S even / dS   [128,256) dP   [256,384) dQ   [384,512) S odd / dS
  auto s_col = [&](int i) { return (i & 1) ? 384u : 0u; };

  if (warp == 8) {
    if (lane == 0 && nsteps > 0) {
      mbar_expect_tx(bar_qdo, 2 * TILE_BYTES);
      tma_tile(sQ, &maps.q[qs], bar_qdo, h * 128, q0, b);
      tma_tile(sdO, &maps.dout[qs], bar_qdo, h * 128, q0, b);
      bool ok = true;
      for (int i = 0; i < nsteps && ok; ++i) {
        const int s = i & 1;
        if (i >= 2) ok = mbar_wait_abortable(bar_kv_empty + 8 * s, ((i >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        const int ks = tile_ks(i), k0 = tile_k0(i);
        const uint32_t bar = bar_kv_full + 8 * s, dK = sK0 + s * 2 * TILE_BYTES;
        mbar_expect_tx(bar, 2 * TILE_BYTES);
        tma_tile(dK, &maps.k[ks], bar, hk * 128, k0, b);
        tma_tile(dK + TILE_BYTES, &maps.v[ks], bar, hk * 128, k0, b);
      }
    }
  } else if (warp == 9) {
    if (lane == 0 && nsteps > 0) {
      bool ok = mbar_wait_abortable(bar_qdo, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_kv_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tmem, kmajor_desc(sQ, kk), kmajor_desc(sK0, kk), IDESC_KK, kk > 0);
        mma_commit(bar_s);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tmem + 128, kmajor_desc(sdO, kk), kmajor_desc(sK0 + TILE_BYTES, kk), IDESC_KK, kk > 0);
        mma_commit(bar_dp);
      }
      for (int i = 0; i < nsteps && ok; ++i) {
        const int s = i & 1;
        const uint32_t cK = sK0 + s * 2 * TILE_BYTES;
        const uint32_t nK = sK0 + (s ^ 1) * 2 * TILE_BYTES, nV = nK + TILE_BYTES;
        if (i + 1 < nsteps) {   // S of the next key tile into the other S buffer
          ok = mbar_wait_abortable(bar_kv_full + 8 * (s ^ 1), ((i + 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) mma_ss(tmem + s_col(i + 1), kmajor_desc(sQ, kk), kmajor_desc(nK, kk), IDESC_KK, kk > 0);
          mma_commit(bar_s + 8 * (s ^ 1));
        }
        // dQ += dS_i K_i   (dS: bf16 pairs at columns [0,32) and [64,96) of this step's S buffer)
        ok = mbar_wait_abortable(bar_ds, i & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tmem + 256, tmem + s_col(i) + (kk < 4 ? kk * 8 : 64 + (kk - 4) * 8), mnmajor_desc(cK, kk), IDESC_KM, (i > 0 || kk > 0) ? 1u : 0u);
        mma_commit(bar_kv_empty + 8 * s);
        if (i + 1 < nsteps) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) mma_ss(tmem + 128, kmajor_desc(sdO, kk), kmajor_desc(nV, kk), IDESC_KK, kk > 0);
          mma_commit(bar_dp);
        }
      }
      mma_commit(bar_done);
    }
  } else {
    const int w = warp >> 2;
    const int r = (warp & 3) * 32 + lane;
    const int row = q0 + r;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = w * 64;
    float lse2 = INFINITY, dsum = 0.f;
    {
      const float z = a.lse[qs][((int64_t)b * a.H + h) * L + row];
      if (isfinite(z)) lse2 = z * LOG2E;
      dsum = a.dsum[qs][((int64_t)b * a.H + h) * L + row];
    }
    int rlo[2], rhi[2];
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) visible_interval(qs, ks, row, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, rlo[ks], rhi[ks]);
    bool ok = true;
    for (int i = 0; i < nsteps; ++i) {
      const int ks = tile_ks(i), k0 = tile_k0(i);
      ok = mbar_wait_abortable(bar_s + 8 * (i & 1), (i >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t ts = tl + s_col(i) + c0;
      uint32_t x[64];
      {
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(x);
        tmem_ld32(ts, c[0]); tmem_ld32(ts + 32, c[1]);
        tmem_wait_ld();
      }
      const bool need_mask = (k0 < lo_last[ks]) || (k0 + TILE > hi_first[ks]);
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        float p = exp2f(__uint_as_float(x[c]) * a.scale_log2 - lse2);
        if (need_mask) { const int jj = k0 + c0 + c; p = (jj >= rlo[ks] && jj < rhi[ks]) ? p : 0.f; }
        x[c] = __float_as_uint(p);
      }
      ok = mbar_wait_abortable(bar_dp, i & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      {
        uint32_t y[64];
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(y);
        tmem_ld32(tl + 128 + c0, c[0]); tmem_ld32(tl + 128 + c0 + 32, c[1]);
        tmem_wait_ld();
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float d0 = __uint_as_float(x[2 * e]) * (__uint_as_float(y[2 * e]) - dsum);
          const float d1 = __uint_as_float(x[2 * e + 1]) * (__uint_as_float(y[2 * e + 1]) - dsum);
          pk[e] = pack_bf16(d0, d1);
        }
        tmem_st32(ts, pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_ds);
    }
    if (ok && nsteps > 0) {
      ok = mbar_wait_abortable(bar_done, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      bf16* dst = a.dq[qs] + (((int64_t)b * L + row) * a.H + h) * 128 + c0;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        if (nsteps > 0) { tmem_ld32(tl + 256 + c0 + c * 32, v); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        store_row_chunk(dst + c * 32, v, a.scale);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tmem, 512);
}

}  // namespace

bool tc_bwd_supported(const KArgs& a) {
  return a.d == 128 && a.L % TILE == 0 && tc_encoder_available();
}
size_t tc_bwd_extra_workspace(const bdlm_params*) { return 0; }

cudaError_t launch_tc_bwd(const KArgs& a, void*, int passes, cudaStream_t st) {
  BwdMaps maps;
  for (int s = 0; s < 2; ++s) {
    if (!tc_make_map(&maps.q[s], a.q[s], a.H, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.dout[s], a.dout[s], a.H, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.k[s], a.k[s], a.Hkv, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.v[s], a.v[s], a.Hkv, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
  }
  int* status = device_status_ptr();
  if (status == nullptr) return cudaErrorUnknown;
  cudaError_t e;
  if (passes & BDLM_BWD_PASS_DKDV) {
    if ((e = cudaFuncSetAttribute(tc_dkdv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DKDV_SMEM)) != cudaSuccess) return e;
    dim3 grid(a.L / TILE, a.Hkv, a.batch * 2);
    tc_dkdv_kernel<<<grid, BWD_THREADS, DKDV_SMEM, st>>>(maps, a, status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (passes & BDLM_BWD_PASS_DQ) {
    if ((e = cudaFuncSetAttribute(tc_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM)) != cudaSuccess) return e;
    dim3 grid(a.L / TILE, a.H, a.batch * 2);
    tc_dq_kernel<<<grid, BWD_THREADS, DQ_SMEM, st>>>(maps, a, status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace bdlm
