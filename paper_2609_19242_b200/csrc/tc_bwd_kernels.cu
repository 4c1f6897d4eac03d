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
//   fused       the dK/dV unit with 64-query steps: the same CTA also forms dQ^T = K^T dS^T per step and a
//               fourth warpgroup adds it into an fp32 dQ accumulator through TMA bulk reductions
//               (5 GEMMs per pair instead of 7; selected with bwd_single_pass).
//
// All are warp-specialised: warp 8 issues TMA loads, warp 9 issues tcgen05.mma (the whole warp walks the
// loop convergently, one elected lane issues), warps 0-7 (two warpgroups, each owning half of the 128
// score columns of every TMEM lane) recompute P = exp(S - LSE) and dS = P * (dP - D) and hand them back
// to the tensor core (dS as a TMEM-resident A operand; P^T of the dK/dV pass through a shared-memory tile).
// Every wait is bounded and abortable.
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
// B MN-major (a [k][n] tile as loaded) with N = the head dimension
__host__ __device__ constexpr uint32_t idesc_km(int d) { return make_idesc(128, d, false, true); }

// One operand tile of head `head`: D / 64 panels of 64 columns (D = head dimension, 128 or 64).
template <int D>
__device__ __forceinline__ void tma_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int head, int row0, int b) {
  tma_load_3d(dst, map, bar, head * D, row0, b);
  if (D == 128) tma_load_3d(dst + PANEL_BYTES, map, bar, head * D + 64, row0, b);
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
// Shared memory: K, V (resident), a 2-stage Q ring, a 2-stage dO ring with the LSE and D rows of
// the same query tile, and one tile for P^T.  P^T goes to the tensor core through shared memory
// rather than through the S^T columns of tensor memory: the S^T columns are then free as soon as
// the compute warps hold S^T(i) in registers, so S^T(i+1) is computed while exp(i) runs, and the
// compute warps never wait for the tensor core in steady state.
constexpr int DKDV_Q0 = 2 * TILE_BYTES;
constexpr int DKDV_DO0 = 4 * TILE_BYTES;
constexpr int DKDV_P = 6 * TILE_BYTES;
constexpr int DKDV_ARR = 7 * TILE_BYTES;            // lse_s[2][128], d_s[2][128]
constexpr int DKDV_BARS = DKDV_ARR + 2048;
constexpr int DKDV_SMEM = DKDV_BARS + 176;
constexpr int DKDV_NWG = 2;                          // compute warpgroups; each owns 128 / NWG query columns of every key row
constexpr int DKDV_CW = 128 / DKDV_NWG;
constexpr int DKDV_THREADS = (4 * DKDV_NWG + 2) * 32;
constexpr int DKDV_PRODUCER = 4 * DKDV_NWG, DKDV_ISSUER = 4 * DKDV_NWG + 1;

struct QStep { int qs, h, q0; };

// The steps of a key tile: every (query tile, query stream, head of the group) that sees it.  Segment A holds the
// clean query tiles [a0, a1) (for a noisy key tile: the noisy ones), segment B the noisy query tiles [b0, b1) of a
// clean key tile, both in units of the step's query rows.  Segment A is walked first, then segment B, each from its
// last query tile down with all heads of the group inside a tile: CTAs that start together then meet the same
// Q / dO tiles -- and, in the fused kernel, the same dQ accumulator tiles -- at the same time, so that those stay in
// L2 between the CTAs that share them.  (Alternating the two streams tile by tile as well was measured and is
// slower: 4.7 against 3.3 ms on the sliding-window workload.)  Counters only, no division; the order is fixed, so
// dK / dV stay bitwise reproducible.
struct StepWalk {
  int a0, a1, b0, b1, G, h_first, qs_a, rows;
  int t, seg, hh;
  __device__ __forceinline__ int count() const { return ((a1 - a0) + (b1 - b0)) * G; }
  __device__ __forceinline__ void init(int a0_, int na, int b0_, int nb, int G_, int h_first_, int qs_a_, int rows_) {
    a0 = a0_; a1 = a0_ + na; b0 = b0_; b1 = b0_ + nb; G = G_; h_first = h_first_; qs_a = qs_a_; rows = rows_;
    hh = 0;
    if (a1 > a0) { seg = 0; t = a1 - 1; } else { seg = 1; t = b1 - 1; }
  }
  __device__ __forceinline__ QStep cur() const {
    QStep s;
    s.h = h_first + hh; s.qs = seg == 0 ? qs_a : NOISY; s.q0 = t * rows;
    return s;
  }
  __device__ __forceinline__ void next() {
    if (++hh < G) return;
    hh = 0;
    --t;
    if (seg == 0 && t < a0) { seg = 1; t = b1 - 1; }
  }
};

template <bool TR, int D>
__global__ void __launch_bounds__(DKDV_THREADS, 1)
tc_dkdv_kernel(const __grid_constant__ BwdMaps maps, const KArgs a, const TileGrid tg, int* __restrict__ status) {
  constexpr uint32_t IDESC_KM = idesc_km(D);
  constexpr int OPER_BYTES = TILE_BYTES * D / 128;   // bytes TMA delivers per operand tile (D = 64: one panel)
  extern __shared__ __align__(1024) uint8_t sm[];
  const uint32_t base = smem_u32(sm);
  const uint32_t sK = base, sV = base + TILE_BYTES, sQ0 = base + DKDV_Q0, sdO0 = base + DKDV_DO0, sP = base + DKDV_P;
  float* lse_s = reinterpret_cast<float*>(sm + DKDV_ARR);          // [2][128], log2 units
  float* d_s = lse_s + 256;                                        // [2][128]
  const uint32_t bars = base + DKDV_BARS;
  const uint32_t bar_kv = bars, bar_q_full = bars + 8 /*[2]*/, bar_q_empty = bars + 24 /*[2]*/,
                 bar_do_full = bars + 40 /*[2]*/, bar_do_empty = bars + 56 /*[2]*/,
                 bar_st = bars + 72, bar_sfree = bars + 80, bar_dpt = bars + 88, bar_pt = bars + 96,
                 bar_pfree = bars + 104, bar_dst = bars + 112, bar_done = bars + 120;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + DKDV_BARS + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + DKDV_BARS + 136);

  int bx, by, bz;
  tile_grid_decode(tg, bx, by, bz);
  const int ks = bz & 1, b = bz >> 1, hk = by;
  const int k0_row = bx * TILE;   // the tile's first key in memory; key tile 0 has the most query tiles: started first
  const int k0 = ks == CLEAN ? clean_key_pos(a, k0_row) : k0_row;   // and its position
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // warp index, provably uniform
  const int L = rows_k(a, ks), M = a.M;   // rows of this stream's K/V tensors
  if (k0_row >= L || a.dk[ks] == nullptr) return;

  // query tiles that see this key tile: segment A (clean queries; noisy ones for a noisy key tile), then
  // segment B (noisy queries of a clean key tile), for each head of the group.  The visible-query interval of
  // a key moves up with the key: the tile's first key gives the lower end, its last key the upper end.
  int tA0 = 0, nA = 0, tB0 = 0, nB = 0;
  if (ks == CLEAN) {
    int lo, hi, tmp;
    if (a.q[CLEAN] != nullptr) {
      visible_queries_of_clean_key(a, CLEAN, k0, lo, tmp);
      visible_queries_of_clean_key(a, CLEAN, k0 + TILE - 1, tmp, hi);
      if (hi > lo) { tA0 = lo / TILE; nA = (hi + TILE - 1) / TILE - tA0; }
    }
    if (a.q[NOISY] != nullptr) {
      visible_queries_of_clean_key(a, NOISY, k0, lo, tmp);
      visible_queries_of_clean_key(a, NOISY, k0 + TILE - 1, tmp, hi);
      if (hi > lo) { tB0 = lo / TILE; nB = (hi + TILE - 1) / TILE - tB0; }
    }
  } else {
    const int lo = (k0 / M) * M, hi = min(L, ((k0 + TILE - 1) / M + 1) * M);
    tA0 = lo / TILE; nA = (hi + TILE - 1) / TILE - tA0;
  }
  // the steps are walked in the same order by every role (see StepWalk)
  StepWalk walk;
  walk.init(tA0, nA, tB0, nB, a.G, hk * a.G, ks == NOISY ? NOISY : CLEAN, TILE);
  const int nsteps = walk.count();
  auto step_cur = [&]() { return walk.cur(); };
  auto step_next = [&]() { walk.next(); };

  if (threadIdx.x == 0) {
    if (base & 1023u) *abort_flag = 1; else *abort_flag = 0;   // swizzled tiles need a 1024-byte aligned base
    mbar_init(bar_kv, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_q_full + 8 * i, 1); mbar_init(bar_q_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_do_full + 8 * i, 2); mbar_init(bar_do_empty + 8 * i, 1 + 4 * DKDV_NWG); }   // full: TMA bytes + LSE/D rows; empty: dV done + every compute warp done with the D rows
    mbar_init(bar_st, 1); mbar_init(bar_dpt, 1); mbar_init(bar_pfree, 1);
    mbar_init(bar_sfree, 128 * DKDV_NWG); mbar_init(bar_pt, 128 * DKDV_NWG); mbar_init(bar_dst, 128 * DKDV_NWG);
    mbar_init(bar_done, 1);
    fence_mbar_init();
  }
  if (warp == DKDV_PRODUCER) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // broadcast: provably warp-uniform
  const bool bad_base = (*abort_flag != 0);
  // TMEM columns: [0,128) S^T   [128,256) dP^T / dS^T   [256,384) dV   [384,512) dK

  if (bad_base) {
    // fall through to the common exit
  } else if (warp == DKDV_PRODUCER) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && nsteps > 0) {   // a key tile no query sees writes zeros and waits for nothing: it must not leave a copy in flight
      mbar_expect_tx(bar_kv, 2 * OPER_BYTES);
      tma_tile<D>(sK, &maps.k[ks], bar_kv, hk, k0_row, b);
      tma_tile<D>(sV, &maps.v[ks], bar_kv, hk, k0_row, b);
    }
    bool ok = true;
    long long w_empty = 0;
    const long long t_begin = tick<TR>();
    // the LSE and D rows of a step are fetched one step ahead, so that the round trip to global memory lies under
    // the waits for the ring stages instead of in front of the stage's full barrier
    auto fetch_rows = [&](const QStep& s, float4& z, float4& dd) {
      const int Lq = rows_q(a, s.qs);
      const int64_t row0 = ((int64_t)b * a.H + s.h) * Lq + s.q0;
      if ((Lq & 3) == 0 && s.q0 + TILE <= Lq) {
        z = reinterpret_cast<const float4*>(a.lse[s.qs] + row0)[lane];
        dd = reinterpret_cast<const float4*>(a.dsum[s.qs] + row0)[lane];
      } else {   // a tile that runs past the end of the tensor (or rows that are not 16-byte aligned): P = 0 and D = 0 there
        float zz[4], ds[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool in = s.q0 + 4 * lane + e < Lq;
          zz[e] = in ? a.lse[s.qs][row0 + 4 * lane + e] : INFINITY;
          ds[e] = in ? a.dsum[s.qs][row0 + 4 * lane + e] : 0.f;
        }
        z = make_float4(zz[0], zz[1], zz[2], zz[3]);
        dd = make_float4(ds[0], ds[1], ds[2], ds[3]);
      }
    };
    float4 z_next = make_float4(0.f, 0.f, 0.f, 0.f), d_next = z_next;
    if (nsteps > 0) fetch_rows(step_cur(), z_next, d_next);
    for (int i = 0; i < nsteps && ok; ++i) {
      const int sd = i & 1;
      const QStep st = step_cur();
      step_next();
      const float4 z = z_next, dd = d_next;
      if (i + 1 < nsteps) fetch_rows(step_cur(), z_next, d_next);
      if (i >= 2) ok = mbar_wait_timed<TR>(bar_q_empty + 8 * sd, ((i >> 1) - 1) & 1, abort_flag, w_empty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(bar_q_full + 8 * sd, OPER_BYTES);
        tma_tile<D>(sQ0 + sd * TILE_BYTES, &maps.q[st.qs], bar_q_full + 8 * sd, st.h, st.q0, b);
      }
      if (i >= 2) ok = mbar_wait_timed<TR>(bar_do_empty + 8 * sd, ((i >> 1) - 1) & 1, abort_flag, w_empty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(bar_do_full + 8 * sd, OPER_BYTES);   // one arrival of two; the LSE/D rows follow
        tma_tile<D>(sdO0 + sd * TILE_BYTES, &maps.dout[st.qs], bar_do_full + 8 * sd, st.h, st.q0, b);
      }
      {
        float4 z2;
        z2.x = isfinite(z.x) ? z.x * LOG2E : INFINITY; z2.y = isfinite(z.y) ? z.y * LOG2E : INFINITY;
        z2.z = isfinite(z.z) ? z.z * LOG2E : INFINITY; z2.w = isfinite(z.w) ? z.w * LOG2E : INFINITY;
        reinterpret_cast<float4*>(lse_s + sd * 128)[lane] = z2;
        reinterpret_cast<float4*>(d_s + sd * 128)[lane] = dd;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_do_full + 8 * sd);
    }
    if (lane == 0) { trace_add(a.trace, 16 + 12, tick<TR>() - t_begin); trace_add(a.trace, 16 + 13, w_empty); }
  } else if (warp == DKDV_ISSUER) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop,
    // one elected lane issues (see elect_one)
    if (nsteps > 0) {
      const uint32_t el = elect_one();
      long long w_pt = 0, w_sf = 0, w_dst = 0;
      const long long t_begin = tick<TR>();
      const uint32_t k_lo = desc_lo_k(sK), v_lo = desc_lo_k(sV), p_lo = desc_lo_k(sP);
      const uint32_t qk_lo0 = desc_lo_k(sQ0), qm_lo0 = desc_lo_mn(sQ0);       // Q ring, as K-major B (S^T) / MN-major B (dK)
      const uint32_t dok_lo0 = desc_lo_k(sdO0), dom_lo0 = desc_lo_mn(sdO0);   // dO ring, as K-major B (dP^T) / MN-major B (dV)
      bool ok = mbar_wait_abortable(bar_kv, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_q_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        gemm_ss_e<D / 16>(tmem, k_lo, qk_lo0, IDESC_KK, 0u, el);
        mma_commit_e(bar_st, el);
      }
      ok = ok && mbar_wait_abortable(bar_do_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        gemm_ss_e<D / 16>(tmem + 128, v_lo, dok_lo0, IDESC_KK, 0u, el);
        mma_commit_e(bar_dpt, el);
      }
      for (int i = 0; i < nsteps && ok; ++i) {
        const int sd = i & 1, sn = sd ^ 1;
        const uint32_t acc = i > 0 ? 1u : 0u;
        // S^T of the next step: its columns are free once every compute thread holds S^T(i) in registers
        if (i + 1 < nsteps) {
          ok = mbar_wait_timed<TR>(bar_sfree, i & 1, abort_flag, w_sf);
          ok = ok && mbar_wait_lean(bar_q_full + 8 * sn, ((i + 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          gemm_ss_e<D / 16>(tmem, k_lo, qk_lo0 + sn * TILE_LO, IDESC_KK, 0u, el);
          mma_commit_e(bar_st, el);
        }
        // dV += P^T dO_i   (P^T from shared memory, K-major: row = key, contraction = query)
        ok = mbar_wait_timed<TR>(bar_pt, i & 1, abort_flag, w_pt);
        if (!ok) break;
        tc_fence_after();
        gemm_ss_km_e(tmem + 256, p_lo, dom_lo0 + sd * TILE_LO, IDESC_KM, acc, el);
        mma_commit_e(bar_do_empty + 8 * sd, el);
        mma_commit_e(bar_pfree, el);
        // dK += dS^T Q_i   (dS^T: bf16 pairs, each warpgroup's share at the start of its own dP^T columns)
        ok = mbar_wait_timed<TR>(bar_dst, i & 1, abort_flag, w_dst);
        if (!ok) break;
        tc_fence_after();
        gemm_ts_mn_cw_e<DKDV_CW>(tmem + 384, tmem + 128, qm_lo0 + sd * TILE_LO, IDESC_KM, acc, el);
        mma_commit_e(bar_q_empty + 8 * sd, el);
        // dP^T of the next step follows dK in the pipe, so it cannot overwrite dS^T(i) early
        if (i + 1 < nsteps) {
          ok = mbar_wait_lean(bar_do_full + 8 * sn, ((i + 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          gemm_ss_e<D / 16>(tmem + 128, v_lo, dok_lo0 + sn * TILE_LO, IDESC_KK, 0u, el);
          mma_commit_e(bar_dpt, el);
        }
      }
      mma_commit_e(bar_done, el);
      if (lane == 0) {
        trace_add(a.trace, 16 + 8, tick<TR>() - t_begin); trace_add(a.trace, 16 + 9, w_pt);
        trace_add(a.trace, 16 + 10, w_sf); trace_add(a.trace, 16 + 11, w_dst);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warpgroups
    constexpr int CW = DKDV_CW;
    const int w = warp >> 2;                                   // column share: query columns [CW w, CW w + CW)
    const int r = (warp & 3) * 32 + lane;                      // TMEM lane = key row of the tile
    const int j = k0 + r;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = w * CW;
    uint8_t* prow = sm + DKDV_P + (c0 >> 6) * PANEL_BYTES + r * 128;   // this thread's row of the P^T tile (panel of its columns)
    const int pch0 = (c0 & 63) >> 3;                           // its first 16-byte chunk in that row
    // query rows that see key j, per query stream (section 3.2 read from the key's side), and the bounds inside
    // which a query tile needs no masking: every key row of this tile sees all of it.  The visible-query
    // interval is monotone in the key, so the last key's lower end and the first key's upper end decide.
    int vqc_lo = 0, vqc_hi = 0, vqn_lo, vqn_hi, fullc_lo = 0, fullc_hi = 0, fulln_lo, fulln_hi;
    if (ks == CLEAN) {
      int tmp;
      if (a.q[CLEAN] != nullptr) {
        visible_queries_of_clean_key(a, CLEAN, j, vqc_lo, vqc_hi);
        visible_queries_of_clean_key(a, CLEAN, k0 + TILE - 1, fullc_lo, tmp);
        visible_queries_of_clean_key(a, CLEAN, k0, tmp, fullc_hi);
      }
      if (a.q[NOISY] != nullptr) {
        visible_queries_of_clean_key(a, NOISY, j, vqn_lo, vqn_hi);
        visible_queries_of_clean_key(a, NOISY, k0 + TILE - 1, fulln_lo, tmp);
        visible_queries_of_clean_key(a, NOISY, k0, tmp, fulln_hi);
      } else {
        vqn_lo = vqn_hi = fulln_lo = fulln_hi = 0;
      }
    } else {
      vqn_lo = (j / M) * M; vqn_hi = vqn_lo + M;
      fulln_lo = ((k0 + TILE - 1) / M) * M; fulln_hi = (k0 / M) * M + M;
    }
    bool ok = true;
    long long w_st = 0, w_dpt = 0, w_pf = 0, c_exp = 0, c_ds = 0, c_ld = 0, c_math = 0;
    const long long t_begin = tick<TR>();
    for (int i = 0; i < nsteps; ++i) {
      const int sd = i & 1;
      const QStep st = step_cur();
      step_next();
      const bool need_mask = (st.qs == CLEAN) ? (st.q0 < fullc_lo || st.q0 + TILE > fullc_hi)
                                              : (st.q0 < fulln_lo || st.q0 + TILE > fulln_hi);
      ok = mbar_wait_timed<TR>(bar_do_full + 8 * sd, (i >> 1) & 1, abort_flag, w_st);
      ok = ok && mbar_wait_timed<TR>(bar_st, i & 1, abort_flag, w_st);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long t0 = tick<TR>();
      uint32_t x[CW];
      {
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(x);
#pragma unroll
        for (int q = 0; q < CW / 32; ++q) tmem_ld32(tl + c0 + 32 * q, c[q]);
        tmem_wait_ld();
      }
      tc_fence_before();
      mbar_arrive(bar_sfree);   // S^T(i) is in registers: the tensor core may overwrite its columns
      const long long t0b = tick<TR>();
      c_ld += t0b - t0;
      const float4* lz4 = reinterpret_cast<const float4*>(lse_s + sd * 128 + c0);
      if (!need_mask) {
#pragma unroll
        for (int c8 = 0; c8 < CW / 8; ++c8) {
          const float4 za = lz4[2 * c8], zb = lz4[2 * c8 + 1];
          float* xf = reinterpret_cast<float*>(x) + 8 * c8;
          xf[0] = exp2f(fmaf(xf[0], a.scale_log2, -za.x));
          xf[1] = exp2f(fmaf(xf[1], a.scale_log2, -za.y));
          xf[2] = exp2f(fmaf(xf[2], a.scale_log2, -za.z));
          xf[3] = exp2f(fmaf(xf[3], a.scale_log2, -za.w));
          xf[4] = exp2f(fmaf(xf[4], a.scale_log2, -zb.x));
          xf[5] = exp2f(fmaf(xf[5], a.scale_log2, -zb.y));
          xf[6] = exp2f(fmaf(xf[6], a.scale_log2, -zb.z));
          xf[7] = exp2f(fmaf(xf[7], a.scale_log2, -zb.w));
        }
      } else {
        // visible columns of this thread's key row inside the tile: [vlo, vhi)
        const int vlo = (st.qs == CLEAN ? vqc_lo : vqn_lo) - st.q0 - c0, vhi = (st.qs == CLEAN ? vqc_hi : vqn_hi) - st.q0 - c0;
#pragma unroll
        for (int c4 = 0; c4 < CW / 4; ++c4) {
          const float4 z = lz4[c4];
          const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = 4 * c4 + e;
            const float p = exp2f(fmaf(__uint_as_float(x[c]), a.scale_log2, -zz[e]));
            x[c] = __float_as_uint((c >= vlo && c < vhi) ? p : 0.f);
          }
        }
      }
      c_math += tick<TR>() - t0b;
      // P^T(i) as bf16 into the shared-memory tile, once dV(i-1) has finished reading P^T(i-1)
      if (i > 0) {
        ok = mbar_wait_timed<TR>(bar_pfree, (i - 1) & 1, abort_flag, w_pf);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
#pragma unroll
      for (int c8 = 0; c8 < CW / 8; ++c8) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(x[c8 * 8 + 0]), __uint_as_float(x[c8 * 8 + 1]));
        v.y = pack_bf16(__uint_as_float(x[c8 * 8 + 2]), __uint_as_float(x[c8 * 8 + 3]));
        v.z = pack_bf16(__uint_as_float(x[c8 * 8 + 4]), __uint_as_float(x[c8 * 8 + 5]));
        v.w = pack_bf16(__uint_as_float(x[c8 * 8 + 6]), __uint_as_float(x[c8 * 8 + 7]));
        *reinterpret_cast<uint4*>(prow + (((pch0 + c8) ^ (r & 7)) << 4)) = v;
      }
      fence_async_smem();
      mbar_arrive(bar_pt);
      const long long t1 = tick<TR>();
      c_exp += t1 - t0;

      ok = mbar_wait_timed<TR>(bar_dpt, i & 1, abort_flag, w_dpt);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long t2 = tick<TR>();
      {
        uint32_t y[CW];
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(y);
#pragma unroll
        for (int q = 0; q < CW / 32; ++q) tmem_ld32(tl + 128 + c0 + 32 * q, c[q]);
        tmem_wait_ld();
        const float4* dz4 = reinterpret_cast<const float4*>(d_s + sd * 128 + c0);
        uint32_t pk[CW / 2];
#pragma unroll
        for (int c4 = 0; c4 < CW / 4; ++c4) {
          const float4 dd = dz4[c4];
          const float d0 = __uint_as_float(x[4 * c4 + 0]) * (__uint_as_float(y[4 * c4 + 0]) - dd.x);
          const float d1 = __uint_as_float(x[4 * c4 + 1]) * (__uint_as_float(y[4 * c4 + 1]) - dd.y);
          const float d2 = __uint_as_float(x[4 * c4 + 2]) * (__uint_as_float(y[4 * c4 + 2]) - dd.z);
          const float d3 = __uint_as_float(x[4 * c4 + 3]) * (__uint_as_float(y[4 * c4 + 3]) - dd.w);
          pk[2 * c4] = pack_bf16(d0, d1);
          pk[2 * c4 + 1] = pack_bf16(d2, d3);
        }
        if constexpr (CW == 64) tmem_st32(tl + 128 + c0, reinterpret_cast<uint32_t (&)[32]>(pk));
        else tmem_st16(tl + 128 + c0, reinterpret_cast<uint32_t (&)[16]>(pk));
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_dst);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_do_empty + 8 * sd);   // this warp is done with the stage's D rows
      c_ds += tick<TR>() - t2;
    }
    if (warp == 0 && lane == 0) {
      trace_add(a.trace, 16 + 0, nsteps); trace_add(a.trace, 16 + 1, w_st); trace_add(a.trace, 16 + 2, w_dpt);
      trace_add(a.trace, 16 + 3, w_pf); trace_add(a.trace, 16 + 4, c_exp); trace_add(a.trace, 16 + 5, c_ds);
      trace_add(a.trace, 16 + 6, tick<TR>() - t_begin);
      trace_add(a.trace, 16 + 14, c_ld); trace_add(a.trace, 16 + 15, c_math);
    }
    // epilogue: the 256 accumulator columns (dV, then dK) are shared out evenly over the warpgroups
    if (ok && nsteps > 0) {
      ok = mbar_wait_abortable(bar_done, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      constexpr int EW = 256 / DKDV_NWG;                       // accumulator columns per thread
      const int acol = w * EW;                                 // first of them, in [0, 256)
      const bool is_dk = acol >= 128;
      bf16* dst = (is_dk ? a.dk[ks] : a.dv[ks]) + (((int64_t)b * L + k0_row + r) * a.Hkv + hk) * D + (acol & 127);
      const float sc = is_dk ? a.scale : 1.f;
      static_assert(EW == 128, "one warpgroup per accumulator");
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        if (nsteps > 0) { tmem_ld32(tl + 256 + acol + c * 32, v); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        if (k0_row + r < L) store_row_chunk(dst + c * 32, v, sc);   // key rows past the end of the tensor are not written
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == DKDV_PRODUCER) tmem_dealloc(tmem, 512);
}

// =============================================================================================
// dQ pass
// =============================================================================================
// Q and dO of the CTA's query tile are copied once from shared memory into tensor memory (bf16
// pairs, one row per lane) and serve as TMEM-resident A operands, so S = Q K^T and dP = dO V^T
// read only K / V from shared memory.  Shared memory: Q, dO staging, a 3-stage K ring (a K tile
// is read first by S and last by dQ) and a 2-stage V ring.
constexpr int DQ_K0 = 2 * TILE_BYTES;
constexpr int DQ_V0 = 5 * TILE_BYTES;
constexpr int DQ_BARS = 7 * TILE_BYTES;
constexpr int DQ_SMEM = DQ_BARS + 192;

// Copy row `r` of a swizzled [128 x 128] bf16 tile into 64 TMEM columns (this thread's lane).
template <int D>
__device__ __forceinline__ void row_smem_to_tmem(const uint8_t* tile, int r, uint32_t taddr) {
#pragma unroll
  for (int half = 0; half < D / 64; ++half) {
    uint32_t v[32];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint4 u = *reinterpret_cast<const uint4*>(tile + half * PANEL_BYTES + r * 128 + ((c ^ (r & 7)) << 4));
      v[4 * c] = u.x; v[4 * c + 1] = u.y; v[4 * c + 2] = u.z; v[4 * c + 3] = u.w;
    }
    tmem_st32(taddr + half * 32, v);
  }
}

template <bool TR, int D>
__global__ void __launch_bounds__(BWD_THREADS, 1)
tc_dq_kernel(const __grid_constant__ BwdMaps maps, const KArgs a, const TileGrid tg, int* __restrict__ status) {
  constexpr uint32_t IDESC_KM = idesc_km(D);
  constexpr int OPER_BYTES = TILE_BYTES * D / 128;
  extern __shared__ __align__(1024) uint8_t sm[];
  const uint32_t base = smem_u32(sm);
  const uint32_t sQ = base, sdO = base + TILE_BYTES, sK0 = base + DQ_K0, sV0 = base + DQ_V0;
  const uint32_t bars = base + DQ_BARS;
  const uint32_t bar_qdo = bars, bar_k_full = bars + 8 /*[3]*/, bar_k_empty = bars + 32 /*[3]*/,
                 bar_v_full = bars + 56 /*[2]*/, bar_v_empty = bars + 72 /*[2]*/,
                 bar_s = bars + 88, bar_sfree = bars + 96, bar_dp = bars + 104, bar_ds = bars + 112,
                 bar_done = bars + 120, bar_aready = bars + 128;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + DQ_BARS + 144);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + DQ_BARS + 152);

  int bx, by, bz;
  tile_grid_decode(tg, bx, by, bz);
  const int qs = bz & 1, b = bz >> 1, h = by, hk = h / a.G;
  const int q0 = (tg.nx - 1 - bx) * TILE;
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // warp index, provably uniform
  if (a.q[qs] == nullptr) return;
  const int L = rows_q(a, qs);   // rows of this stream's query tensors
  if (q0 >= L) return;

  // key tiles visible from this query tile: clean segment, then noisy segment
  int lo0, lo1, nt0, nt1, lo_last0, lo_last1, hi_first0, hi_first1;
  {
    int lo_f, hi_f, lo_l, hi_l;
    visible_interval(a, qs, 0, q0, lo_f, hi_f);
    const int q_last = min(q0 + TILE, L) - 1;
    visible_interval(a, qs, 0, q_last, lo_l, hi_l);
    lo0 = lo_f; lo_last0 = lo_l; hi_first0 = hi_f; nt0 = hi_l > lo_f ? (hi_l - lo_f + TILE - 1) / TILE : 0;
    visible_interval(a, qs, 1, q0, lo_f, hi_f);
    visible_interval(a, qs, 1, q_last, lo_l, hi_l);
    lo1 = lo_f; lo_last1 = lo_l; hi_first1 = hi_f; nt1 = hi_l > lo_f ? (hi_l - lo_f + TILE - 1) / TILE : 0;
  }
  const int nsteps = nt0 + nt1;
  auto tile_ks = [&](int i) { return i < nt0 ? 0 : 1; };
  auto tile_k0 = [&](int i) { return i < nt0 ? lo0 + i * TILE : lo1 + (i - nt0) * TILE; };

  if (threadIdx.x == 0) {
    if (base & 1023u) *abort_flag = 1; else *abort_flag = 0;
    mbar_init(bar_qdo, 1);
    for (int i = 0; i < 3; ++i) { mbar_init(bar_k_full + 8 * i, 1); mbar_init(bar_k_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_v_full + 8 * i, 1); mbar_init(bar_v_empty + 8 * i, 1); }
    mbar_init(bar_s, 1); mbar_init(bar_sfree, 256);
    mbar_init(bar_dp, 1); mbar_init(bar_ds, 256); mbar_init(bar_done, 1); mbar_init(bar_aready, 256);
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // broadcast: provably warp-uniform
  const bool bad_base = (*abort_flag != 0);
  // TMEM columns: [0,64) Q (bf16 pairs)  [64,128) dO (bf16 pairs)  [128,256) S  [256,384) dP / dS  [384,512) dQ
  constexpr uint32_t C_Q = 0, C_DO = 64, C_S = 128, C_DP = 256, C_DQ = 384;

  if (bad_base) {
    // fall through to the common exit
  } else if (warp == 8) {
    if (lane == 0 && nsteps > 0) {
      mbar_expect_tx(bar_qdo, 2 * OPER_BYTES);
      tma_tile<D>(sQ, &maps.q[qs], bar_qdo, h, q0, b);
      tma_tile<D>(sdO, &maps.dout[qs], bar_qdo, h, q0, b);
      bool ok = true;
      long long w_empty = 0;
      const long long t_begin = tick<TR>();
      for (int i = 0; i < nsteps && ok; ++i) {
        const int sk = i % 3, sv = i & 1;
        const int ks = tile_ks(i), k0 = tile_k0(i);
        if (i >= 3) ok = mbar_wait_timed<TR>(bar_k_empty + 8 * sk, ((i / 3) - 1) & 1, abort_flag, w_empty);
        if (!ok) break;
        mbar_expect_tx(bar_k_full + 8 * sk, OPER_BYTES);
        const int krow = ks == CLEAN ? clean_key_row(a, k0) : k0;   // where the tile's first key is stored
        tma_tile<D>(sK0 + sk * TILE_BYTES, &maps.k[ks], bar_k_full + 8 * sk, hk, krow, b);
        if (i >= 2) ok = mbar_wait_timed<TR>(bar_v_empty + 8 * sv, ((i >> 1) - 1) & 1, abort_flag, w_empty);
        if (!ok) break;
        mbar_expect_tx(bar_v_full + 8 * sv, OPER_BYTES);
        tma_tile<D>(sV0 + sv * TILE_BYTES, &maps.v[ks], bar_v_full + 8 * sv, hk, krow, b);
      }
      trace_add(a.trace, 32 + 12, tick<TR>() - t_begin); trace_add(a.trace, 32 + 13, w_empty);
    }
  } else if (warp == 9) {
    // the whole warp walks the loop; one elected lane issues (see elect_one)
    if (nsteps > 0) {
      const uint32_t el = elect_one();
      long long w_kv = 0, w_ds = 0, w_sf = 0, t_issue = 0;
      const long long t_begin = tick<TR>();
      const uint32_t kk_lo0 = desc_lo_k(sK0), km_lo0 = desc_lo_mn(sK0);   // K ring as K-major B (S) / MN-major B (dQ)
      const uint32_t vk_lo0 = desc_lo_k(sV0);
      bool ok = mbar_wait_abortable(bar_aready, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_k_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        gemm_ts_e<D / 16>(tmem + C_S, tmem + C_Q, kk_lo0, IDESC_KK, 0u, el);
        mma_commit_e(bar_s, el);
      }
      ok = ok && mbar_wait_abortable(bar_v_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        gemm_ts_e<D / 16>(tmem + C_DP, tmem + C_DO, vk_lo0, IDESC_KK, 0u, el);
        mma_commit_e(bar_dp, el);
        mma_commit_e(bar_v_empty, el);
      }
      int sk = 0;   // i % 3
      for (int i = 0; i < nsteps && ok; ++i) {
        const int nk = (sk == 2) ? 0 : sk + 1;
        if (i + 1 < nsteps) {   // S of the next key tile, once both warpgroups have read S of this one
          ok = mbar_wait_timed<TR>(bar_sfree, i & 1, abort_flag, w_sf);
          ok = ok && mbar_wait_timed<TR>(bar_k_full + 8 * nk, ((i + 1) / 3) & 1, abort_flag, w_kv);
          if (!ok) break;
          tc_fence_after();
          const long long g0 = tick<TR>();
          gemm_ts_e<D / 16>(tmem + C_S, tmem + C_Q, kk_lo0 + nk * TILE_LO, IDESC_KK, 0u, el);
          mma_commit_e(bar_s, el);
          t_issue += tick<TR>() - g0;
        }
        // dQ += dS_i K_i   (dS: bf16 pairs at columns [0,32) and [64,96) of the dP region)
        ok = mbar_wait_timed<TR>(bar_ds, i & 1, abort_flag, w_ds);
        if (!ok) break;
        tc_fence_after();
        const long long g1 = tick<TR>();
        gemm_ts_mn_cw_e<64>(tmem + C_DQ, tmem + C_DP, km_lo0 + sk * TILE_LO, IDESC_KM, i > 0 ? 1u : 0u, el);
        mma_commit_e(bar_k_empty + 8 * sk, el);
        t_issue += tick<TR>() - g1;
        if (i + 1 < nsteps) {
          const int nv = (i + 1) & 1;
          ok = mbar_wait_timed<TR>(bar_v_full + 8 * nv, ((i + 1) >> 1) & 1, abort_flag, w_kv);
          if (!ok) break;
          tc_fence_after();
          const long long g2 = tick<TR>();
          gemm_ts_e<D / 16>(tmem + C_DP, tmem + C_DO, vk_lo0 + nv * TILE_LO, IDESC_KK, 0u, el);
          mma_commit_e(bar_dp, el);
          mma_commit_e(bar_v_empty + 8 * nv, el);
          t_issue += tick<TR>() - g2;
        }
        sk = nk;
      }
      mma_commit_e(bar_done, el);
      if (lane == 0) {
      trace_add(a.trace, 32 + 8, tick<TR>() - t_begin); trace_add(a.trace, 32 + 9, w_kv); trace_add(a.trace, 32 + 10, w_ds);
      trace_add(a.trace, 32 + 11, w_sf); trace_add(a.trace, 32 + 14, t_issue);
      }
    }
  } else {
    const int w = warp >> 2;
    const int r = (warp & 3) * 32 + lane;
    const int row = q0 + r;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = w * 64;
    const bool row_ok = row < L;   // a row past the end of the tensor: P = 0, nothing read or written
    float lse2 = INFINITY, dsum = 0.f;
    int rlo0 = 0, rhi0 = 0, rlo1 = 0, rhi1 = 0;
    if (row_ok) {
      const float z = a.lse[qs][((int64_t)b * a.H + h) * L + row];
      if (isfinite(z)) lse2 = z * LOG2E;
      dsum = a.dsum[qs][((int64_t)b * a.H + h) * L + row];
      visible_interval(a, qs, 0, row, rlo0, rhi0);
      visible_interval(a, qs, 1, row, rlo1, rhi1);
    }
    bool ok = true;
    long long w_s = 0, w_dp = 0, c_ld = 0, c_exp = 0, c_ds = 0;
    Stopwatch<TR> sw;
    const long long t_begin = tick<TR>();
    if (nsteps > 0) {   // stage the A operands: warpgroup 0 copies Q, warpgroup 1 copies dO
      ok = mbar_wait_abortable(bar_qdo, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        row_smem_to_tmem<D>(sm + (w == 0 ? 0 : TILE_BYTES), r, tl + (w == 0 ? C_Q : C_DO));
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_aready);
      }
    }
    for (int i = 0; i < nsteps && ok; ++i) {
      const int ks = tile_ks(i), k0 = tile_k0(i);
      ok = mbar_wait_timed<TR>(bar_s, i & 1, abort_flag, w_s);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t x[64];
      sw.start();
      {
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(x);
        tmem_ld32(tl + C_S + c0, c[0]); tmem_ld32(tl + C_S + c0 + 32, c[1]);
        tmem_wait_ld();
      }
      tc_fence_before();
      mbar_arrive(bar_sfree);
      sw.lap(c_ld);
      const bool need_mask = (ks == 0 ? (k0 < lo_last0 || k0 + TILE > hi_first0) : (k0 < lo_last1 || k0 + TILE > hi_first1)) ||
                             q0 + TILE > L;
      if (!need_mask) {
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          float* xf = reinterpret_cast<float*>(x) + 8 * c8;
          xf[0] = exp2f(fmaf(xf[0], a.scale_log2, -lse2));
          xf[1] = exp2f(fmaf(xf[1], a.scale_log2, -lse2));
          xf[2] = exp2f(fmaf(xf[2], a.scale_log2, -lse2));
          xf[3] = exp2f(fmaf(xf[3], a.scale_log2, -lse2));
          xf[4] = exp2f(fmaf(xf[4], a.scale_log2, -lse2));
          xf[5] = exp2f(fmaf(xf[5], a.scale_log2, -lse2));
          xf[6] = exp2f(fmaf(xf[6], a.scale_log2, -lse2));
          xf[7] = exp2f(fmaf(xf[7], a.scale_log2, -lse2));
        }
      } else {
        const int vlo = (ks == 0 ? rlo0 : rlo1) - k0 - c0, vhi = (ks == 0 ? rhi0 : rhi1) - k0 - c0;
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          const float p = exp2f(fmaf(__uint_as_float(x[c]), a.scale_log2, -lse2));
          x[c] = __float_as_uint((c >= vlo && c < vhi) ? p : 0.f);
        }
      }
      sw.lap(c_exp);
      ok = mbar_wait_timed<TR>(bar_dp, i & 1, abort_flag, w_dp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      sw.start();
      {
        uint32_t y[64];
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(y);
        tmem_ld32(tl + C_DP + c0, c[0]); tmem_ld32(tl + C_DP + c0 + 32, c[1]);
        tmem_wait_ld();
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float d0 = __uint_as_float(x[2 * e]) * (__uint_as_float(y[2 * e]) - dsum);
          const float d1 = __uint_as_float(x[2 * e + 1]) * (__uint_as_float(y[2 * e + 1]) - dsum);
          pk[e] = pack_bf16(d0, d1);
        }
        tmem_st32(tl + C_DP + c0, pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_ds);
      sw.lap(c_ds);
    }
    if (warp == 0 && lane == 0) {
      trace_add(a.trace, 32 + 0, nsteps); trace_add(a.trace, 32 + 1, w_s); trace_add(a.trace, 32 + 2, w_dp);
      trace_add(a.trace, 32 + 6, tick<TR>() - t_begin);
      trace_add(a.trace, 32 + 3, c_ld); trace_add(a.trace, 32 + 4, c_exp); trace_add(a.trace, 32 + 5, c_ds);
    }
    if (ok && nsteps > 0) {
      ok = mbar_wait_abortable(bar_done, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      // each warpgroup writes half of the row's D gradient columns
      constexpr int EC = D / 2;
      bf16* dst = a.dq[qs] + (((int64_t)b * L + row) * a.H + h) * D + w * EC;
#pragma unroll
      for (int c = 0; c < EC / 32; ++c) {
        uint32_t v[32];
        if (nsteps > 0) { tmem_ld32(tl + C_DQ + w * EC + c * 32, v); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        if (row_ok) store_row_chunk(dst + c * 32, v, a.scale);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tmem, 512);
}


// =============================================================================================
// fused backward: one kernel produces dK, dV and dQ
// =============================================================================================
// Same CTA unit as tc_dkdv_kernel (one 128-key tile of one KV head, K and V resident), but a step is the
// key tile against 64 query rows, so that tensor memory also holds a dQ^T tile and shared memory a staging
// area for it: 5 GEMMs and one exp phase per (key tile, query rows) pair instead of the 7 + 2 of the
// two-pass backward.
//   tensor memory  [0,64) S^T / P^T   [64,128) K as bf16 pairs   [128,192) dP^T   [192,256) dQ^T
//                  [256,384) dV   [384,512) dK
//   per step       S^T = K Q^T and dP^T = V dO^T (N = 64).  An N = 64 MMA with both operands in shared memory
//                  asks it for 6 KB per 32 clocks, half as much again as it delivers, so K is also kept in
//                  tensor memory and S^T reads only Q from shared memory.  P^T overwrites its own S^T columns as bf16 pairs
//                  and is the TMEM-resident A operand of dV += P^T dO; dS^T goes to a shared-memory tile
//                  (row = key, 64 queries = 128 bytes), the K-major A operand of dK += dS^T Q and the
//                  MN-major B operand of dQ^T = K^T dS^T (K, resident, is the MN-major A operand).
//   dQ             a fourth warpgroup copies each dQ^T tile (lane = head-dim index, column = query) into a
//                  [64 query x 128] fp32 staging tile, and one of its threads hands it to the TMA engine as
//                  a bulk add-reduction into the fp32 dQ accumulator [batch, H, rows, 128] (32 KB
//                  contiguous).  The compute warps never touch dQ; the reduction runs behind the GEMMs.
// dQ depends on the order in which the key tiles' reductions arrive (fp32 rounding only).
// Shared memory: K, V, a 3-stage Q ring and a 2-stage dO ring of 64-row tiles (+ LSE, D rows, fetched one step
// ahead by the producer), dS^T, 2 dQ staging tiles of 64 query rows: one reduction per step, the next step's tile
// is written while it runs (the engine takes a fixed few hundred clocks per reduction on top of about 25 bytes per
// clock, so one 32 KB operation beats two of 16 KB).
constexpr int HT = 64;                              // query rows per step
constexpr int HPANEL_BYTES = HT * 128;              // one 64-row x 64-column bf16 panel
constexpr int HT_BYTES = 2 * HPANEL_BYTES;          // a [64 x 128] bf16 tile
constexpr int BF_QS = 3;                            // Q ring stages
constexpr int BF_DOS = 2;                           // dO ring stages
constexpr int STG_BYTES = HT * 128 * 4;             // a [64 query x 128] fp32 staging tile
constexpr int BF_Q0 = 2 * TILE_BYTES;
constexpr int BF_DO0 = BF_Q0 + BF_QS * HT_BYTES;
constexpr int BF_DS = BF_DO0 + BF_DOS * HT_BYTES;
constexpr int BF_STG = BF_DS + PANEL_BYTES;
constexpr int BF_ARR = BF_STG + 2 * STG_BYTES;      // lse_s[4][64], d_s[4][64]: the LSE / D rows have a ring of their own
constexpr int BF_BARS = BF_ARR + 2048;
constexpr int BF_SMEM = BF_BARS + 320;
constexpr int BF_THREADS = 448;                     // warps 0-7 compute, 8 producer, 9 MMA issue, 10-13 dQ read-out
constexpr uint32_t IDESC_N64 = make_idesc(128, 64, false, false);   // S^T, dP^T: A, B K-major, N = 64
constexpr uint32_t IDESC_DQT = make_idesc(128, 64, true, true);     // dQ^T: A, B MN-major, N = 64
constexpr uint32_t HPANEL_LO = HPANEL_BYTES >> 4, HT_LO = HT_BYTES >> 4;
__host__ __device__ constexpr uint32_t koff_h(int kk) { return (kk >> 2) * HPANEL_LO + (kk & 3) * 2; }   // K-major slice of a 64-row tile
__device__ __forceinline__ uint32_t desc_lo_mn_h(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (HPANEL_LO << 16); }

// D = head dimension.  With D = 64 the operand tiles are one panel wide, the contractions over the head dimension take
// four k-slices and dV / dK have 64 columns; dQ^T keeps its 128 lanes (the upper 64 hold nothing of value and land in
// the unused half of the 128-wide fp32 accumulator rows).
template <bool TR, int D>
__global__ void __launch_bounds__(BF_THREADS, 1)
tc_bwdf_kernel(const __grid_constant__ BwdMaps maps, const KArgs a, const TileGrid tg, int* __restrict__ status) {
  constexpr uint32_t IDESC_KM = idesc_km(D);
  constexpr int OPER_BYTES = TILE_BYTES * D / 128, HOPER_BYTES = HT_BYTES * D / 128;   // bytes TMA delivers per 128- / 64-row tile
  extern __shared__ __align__(1024) uint8_t sm[];
  const uint32_t base = smem_u32(sm);
  const uint32_t sK = base, sV = base + TILE_BYTES, sQ0 = base + BF_Q0, sdO0 = base + BF_DO0, sDS = base + BF_DS,
                 sSTG = base + BF_STG;
  float* lse_s = reinterpret_cast<float*>(sm + BF_ARR);            // [4][64], log2 units
  float* d_s = lse_s + 256;                                        // [4][64]
  const uint32_t bars = base + BF_BARS;
  const uint32_t bar_kv = bars, bar_q_full = bars + 8 /*[4]*/, bar_q_empty = bars + 40 /*[4]*/,
                 bar_do_full = bars + 72 /*[3]*/, bar_do_empty = bars + 96 /*[3]*/,
                 bar_st = bars + 120, bar_kready = bars + 128, bar_pt = bars + 136, bar_dpt = bars + 152, bar_dpfree = bars + 160,
                 bar_dst = bars + 168, bar_dsfree = bars + 176, bar_dqf = bars + 184, bar_dqr = bars + 192,
                 bar_done = bars + 200, bar_rows_full = bars + 224 /*[4]*/, bar_rows_empty = bars + 256 /*[4]*/;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + BF_BARS + 208);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + BF_BARS + 216);

  int bx, by, bz;
  tile_grid_decode(tg, bx, by, bz);
  const int ks = bz & 1, b = bz >> 1, hk = by;
  const int k0_row = bx * TILE;   // the tile's first key in memory; key tile 0 has the most query tiles: started first
  const int k0 = ks == CLEAN ? clean_key_pos(a, k0_row) : k0_row;   // and its position
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // warp index, provably uniform
  const int L = rows_k(a, ks), M = a.M;
  if (k0_row >= L || a.dk[ks] == nullptr) return;

  // 64-row query tiles that see this key tile: segment A (clean queries; noisy ones for a noisy key tile),
  // then segment B (noisy queries of a clean key tile), for each head of the group
  int tA0 = 0, nA = 0, tB0 = 0, nB = 0;
  if (ks == CLEAN) {
    int lo, hi, tmp;
    if (a.q[CLEAN] != nullptr) {
      visible_queries_of_clean_key(a, CLEAN, k0, lo, tmp);
      visible_queries_of_clean_key(a, CLEAN, k0 + TILE - 1, tmp, hi);
      if (hi > lo) { tA0 = lo / HT; nA = (hi + HT - 1) / HT - tA0; }
    }
    if (a.q[NOISY] != nullptr) {
      visible_queries_of_clean_key(a, NOISY, k0, lo, tmp);
      visible_queries_of_clean_key(a, NOISY, k0 + TILE - 1, tmp, hi);
      if (hi > lo) { tB0 = lo / HT; nB = (hi + HT - 1) / HT - tB0; }
    }
  } else {
    const int lo = (k0 / M) * M, hi = min(L, ((k0 + TILE - 1) / M + 1) * M);
    tA0 = lo / HT; nA = (hi + HT - 1) / HT - tA0;
  }
  StepWalk walk;
  walk.init(tA0, nA, tB0, nB, a.G, hk * a.G, ks == NOISY ? NOISY : CLEAN, HT);
  const int nsteps = walk.count();
  auto step_cur = [&]() { return walk.cur(); };
  auto step_next = [&]() { walk.next(); };

  if (threadIdx.x == 0) {
    if (base & 1023u) *abort_flag = 1; else *abort_flag = 0;   // swizzled tiles need a 1024-byte aligned base
    mbar_init(bar_kv, 1);
    for (int i = 0; i < 4; ++i) { mbar_init(bar_q_full + 8 * i, 1); mbar_init(bar_q_empty + 8 * i, 1); }
    for (int i = 0; i < 3; ++i) { mbar_init(bar_do_full + 8 * i, 1); mbar_init(bar_do_empty + 8 * i, 1); }   // empty: dV done
    for (int i = 0; i < 4; ++i) { mbar_init(bar_rows_full + 8 * i, 1); mbar_init(bar_rows_empty + 8 * i, 8); }   // empty: the 8 compute warps are done with the stage's LSE / D rows
    mbar_init(bar_st, 1); mbar_init(bar_pt, 256); mbar_init(bar_kready, 128);
    mbar_init(bar_dpt, 1); mbar_init(bar_dpfree, 256); mbar_init(bar_dst, 256); mbar_init(bar_dsfree, 1);
    mbar_init(bar_dqf, 1); mbar_init(bar_dqr, 128); mbar_init(bar_done, 1);
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // broadcast: provably warp-uniform
  const bool bad_base = (*abort_flag != 0);

  if (bad_base) {
    // fall through to the common exit
  } else if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && nsteps > 0) {   // a key tile no query sees writes zeros and waits for nothing: it must not leave a copy in flight
      mbar_expect_tx(bar_kv, 2 * OPER_BYTES);
      tma_tile<D>(sK, &maps.k[ks], bar_kv, hk, k0_row, b);
      tma_tile<D>(sV, &maps.v[ks], bar_kv, hk, k0_row, b);
    }
    bool ok = true;
    long long w_empty = 0;
    const long long t_begin = tick<TR>();
    int sd = 0, kd = 0;   // dO ring stage of step i and how many times the ring has wrapped
    // the LSE (lanes 0-15) and D (lanes 16-31) rows of a step are fetched one step ahead, so that the round trip
    // to global memory lies under the waits for the ring stages instead of in front of the stage's full barrier
    auto fetch_rows = [&](const QStep& s) {
      const int Lq = rows_q(a, s.qs);
      const int64_t row0 = ((int64_t)b * a.H + s.h) * Lq + s.q0;
      const float* src = (lane < 16 ? a.lse[s.qs] : a.dsum[s.qs]) + row0;
      if ((Lq & 3) == 0 && s.q0 + HT <= Lq) return reinterpret_cast<const float4*>(src)[lane & 15];
      // a step that runs past the end of the tensor (or rows that are not 16-byte aligned): P = 0 and D = 0 there
      const float fill = lane < 16 ? INFINITY : 0.f;
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = (s.q0 + 4 * (lane & 15) + e < Lq) ? src[4 * (lane & 15) + e] : fill;
      return make_float4(v[0], v[1], v[2], v[3]);
    };
    float4 rows_next = make_float4(0.f, 0.f, 0.f, 0.f);
    if (nsteps > 0) rows_next = fetch_rows(step_cur());
    int sq = 0, kq = 0;   // Q ring stage of step i and its wrap count
    for (int i = 0; i < nsteps && ok; ++i) {
      const QStep st = step_cur();
      step_next();
      const float4 rows = rows_next;
      if (i + 1 < nsteps) rows_next = fetch_rows(step_cur());
      if (kq >= 1) ok = mbar_wait_timed<TR>(bar_q_empty + 8 * sq, (kq - 1) & 1, abort_flag, w_empty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane == 0) {
        const uint32_t dst = sQ0 + sq * HT_BYTES, bar = bar_q_full + 8 * sq;
        mbar_expect_tx(bar, HOPER_BYTES);
        tma_load_3d(dst, &maps.q[st.qs], bar, st.h * D, st.q0, b);
        if (D == 128) tma_load_3d(dst + HPANEL_BYTES, &maps.q[st.qs], bar, st.h * D + 64, st.q0, b);
      }
      if (kd >= 1) ok = mbar_wait_timed<TR>(bar_do_empty + 8 * sd, (kd - 1) & 1, abort_flag, w_empty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane == 0) {
        const uint32_t dst = sdO0 + sd * HT_BYTES, bar = bar_do_full + 8 * sd;
        mbar_expect_tx(bar, HOPER_BYTES);
        tma_load_3d(dst, &maps.dout[st.qs], bar, st.h * D, st.q0, b);
        if (D == 128) tma_load_3d(dst + HPANEL_BYTES, &maps.dout[st.qs], bar, st.h * D + 64, st.q0, b);
      }
      // the rows live in a ring of their own: the dO tile is free again as soon as dV has read it, the D rows
      // only when the compute warps have formed dS
      const int sr = i & 3;
      if (i >= 4) ok = mbar_wait_timed<TR>(bar_rows_empty + 8 * sr, ((i >> 2) - 1) & 1, abort_flag, w_empty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (lane < 16) {
        float4 z2;
        z2.x = isfinite(rows.x) ? rows.x * LOG2E : INFINITY; z2.y = isfinite(rows.y) ? rows.y * LOG2E : INFINITY;
        z2.z = isfinite(rows.z) ? rows.z * LOG2E : INFINITY; z2.w = isfinite(rows.w) ? rows.w * LOG2E : INFINITY;
        reinterpret_cast<float4*>(lse_s + sr * 64)[lane] = z2;
      } else {
        reinterpret_cast<float4*>(d_s + sr * 64)[lane - 16] = rows;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_rows_full + 8 * sr);
      if (++sd == BF_DOS) { sd = 0; ++kd; }
      if (++sq == BF_QS) { sq = 0; ++kq; }
    }
    if (lane == 0) trace_add(a.trace, 16 + 13, w_empty);
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop,
    // one elected lane issues (see elect_one)
    if (nsteps > 0) {
      const uint32_t el = elect_one();
      long long w_pt = 0, w_dpf = 0, w_dst = 0, w_q = 0, w_do = 0;
      const long long t_begin = tick<TR>();
      const uint32_t k_lo = desc_lo_k(sK), v_lo = desc_lo_k(sV), kt_lo = desc_lo_mn(sK);
      const uint32_t qk_lo0 = desc_lo_k(sQ0), qm_lo0 = desc_lo_mn_h(sQ0);       // Q ring, as K-major B (S^T) / MN-major B (dK)
      const uint32_t dok_lo0 = desc_lo_k(sdO0), dom_lo0 = desc_lo_mn_h(sdO0);   // dO ring, as K-major B (dP^T) / MN-major B (dV)
      const uint32_t dsk_lo = desc_lo_k(sDS), dsm_lo = desc_lo_k(sDS);          // dS^T: K-major A (dK) / MN-major B with one 64-query group (dQ^T)
      auto issue_st = [&](int sq) {     // S^T = K Q^T, K from tensor memory
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          mma_ts_e(tmem, tmem + 64 + kk * 8, desc64(qk_lo0 + sq * HT_LO + koff_h(kk)), IDESC_N64, kk == 0 ? 0u : 1u, el);
        mma_commit_e(bar_st, el);
      };
      auto issue_dpt = [&](int sd) {             // dP^T = V dO^T
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          mma_ss_e(tmem + 128, desc64(v_lo + koff(kk)), desc64(dok_lo0 + sd * HT_LO + koff_h(kk)), IDESC_N64, kk == 0 ? 0u : 1u, el);
        mma_commit_e(bar_dpt, el);
      };
      bool ok = mbar_wait_abortable(bar_kv, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_kready, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_q_full, 0, abort_flag);
      if (ok) { tc_fence_after(); issue_st(0); }
      ok = ok && mbar_wait_abortable(bar_do_full, 0, abort_flag);
      if (ok) { tc_fence_after(); issue_dpt(0); }
      int sd = 0, sn = 1 % BF_DOS, kn = 1 / BF_DOS;   // dO ring stage of step i, of step i + 1, and that one's wrap count
      int sq = 0, sqn = 1 % BF_QS, kqn = 1 / BF_QS;   // Q ring stage of step i, of step i + 1, and that one's wrap count
      for (int i = 0; i < nsteps && ok; ++i) {
        const uint32_t acc = i > 0 ? 1u : 0u;
        // dV += P^T dO_i   (P^T: bf16 pairs at the start of each warpgroup's 32 S^T columns)
        ok = mbar_wait_timed<TR>(bar_pt, i & 1, abort_flag, w_pt);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_e(tmem + 256, tmem + (kk >> 1) * 32 + (kk & 1) * 8, desc64(dom_lo0 + sd * HT_LO + moff(kk)), IDESC_KM,
                   kk == 0 ? acc : 1u, el);
        mma_commit_e(bar_do_empty + 8 * sd, el);
        // S^T of the next step over P^T(i): its reader, dV(i), is ahead in the pipe
        if (i + 1 < nsteps) {
          ok = mbar_wait_timed<TR>(bar_q_full + 8 * sqn, kqn & 1, abort_flag, w_q);
          if (!ok) break;
          tc_fence_after();
          issue_st(sqn);
        }
        // dP^T of the next step, once every compute thread holds dP^T(i) in registers -- now, if its dO tile has
        // landed; after dQ^T and dK otherwise (a late load does not hold up the GEMMs that are ready)
        bool dpt_due = i + 1 < nsteps;
        if (dpt_due && mbar_try_wait(bar_dpfree, i & 1) && mbar_try_wait(bar_do_full + 8 * sn, kn & 1)) {
          tc_fence_after();
          issue_dpt(sn);
          dpt_due = false;
        }
        // dQ^T = K^T dS^T (once the read-out warps hold the previous dQ^T), then dK += dS^T Q_i
        ok = mbar_wait_timed<TR>(bar_dst, i & 1, abort_flag, w_dst);
        if (i > 0) ok = ok && mbar_wait_timed<TR>(bar_dqr, (i - 1) & 1, abort_flag, w_dst);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ss_e(tmem + 192, desc64(kt_lo + moff(kk)), desc64(dsm_lo + moff(kk)), IDESC_DQT, kk == 0 ? 0u : 1u, el);
        mma_commit_e(bar_dqf, el);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ss_e(tmem + 384, desc64(dsk_lo + 2 * kk), desc64(qm_lo0 + sq * HT_LO + moff(kk)), IDESC_KM, kk == 0 ? acc : 1u, el);
        mma_commit_e(bar_q_empty + 8 * sq, el);
        mma_commit_e(bar_dsfree, el);
        if (dpt_due) {
          ok = mbar_wait_timed<TR>(bar_dpfree, i & 1, abort_flag, w_dpf);
          ok = ok && mbar_wait_timed<TR>(bar_do_full + 8 * sn, kn & 1, abort_flag, w_do);
          if (!ok) break;
          tc_fence_after();
          issue_dpt(sn);
        }
        sd = sn;
        if (++sn == BF_DOS) { sn = 0; ++kn; }
        sq = sqn;
        if (++sqn == BF_QS) { sqn = 0; ++kqn; }
      }
      mma_commit_e(bar_done, el);
      if (lane == 0) {
        trace_add(a.trace, 16 + 8, tick<TR>() - t_begin); trace_add(a.trace, 16 + 9, w_pt);
        trace_add(a.trace, 16 + 10, w_dpf); trace_add(a.trace, 16 + 11, w_dst);
        trace_add(a.trace, 16 + 7, w_q); trace_add(a.trace, 16 + 12, w_do);
      }
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------------ dQ read-out warpgroup
    const int dd = (warp & 3) * 32 + lane;                      // TMEM lane = head-dim index
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const bool leader = threadIdx.x == 320;
    bool ok = true;
    long long w_dqf = 0, c_ro = 0;
    for (int i = 0; i < nsteps; ++i) {
      const QStep st = step_cur();
      step_next();
      // after a failed wait the warp still meets the others at the named barrier, then all leave together
      if (ok) {
        ok = mbar_wait_timed<TR>(bar_dqf, i & 1, abort_flag, w_dqf);
        ok = __all_sync(0xffffffffu, ok);
      }
      const long long t0 = tick<TR>();
      if (ok) tc_fence_after();
      float* dst = a.dq32[st.qs] + (((int64_t)b * a.H + st.h) * a.dq32_rows[st.qs] + st.q0) * 128;
      uint32_t v[64];
      if (ok) {   // the whole tile into registers first: the tensor core gets its columns back at once
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(v);
        tmem_ld32(tl + 192, c[0]); tmem_ld32(tl + 224, c[1]);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_dqr);
      }
      // staging tile i & 1: the reduction that read it last (two steps ago) must have finished reading it; the one
      // issued for the other tile stays in flight
      if (leader) bulk_wait_read1();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok) {
        float* sg = reinterpret_cast<float*>(sm + BF_STG + (i & 1) * STG_BYTES) + dd;
#pragma unroll
        for (int e = 0; e < HT; ++e) sg[e * 128] = __uint_as_float(v[e]) * a.scale;
        fence_async_smem();
      }
      // the second meeting also takes the decision to leave, for all 128 threads at once (a flag raised between two
      // threads' reads must not send some of them to the exit and the rest to the next meeting)
      uint32_t leave;
      asm volatile(
          "{\n\t.reg .pred p, q;\n\t"
          "setp.ne.b32 q, %1, 0;\n\t"
          "bar.red.or.pred p, 1, 128, q;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(leave) : "r"(*abort_flag) : "memory");
      if (leave) break;
      if (leader) {
        bulk_reduce_add_f32(dst, sSTG + (i & 1) * STG_BYTES, STG_BYTES);
        bulk_commit();
      }
      c_ro += tick<TR>() - t0;
    }
    if (leader) {
      bulk_wait_all();
      trace_add(a.trace, 16 + 14, w_dqf); trace_add(a.trace, 16 + 15, c_ro);
    }
  } else {
    // ------------------------------------------------------------------ compute warpgroups
    const int w = warp >> 2;                                   // column share: query columns [32 w, 32 w + 32) of the step's 64
    const int r = (warp & 3) * 32 + lane;                      // TMEM lane = key row of the tile
    const int j = k0 + r;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = w * 32;
    uint8_t* dsrow = sm + BF_DS + r * 128;                     // this thread's row of the dS^T tile
    // query rows that see key j, per query stream (section 3.2 read from the key's side), and the bounds inside
    // which a step needs no masking: every key row of this tile sees all of its queries
    int vqc_lo = 0, vqc_hi = 0, vqn_lo, vqn_hi, fullc_lo = 0, fullc_hi = 0, fulln_lo, fulln_hi;
    if (ks == CLEAN) {
      int tmp;
      if (a.q[CLEAN] != nullptr) {
        visible_queries_of_clean_key(a, CLEAN, j, vqc_lo, vqc_hi);
        visible_queries_of_clean_key(a, CLEAN, k0 + TILE - 1, fullc_lo, tmp);
        visible_queries_of_clean_key(a, CLEAN, k0, tmp, fullc_hi);
      }
      if (a.q[NOISY] != nullptr) {
        visible_queries_of_clean_key(a, NOISY, j, vqn_lo, vqn_hi);
        visible_queries_of_clean_key(a, NOISY, k0 + TILE - 1, fulln_lo, tmp);
        visible_queries_of_clean_key(a, NOISY, k0, tmp, fulln_hi);
      } else {
        vqn_lo = vqn_hi = fulln_lo = fulln_hi = 0;
      }
    } else {
      vqn_lo = (j / M) * M; vqn_hi = vqn_lo + M;
      fulln_lo = ((k0 + TILE - 1) / M) * M; fulln_hi = (k0 / M) * M + M;
    }
    bool ok = true;
    long long w_st = 0, w_dpt = 0, w_dsf = 0, c_exp = 0, c_ds = 0;
    const long long t_begin = tick<TR>();
    if (w == 0 && nsteps > 0) {   // warpgroup 0 copies K into tensor memory (one key row per lane)
      ok = mbar_wait_abortable(bar_kv, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        row_smem_to_tmem<D>(sm, r, tl + 64);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_kready);
      }
    }
    for (int i = 0; i < nsteps && ok; ++i) {
      const QStep st = step_cur();
      step_next();
      const bool need_mask = (st.qs == CLEAN) ? (st.q0 < fullc_lo || st.q0 + HT > fullc_hi)
                                              : (st.q0 < fulln_lo || st.q0 + HT > fulln_hi);
      const int sr = i & 3;
      ok = mbar_wait_timed<TR>(bar_rows_full + 8 * sr, (i >> 2) & 1, abort_flag, w_st);
      ok = ok && mbar_wait_timed<TR>(bar_st, i & 1, abort_flag, w_st);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long t0 = tick<TR>();
      uint32_t x[32];
      tmem_ld32(tl + c0, x);
      tmem_wait_ld();
      const float4* lz4 = reinterpret_cast<const float4*>(lse_s + sr * 64 + c0);
      if (!need_mask) {
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 z = lz4[c4];
          float* xf = reinterpret_cast<float*>(x) + 4 * c4;
          xf[0] = exp2f(fmaf(xf[0], a.scale_log2, -z.x));
          xf[1] = exp2f(fmaf(xf[1], a.scale_log2, -z.y));
          xf[2] = exp2f(fmaf(xf[2], a.scale_log2, -z.z));
          xf[3] = exp2f(fmaf(xf[3], a.scale_log2, -z.w));
        }
      } else {
        // visible columns of this thread's key row inside the step: [vlo, vhi)
        const int vlo = (st.qs == CLEAN ? vqc_lo : vqn_lo) - st.q0 - c0, vhi = (st.qs == CLEAN ? vqc_hi : vqn_hi) - st.q0 - c0;
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 z = lz4[c4];
          const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = 4 * c4 + e;
            const float p = exp2f(fmaf(__uint_as_float(x[c]), a.scale_log2, -zz[e]));
            x[c] = __float_as_uint((c >= vlo && c < vhi) ? p : 0.f);
          }
        }
      }
      {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) pk[e] = pack_bf16(__uint_as_float(x[2 * e]), __uint_as_float(x[2 * e + 1]));
        tmem_st16(tl + c0, pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar_pt);
      const long long t1 = tick<TR>();
      c_exp += t1 - t0;

      ok = mbar_wait_timed<TR>(bar_dpt, i & 1, abort_flag, w_dpt);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long t2 = tick<TR>();
      uint32_t pk[16];
      {
        uint32_t y[32];
        tmem_ld32(tl + 128 + c0, y);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_dpfree);   // dP^T(i) is in registers: the tensor core may overwrite its columns
        const float4* dz4 = reinterpret_cast<const float4*>(d_s + sr * 64 + c0);
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 dz = dz4[c4];
          const float d0 = __uint_as_float(x[4 * c4 + 0]) * (__uint_as_float(y[4 * c4 + 0]) - dz.x);
          const float d1 = __uint_as_float(x[4 * c4 + 1]) * (__uint_as_float(y[4 * c4 + 1]) - dz.y);
          const float d2 = __uint_as_float(x[4 * c4 + 2]) * (__uint_as_float(y[4 * c4 + 2]) - dz.z);
          const float d3 = __uint_as_float(x[4 * c4 + 3]) * (__uint_as_float(y[4 * c4 + 3]) - dz.w);
          pk[2 * c4] = pack_bf16(d0, d1);
          pk[2 * c4 + 1] = pack_bf16(d2, d3);
        }
      }
      c_ds += tick<TR>() - t2;
      // dS^T(i) into the shared-memory tile, once dK and dQ^T of step i-1 have read dS^T(i-1)
      if (i > 0) {
        ok = mbar_wait_timed<TR>(bar_dsfree, (i - 1) & 1, abort_flag, w_dsf);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
#pragma unroll
      for (int c8 = 0; c8 < 4; ++c8)
        *reinterpret_cast<uint4*>(dsrow + (((4 * w + c8) ^ (r & 7)) << 4)) = make_uint4(pk[4 * c8], pk[4 * c8 + 1], pk[4 * c8 + 2], pk[4 * c8 + 3]);
      fence_async_smem();
      mbar_arrive(bar_dst);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_rows_empty + 8 * sr);   // this warp is done with the stage's LSE / D rows
    }
    if (warp == 0 && lane == 0) {
      trace_add(a.trace, 16 + 0, nsteps); trace_add(a.trace, 16 + 1, w_st); trace_add(a.trace, 16 + 2, w_dpt);
      trace_add(a.trace, 16 + 3, w_dsf); trace_add(a.trace, 16 + 4, c_exp); trace_add(a.trace, 16 + 5, c_ds);
      trace_add(a.trace, 16 + 6, tick<TR>() - t_begin);
    }
    // epilogue: warpgroup 0 writes dV, warpgroup 1 writes dK (scaled)
    if (ok && nsteps > 0) {
      ok = mbar_wait_abortable(bar_done, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      bf16* dst = (w == 0 ? a.dv[ks] : a.dk[ks]) + (((int64_t)b * L + k0_row + r) * a.Hkv + hk) * D;
      const float sc = (w == 0) ? 1.f : a.scale;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        if (nsteps > 0) { tmem_ld32(tl + 256 + w * 128 + c * 32, v); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        if (k0_row + r < L) store_row_chunk(dst + c * 32, v, sc);   // key rows past the end of the tensor are not written
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tmem, 512);
}

// fp32 dQ accumulator [batch, H, rows, 128] -> bf16 dQ [batch, rows, H, D]; one warp per row (D = 64: the first 64
// of the accumulator row's 128 floats)
template <int D>
__global__ void __launch_bounds__(256) dq_convert_kernel(const float* __restrict__ src, bf16* __restrict__ dst, int batch, int H, int rows,
                                                         int src_rows) {
  constexpr int U = 4;   // rows per warp in flight: the kernel is a pure stream
  const int lane = threadIdx.x & 31;
  const int64_t n = (int64_t)batch * rows * H;
  const int64_t warps = (int64_t)gridDim.x * 8;
  for (int64_t o0 = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * U; o0 < n; o0 += warps * U) {
    float4 u4[U];
    float2 u2[U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int64_t o = o0 + j;
      if (o < n) {
        const int h = (int)(o % H);
        const int64_t bl = o / H;
        const int l = (int)(bl % rows), b = (int)(bl / rows);
        const float* row = src + (((int64_t)b * H + h) * src_rows + l) * 128;
        if (D == 128) u4[j] = reinterpret_cast<const float4*>(row)[lane];
        else u2[j] = reinterpret_cast<const float2*>(row)[lane];
      }
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int64_t o = o0 + j;
      if (o < n) {
        if (D == 128) {
          uint2 v;
          v.x = pack_bf16(u4[j].x, u4[j].y); v.y = pack_bf16(u4[j].z, u4[j].w);
          reinterpret_cast<uint2*>(dst + o * D)[lane] = v;
        } else {
          reinterpret_cast<uint32_t*>(dst + o * D)[lane] = pack_bf16(u2[j].x, u2[j].y);
        }
      }
    }
  }
}

}  // namespace

static size_t pad64(size_t rows) { return (rows + 63) / 64 * 64; }

bool tc_bwd_supported(const KArgs& a) {
  return (a.d == 128 || a.d == 64) && tc_rows_ok(a) && tc_encoder_available();
}
// fp32 dQ accumulators of the fused backward: one [batch, H, rows, 128] tensor per query stream
size_t tc_bwd_fused_workspace(const bdlm_params* p, const bdlm_packed_geometry* g) {
  if ((p->d != 128 && p->d != 64) || p->impl == 1) return 0;
  const size_t rows_c = g != nullptr ? (size_t)g->Lq_clean : (size_t)p->L;
  const size_t rows_n = g != nullptr ? (size_t)g->n_blocks * p->block_size : (size_t)p->L;
  // rows rounded up to the kernel's 64-row steps: a reduction always covers a whole step
  return (pad64(rows_c) + pad64(rows_n)) * p->batch * p->H * 128 * sizeof(float);
}

template <int D>
static cudaError_t launch_tc_bwd_d(const KArgs& a_in, void* extra_ws, int passes, cudaStream_t st) {
  KArgs a = a_in;
  a.dq32_rows[CLEAN] = a.q[CLEAN] != nullptr ? (int)pad64(a.Lqc) : 0;
  a.dq32_rows[NOISY] = a.q[NOISY] != nullptr ? (int)pad64(a.Ln) : 0;
  const size_t dq32_elems[2] = {(size_t)a.batch * a.H * a.dq32_rows[CLEAN] * 128, (size_t)a.batch * a.H * a.dq32_rows[NOISY] * 128};
  if (a.single_pass) {
    a.dq32[0] = static_cast<float*>(extra_ws);
    a.dq32[1] = a.dq32[0] + dq32_elems[0];
  }
  BwdMaps maps;
  for (int s = 0; s < 2; ++s) {
    // a stream that is left out gets the other stream's tensors as placeholders: its maps are never used
    const int sq = a.q[s] != nullptr ? s : 1 - s;
    const int sk = a.k[s] != nullptr ? s : CLEAN;
    const int qbox = a.single_pass ? HT : TILE;   // the fused kernel loads 64 query rows per step
    if (!tc_make_map(&maps.q[s], a.q[sq], a.H, rows_q(a, sq), a.batch, qbox, D)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.dout[s], a.dout[sq], a.H, rows_q(a, sq), a.batch, qbox, D)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.k[s], a.k[sk], a.Hkv, rows_k(a, sk), a.batch, TILE, D)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.v[s], a.v[sk], a.Hkv, rows_k(a, sk), a.batch, TILE, D)) return cudaErrorInvalidValue;
  }
  int* status = device_status_ptr();
  if (status == nullptr) return cudaErrorUnknown;
  cudaError_t e;
  if (a.single_pass) {
    // one kernel produces dK, dV and (through fp32 add-reductions) dQ; it runs for the DKDV pass bit, the DQ bit is a no-op
    if (passes & BDLM_BWD_PASS_DKDV) {
      if ((e = cudaMemsetAsync(a.dq32[0], 0, (dq32_elems[0] + dq32_elems[1]) * sizeof(float), st)) != cudaSuccess) return e;
      auto kern = a.trace ? tc_bwdf_kernel<true, D> : tc_bwdf_kernel<false, D>;
      if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, BF_SMEM)) != cudaSuccess) return e;
      const TileGrid tg = make_tile_grid((max(a.L, a.k[NOISY] != nullptr ? a.Ln : 0) + TILE - 1) / TILE, a.Hkv, a.batch * 2);
      if (tile_grid_blocks(tg) == 0) return cudaErrorInvalidValue;
      kern<<<tile_grid_blocks(tg), BF_THREADS, BF_SMEM, st>>>(maps, a, tg, status);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      for (int s2 = 0; s2 < 2; ++s2) {
        if (dq32_elems[s2] == 0) continue;
        dq_convert_kernel<D><<<device_sm_count() * 16, 256, 0, st>>>(a.dq32[s2], a.dq[s2], a.batch, a.H, rows_q(a, s2), a.dq32_rows[s2]);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
      }
    }
    return cudaSuccess;
  }
  if (passes & BDLM_BWD_PASS_DKDV) {
    auto kern = a.trace ? tc_dkdv_kernel<true, D> : tc_dkdv_kernel<false, D>;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, DKDV_SMEM)) != cudaSuccess) return e;
    const TileGrid tg = make_tile_grid((max(a.L, a.k[NOISY] != nullptr ? a.Ln : 0) + TILE - 1) / TILE, a.Hkv, a.batch * 2);
    if (tile_grid_blocks(tg) == 0) return cudaErrorInvalidValue;
    kern<<<tile_grid_blocks(tg), DKDV_THREADS, DKDV_SMEM, st>>>(maps, a, tg, status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (passes & BDLM_BWD_PASS_DQ) {
    auto kern = a.trace ? tc_dq_kernel<true, D> : tc_dq_kernel<false, D>;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM)) != cudaSuccess) return e;
    const TileGrid tg = make_tile_grid((max(a.q[CLEAN] != nullptr ? a.Lqc : 0, a.q[NOISY] != nullptr ? a.Ln : 0) + TILE - 1) / TILE, a.H, a.batch * 2);
    if (tile_grid_blocks(tg) == 0) return cudaErrorInvalidValue;
    kern<<<tile_grid_blocks(tg), BWD_THREADS, DQ_SMEM, st>>>(maps, a, tg, status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_tc_bwd(const KArgs& a, void* extra_ws, int passes, cudaStream_t st) {
  return a.d == 64 ? launch_tc_bwd_d<64>(a, extra_ws, passes, st) : launch_tc_bwd_d<128>(a, extra_ws, passes, st);
}

}  // namespace bdlm
