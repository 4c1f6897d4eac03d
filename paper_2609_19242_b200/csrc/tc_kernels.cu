// BDLM attention on the 5th-generation tensor cores (tcgen05): Q.K^T and P.V are issued as
// tcgen05.mma with operands staged in shared memory by TMA (128-byte swizzle) and fp32
// accumulators in tensor memory; the online softmax runs in registers, one thread per query
// row.  The tile schedule enumerates only the key tiles a query tile can see (Algorithm 1:
// clean-prefix tiles, then the noisy-diagonal tiles); no mask is materialised.
#include "tc_common.cuh"
#include "tc_launch.h"

namespace bdlm {
namespace {

using namespace tc;
using bf16 = __nv_bfloat16;

struct FwdMaps {
  CUtensorMap q[2], k[2], v[2];
};

// ---------------------------------------------------------------- host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

namespace {
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
    if (q != cudaDriverEntryPointSuccess) p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace

bool tc_encoder_available() { return encode_fn() != nullptr; }

// [batch, L, heads, d] bf16 viewed as 3-D (heads*d, L, batch); box = 64 columns x `rows` rows.
// Encoding a map costs the host a microsecond or two and a call needs six to eight of them, which shows at sizes
// where a whole step takes a few milliseconds; a training loop passes the same tensors again and again, so each host
// thread keeps the maps it encoded last in a small direct-mapped table keyed by (address, shape, box).  A map is a
// plain 128-byte value that describes addresses and strides only, so a copy of it is as good as a fresh encode.
bool tc_make_map(CUtensorMap* m, const void* ptr, int heads_in, int L, int batch, int rows, int d) {
  const int heads = heads_in * (d / 64);   // in units of 64-column panels: the map only knows the row length
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || ptr == nullptr) return false;
  struct Entry { const void* ptr; int heads, L, batch, rows; bool valid; CUtensorMap map; };
  constexpr int kEntries = 64;
  thread_local Entry cache[kEntries] = {};
  const uint64_t key = (reinterpret_cast<uint64_t>(ptr) >> 8) * 0x9E3779B97F4A7C15ull + (uint64_t)rows * 0x632BE59BD9B4E019ull +
                       (uint64_t)L * 31 + (uint64_t)heads;
  Entry& e = cache[(key >> 32) % kEntries];
  if (e.valid && e.ptr == ptr && e.heads == heads && e.L == L && e.batch == batch && e.rows == rows) {
    *m = e.map;
    return true;
  }
  cuuint64_t gdim[3] = {(cuuint64_t)heads * 64, (cuuint64_t)L, (cuuint64_t)batch};
  cuuint64_t gstride[2] = {(cuuint64_t)heads * 64 * 2, (cuuint64_t)L * heads * 64 * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  e.ptr = ptr; e.heads = heads; e.L = L; e.batch = batch; e.rows = rows; e.map = *m; e.valid = true;
  return true;
}

bool tc_make_map_2d(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || ptr == nullptr) return false;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
// ---------------------------------------------------------------- forward kernel
constexpr uint32_t IDESC_QK = make_idesc(128, 128, false, false);
constexpr int TILE_BYTES = 2 * PANEL_BYTES;   // 128 x 128 bf16

// Key tiles visible from a run of query rows: a clean segment then a noisy segment, each a run
// of 128-key tiles starting at the first visible key; scalars only (no indexed arrays).
struct TileSched {
  int lo0, lo1, nt0, nt1, lo_last0, lo_last1, hi_first0, hi_first1;
  // key tiles seen by the query rows [q0, q_last]: the visible interval of a row moves up with the row, so the
  // first row gives the lower end and the last row the upper end
  __device__ __forceinline__ void init(int qs, int q0, int q_last, const KArgs& a) {
    int lo_f, hi_f, lo_l, hi_l;
    visible_interval(a, qs, 0, q0, lo_f, hi_f);
    visible_interval(a, qs, 0, q_last, lo_l, hi_l);
    lo0 = lo_f; lo_last0 = lo_l; hi_first0 = hi_f; nt0 = hi_l > lo_f ? (hi_l - lo_f + TILE - 1) / TILE : 0;
    visible_interval(a, qs, 1, q0, lo_f, hi_f);
    visible_interval(a, qs, 1, q_last, lo_l, hi_l);
    lo1 = lo_f; lo_last1 = lo_l; hi_first1 = hi_f; nt1 = hi_l > lo_f ? (hi_l - lo_f + TILE - 1) / TILE : 0;
  }
  // a tile needs per-element masking unless every one of the query rows sees all of its 128 keys
  __device__ __forceinline__ bool need_mask(int ks, int k0) const {
    return ks == 0 ? (k0 < lo_last0 || k0 + TILE > hi_first0) : (k0 < lo_last1 || k0 + TILE > hi_first1);
  }
};

// ---------------------------------------------------------------- forward, warp-specialised
// One CTA = one 128-row query tile of TWO query heads of the same KV group (same stream, same rows, so
// the same key tiles and the same masks).  Warp 8 loads Q of both heads once and streams K/V tiles through
// a 2-stage ring; warp 9 issues tcgen05.mma (QK^T from shared memory, PV with P as a TMEM operand: the whole
// warp walks the loop, one elected lane issues); warps 0-7 run the online softmax, one warpgroup per head and
// one thread per query row: the thread holds the tile's 128 scores in registers (one pass over S, no exchange
// between threads; 320 threads leave it up to 200 registers).  While one head's warpgroup is in its
// exponentials the tensor core runs the other head's P V and next Q K^T.  P (bf16) overwrites the first 64 of
// the S columns it was computed from; O is rescaled only when the running maximum grew by more than 2^8 (the
// stale maximum is exact in the final LSE and normalisation).
// With an odd number of query heads per KV head (PAIRQ) the two warpgroups take two consecutive query tiles of
// ONE head instead: the CTA walks the union of their key tiles (the later tile's list contains the earlier
// one's except for noisy diagonal tiles), a tile that one of them does not see at all is masked out for it
// like any other hidden key, and a second tile past the end of the tensor stays masked and is not written.
// TMEM columns: [0,128) S/P head A   [128,256) S/P head B   [256,384) O head A   [384,512) O head B
constexpr int FWDR_THREADS = 320;                            // 8 softmax warps, producer warp, MMA warp
constexpr int FWDR_BARS = 6 * TILE_BYTES;                    // after Q (2 tiles) and the K/V ring (2 stages x 2 tiles)
constexpr int FWDR_SMEM = FWDR_BARS + 256 + 1024;

// D = head dimension (128 or 64).  With D = 64 a tile is one 64-column panel: the second panel of every shared-memory
// tile stays unused, Q K^T contracts over four k-slices and P V produces 64 output columns.
template <bool TR, bool PAIRQ, int D>
__global__ void __launch_bounds__(FWDR_THREADS, 1)
tc_fwdr_kernel(const __grid_constant__ FwdMaps maps, const KArgs a, const TileGrid tg, int* __restrict__ status) {
  constexpr uint32_t IDESC_PV = make_idesc(128, D, false, true);
  constexpr int OPER_BYTES = TILE_BYTES * D / 128;   // bytes TMA delivers per operand tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base, sK0 = base + 2 * TILE_BYTES;   // stage s: K at sK0 + s*2*TILE, V after it
  const uint32_t bars = base + FWDR_BARS;
  const uint32_t bar_q = bars, bar_k_full = bars + 8 /*[2]*/, bar_v_full = bars + 24 /*[2]*/, bar_kv_empty = bars + 40 /*[2]*/,
                 bar_s = bars + 56 /*[2]*/, bar_o = bars + 72 /*[2]*/, bar_p = bars + 88 /*[head][key half]*/;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + FWDR_BARS + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + FWDR_BARS + 136);

  int bx, by, bz;
  tile_grid_decode(tg, bx, by, bz);
  const int qs = bz & 1, b = bz >> 1;
  if (a.q[qs] == nullptr) return;
  // warpgroup w works on head h0 + w * HSTEP, query rows q0 + w * QSTEP ...
  constexpr int HSTEP = PAIRQ ? 0 : 1, QSTEP = PAIRQ ? TILE : 0, QROWS = PAIRQ ? 2 * TILE : TILE;
  const int h0 = PAIRQ ? by : by * 2, hk = h0 / a.G;
  const int q0 = (tg.nx - 1 - bx) * QROWS;   // the last query tile sees the most keys: started first
  const int Lq = rows_q(a, qs);
  if (q0 >= Lq) return;
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // warp index, provably uniform

  TileSched sch;
  sch.init(qs, q0, min(q0 + QROWS, Lq) - 1, a);
  const int nt = sch.nt0 + sch.nt1;
  auto tile_ks = [&](int t) { return t < sch.nt0 ? 0 : 1; };
  auto tile_k0 = [&](int t) { return t < sch.nt0 ? sch.lo0 + t * TILE : sch.lo1 + (t - sch.nt0) * TILE; };

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_k_full + 8 * i, 1); mbar_init(bar_v_full + 8 * i, 1); mbar_init(bar_kv_empty + 8 * i, 1);
      mbar_init(bar_s + 8 * i, 1); mbar_init(bar_o + 8 * i, 1);
      mbar_init(bar_p + 16 * i, 128); mbar_init(bar_p + 16 * i + 8, 128);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // broadcast: provably warp-uniform
  // TMEM columns: [0,128) S/P head A   [128,256) S/P head B   [256,384) O head A   [384,512) O head B

  if (warp == 8) {
    if (lane == 0 && nt > 0) {
      mbar_expect_tx(bar_q, 2 * OPER_BYTES);
      tma_load_3d(sQ, &maps.q[qs], bar_q, h0 * D, q0, b);
      if (D == 128) tma_load_3d(sQ + PANEL_BYTES, &maps.q[qs], bar_q, h0 * D + 64, q0, b);
      // (rows past the end of the tensor are filled with zeros)
      tma_load_3d(sQ + TILE_BYTES, &maps.q[qs], bar_q, (h0 + HSTEP) * D, q0 + QSTEP, b);
      if (D == 128) tma_load_3d(sQ + TILE_BYTES + PANEL_BYTES, &maps.q[qs], bar_q, (h0 + HSTEP) * D + 64, q0 + QSTEP, b);
      bool ok = true;
      for (int t = 0; t < nt && ok; ++t) {
        const int s = t & 1;
        if (t >= 2) ok = mbar_wait_abortable(bar_kv_empty + 8 * s, ((t >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        const int ks = tile_ks(t), k0 = tile_k0(t);
        const uint32_t dK = sK0 + s * 2 * TILE_BYTES, dV = dK + TILE_BYTES;
        mbar_expect_tx(bar_k_full + 8 * s, OPER_BYTES);
        const int krow = ks == CLEAN ? clean_key_row(a, k0) : k0;   // where the tile's first key is stored
        tma_load_3d(dK, &maps.k[ks], bar_k_full + 8 * s, hk * D, krow, b);
        if (D == 128) tma_load_3d(dK + PANEL_BYTES, &maps.k[ks], bar_k_full + 8 * s, hk * D + 64, krow, b);
        mbar_expect_tx(bar_v_full + 8 * s, OPER_BYTES);
        tma_load_3d(dV, &maps.v[ks], bar_v_full + 8 * s, hk * D, krow, b);
        if (D == 128) tma_load_3d(dV + PANEL_BYTES, &maps.v[ks], bar_v_full + 8 * s, hk * D + 64, krow, b);
      }
    }
  } else if (warp == 9) {
    // the whole warp walks the MMA loop; one elected lane issues (see elect_one)
    if (nt > 0) {
      const uint32_t el = elect_one();
      const uint32_t qa_lo = desc_lo_k(sQ), qb_lo = qa_lo + TILE_LO;
      const uint32_t k_lo0 = desc_lo_k(sK0), v_lo0 = desc_lo_mn(sK0 + TILE_BYTES);
      bool ok = mbar_wait_abortable(bar_q, 0, abort_flag);
      ok = ok && mbar_wait_abortable(bar_k_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        gemm_ss_e<D / 16>(tmem, qa_lo, k_lo0, IDESC_QK, 0u, el);
        mma_commit_e(bar_s, el);
        gemm_ss_e<D / 16>(tmem + 128, qb_lo, k_lo0, IDESC_QK, 0u, el);
        mma_commit_e(bar_s + 8, el);
      }
      // O += P V over key half j of the tile: four k-slices of 16 keys
      auto pv_half = [&](uint32_t d, uint32_t p_tmem, uint32_t v_lo, int j, uint32_t acc_first) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_e(d, p_tmem + (4 * j + kk) * 8, desc64(v_lo + moff(4 * j + kk)), IDESC_PV, kk == 0 ? acc_first : 1u, el);
      };
      long long w_p = 0, w_v = 0, w_k = 0;
      const long long tm0 = tick<TR>();
      for (int t = 0; t < nt && ok; ++t) {
        const int s = t & 1;
        const uint32_t cv_lo = v_lo0 + s * 2 * TILE_LO;
        const uint32_t nk_lo = k_lo0 + (s ^ 1) * 2 * TILE_LO;
        const uint32_t acc = t > 0 ? 1u : 0u;
        // head A: P arrives in two halves of the keys (bf16 pairs at columns [0,32) and [32,64) of the head's S
        // region), so P V over the first 64 keys runs while the softmax is still in the exponentials of the rest
        ok = mbar_wait_timed<TR>(bar_p, t & 1, abort_flag, w_p);
        ok = ok && mbar_wait_timed<TR>(bar_v_full + 8 * s, (t >> 1) & 1, abort_flag, w_v);
        if (!ok) break;
        tc_fence_after();
        pv_half(tmem + 256, tmem, cv_lo, 0, acc);
        ok = mbar_wait_timed<TR>(bar_p + 8, t & 1, abort_flag, w_p);
        if (!ok) break;
        tc_fence_after();
        pv_half(tmem + 256, tmem, cv_lo, 1, 1u);
        mma_commit_e(bar_o, el);
        if (t + 1 < nt) {
          ok = mbar_wait_timed<TR>(bar_k_full + 8 * (s ^ 1), ((t + 1) >> 1) & 1, abort_flag, w_k);
          if (!ok) break;
          tc_fence_after();
          gemm_ss_e<D / 16>(tmem, qa_lo, nk_lo, IDESC_QK, 0u, el);
          mma_commit_e(bar_s, el);
        }
        // head B
        ok = mbar_wait_timed<TR>(bar_p + 16, t & 1, abort_flag, w_p);
        if (!ok) break;
        tc_fence_after();
        pv_half(tmem + 384, tmem + 128, cv_lo, 0, acc);
        ok = mbar_wait_timed<TR>(bar_p + 24, t & 1, abort_flag, w_p);
        if (!ok) break;
        tc_fence_after();
        pv_half(tmem + 384, tmem + 128, cv_lo, 1, 1u);
        mma_commit_e(bar_o + 8, el);
        mma_commit_e(bar_kv_empty + 8 * s, el);
        if (t + 1 < nt) {
          gemm_ss_e<D / 16>(tmem + 128, qb_lo, nk_lo, IDESC_QK, 0u, el);
          mma_commit_e(bar_s + 8, el);
        }
      }
      if (lane == 0) {
        trace_add(a.trace, 8, tick<TR>() - tm0); trace_add(a.trace, 9, w_p); trace_add(a.trace, 10, w_v); trace_add(a.trace, 11, w_k);
      }
    }
  } else {
    const int w = warp >> 2;                               // head: one warpgroup per head, one thread per query row
    const int r = (warp & 3) * 32 + lane;
    const int row = q0 + w * QSTEP + r;
    const int h = h0 + w * HSTEP;
    const bool row_ok = row < Lq;                            // PAIRQ: the second tile may lie past the end
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + w * 128;          // this row's 128 score columns
    const uint32_t tO = tmem + lane_base + 256 + w * 128;    // and its 128 output columns
    int rlo0 = 0, rhi0 = 0, rlo1 = 0, rhi1 = 0;
    if (row_ok) {
      visible_interval(a, qs, 0, row, rlo0, rhi0);
      visible_interval(a, qs, 1, row, rlo1, rhi1);
    }
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    long long w_s = 0, c_ld = 0, c_max = 0, c_exp = 0;
    const long long t_begin = tick<TR>();
    for (int t = 0; t < nt && ok; ++t) {
      const int ks = tile_ks(t), k0 = tile_k0(t);
      ok = mbar_wait_timed<TR>(bar_s + 8 * w, t & 1, abort_flag, w_s);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool need_mask = sch.need_mask(ks, k0) || q0 + QROWS > Lq;   // rows past the end of the tensor see nothing
      const int vlo = (ks == 0 ? rlo0 : rlo1) - k0, vhi = (ks == 0 ? rhi0 : rhi1) - k0;
      // the whole row of the tile in registers: one pass over S
      const long long tp0 = tick<TR>();
      uint32_t v[128];
      {
        uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(v);
        tmem_ld32(tS, c[0]); tmem_ld32(tS + 32, c[1]); tmem_ld32(tS + 64, c[2]); tmem_ld32(tS + 96, c[3]);
        tmem_wait_ld();
      }
      const long long tp1 = tick<TR>();
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
      if (need_mask) {
#pragma unroll
        for (int e = 0; e < 128; ++e) v[e] = (e >= vlo && e < vhi) ? v[e] : 0xff800000u;   // -inf on hidden keys
      }
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        mx0 = fmaxf(mx0, __uint_as_float(v[e])); mx1 = fmaxf(mx1, __uint_as_float(v[32 + e]));
        mx2 = fmaxf(mx2, __uint_as_float(v[64 + e])); mx3 = fmaxf(mx3, __uint_as_float(v[96 + e]));
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * a.scale_log2;
      const float m_new = fmaxf(m_ref, mx);
      const bool grow = m_new > m_ref + 8.0f;
      if (__any_sync(0xffffffffu, grow)) {
        const float mb_new = (m_new == -INFINITY) ? 0.f : m_new;
        const float corr = exp2f(m_ref - mb_new);
        m_ref = m_new;
        l *= corr;
        if (t > 0) {
          ok = mbar_wait_abortable(bar_o + 8 * w, (t - 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * corr);
            tmem_st32(tO + c * 32, o);
          }
        }
      }
      const float mb = (m_ref == -INFINITY) ? 0.f : m_ref;
      const long long tp2 = tick<TR>();
      // p = exp2(s * scale - m) (exp2(-inf) = 0 on hidden keys); bf16 pairs over the first 64 columns
      float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          if (half == 1 && e == 4) {   // the first half's store has landed by now: hand it over without stalling for it
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p + 16 * w);
          }
          const int c = 64 * half + 4 * e;
          const float p0 = exp2f(fmaf(__uint_as_float(v[c]), a.scale_log2, -mb));
          const float p1 = exp2f(fmaf(__uint_as_float(v[c + 1]), a.scale_log2, -mb));
          const float p2 = exp2f(fmaf(__uint_as_float(v[c + 2]), a.scale_log2, -mb));
          const float p3 = exp2f(fmaf(__uint_as_float(v[c + 3]), a.scale_log2, -mb));
          ps0 += p0; ps1 += p1; ps2 += p2; ps3 += p3;
          pk[2 * e] = pack_bf16(p0, p1);
          pk[2 * e + 1] = pack_bf16(p2, p3);
        }
        tmem_st32(tS + 32 * half, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p + 16 * w + 8);
      l += (ps0 + ps1) + (ps2 + ps3);
      c_ld += tp1 - tp0; c_max += tp2 - tp1; c_exp += tick<TR>() - tp2;
    }
    if (warp == 0 && lane == 0) { trace_add(a.trace, 0, nt); trace_add(a.trace, 1, w_s); trace_add(a.trace, 6, tick<TR>() - t_begin);
      trace_add(a.trace, 3, c_ld); trace_add(a.trace, 4, c_max); trace_add(a.trace, 5, c_exp); }
    if (ok && nt > 0) {
      ok = mbar_wait_abortable(bar_o + 8 * w, (nt - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      bf16* orow = a.o[qs] + (((int64_t)b * Lq + row) * a.H + h) * D;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        if (nt > 0) { tmem_ld32(tO + c * 32, o); tmem_wait_ld(); }
#pragma unroll
        for (int e8 = 0; e8 < 4; ++e8) {
          uint4 vv;
          uint32_t* pv = reinterpret_cast<uint32_t*>(&vv);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float x0 = nt > 0 ? __uint_as_float(o[e8 * 8 + 2 * e]) * inv : 0.f;
            const float x1 = nt > 0 ? __uint_as_float(o[e8 * 8 + 2 * e + 1]) * inv : 0.f;
            pv[e] = pack_bf16(x0, x1);
          }
          if (row_ok) *reinterpret_cast<uint4*>(orow + c * 32 + e8 * 8) = vv;
        }
      }
      if (row_ok) a.lse[qs][((int64_t)b * a.H + h) * Lq + row] = l > 0.f ? (m_ref + log2f(l)) * LN2 : -INFINITY;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tmem, 512);
}

}  // namespace

// Row counts need not be multiples of the 128-row tile: TMA fills the rows of a tile that lie past the end of a tensor
// with zeros, the masks never show a key past the end, and rows past the end are neither read from the per-row arrays
// nor written.  Only the gathered K/V order keeps its own rule (chunks of a multiple of 128 rows: checked at the boundary).
bool tc_rows_ok(const KArgs& a) {
  if (a.L <= 0) return false;
  if (a.q[CLEAN] != nullptr && a.Lqc <= 0) return false;
  if (a.q[NOISY] != nullptr && a.Ln <= 0) return false;
  return true;
}

bool tc_fwd_supported(const KArgs& a) {
  return (a.d == 128 || a.d == 64) && tc_rows_ok(a) && encode_fn() != nullptr;
}

template <int D>
static cudaError_t launch_tc_fwd_d(const KArgs& a, cudaStream_t st) {
  FwdMaps maps;
  for (int s = 0; s < 2; ++s) {
    // a stream that is left out gets the other stream's tensors as placeholders: its maps are never used
    const int sq = a.q[s] ? s : 1 - s;
    if (!tc_make_map(&maps.q[s], a.q[sq], a.H, rows_q(a, sq), a.batch, TILE, D)) return cudaErrorInvalidValue;
    const int sk = (s == NOISY && (a.q[NOISY] == nullptr || a.Ln == 0 || !a.diag)) ? CLEAN : s;
    if (!tc_make_map(&maps.k[s], a.k[sk], a.Hkv, rows_k(a, sk), a.batch, TILE, D)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.v[s], a.v[sk], a.Hkv, rows_k(a, sk), a.batch, TILE, D)) return cudaErrorInvalidValue;
  }
  const int qrows = max(a.q[CLEAN] != nullptr ? a.Lqc : 0, a.q[NOISY] != nullptr ? a.Ln : 0);
  int* status = device_status_ptr();
  if (status == nullptr) return cudaErrorUnknown;
  cudaError_t e;
  if (a.G % 2 == 0) {   // two heads of one KV group per CTA, one softmax warpgroup per head
    auto kern = a.trace ? tc_fwdr_kernel<true, false, D> : tc_fwdr_kernel<false, false, D>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FWDR_SMEM);
    if (e != cudaSuccess) return e;
    const TileGrid tg = make_tile_grid((qrows + TILE - 1) / TILE, a.H / 2, a.batch * 2);
    if (tile_grid_blocks(tg) == 0) return cudaErrorInvalidValue;
    kern<<<tile_grid_blocks(tg), FWDR_THREADS, FWDR_SMEM, st>>>(maps, a, tg, status);
    return cudaGetLastError();
  }
  // odd group size: two consecutive query tiles of one head per CTA
  auto kern = a.trace ? tc_fwdr_kernel<true, true, D> : tc_fwdr_kernel<false, true, D>;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FWDR_SMEM);
  if (e != cudaSuccess) return e;
  const TileGrid tg = make_tile_grid(((qrows + TILE - 1) / TILE + 1) / 2, a.H, a.batch * 2);
  if (tile_grid_blocks(tg) == 0) return cudaErrorInvalidValue;
  kern<<<tile_grid_blocks(tg), FWDR_THREADS, FWDR_SMEM, st>>>(maps, a, tg, status);
  return cudaGetLastError();
}

cudaError_t launch_tc_fwd(const KArgs& a, cudaStream_t st) {
  return a.d == 64 ? launch_tc_fwd_d<64>(a, st) : launch_tc_fwd_d<128>(a, st);
}

}  // namespace bdlm
