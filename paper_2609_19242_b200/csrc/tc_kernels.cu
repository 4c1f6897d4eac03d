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

// [batch, L, heads, 128] bf16 viewed as 3-D (heads*128, L, batch); box = 64 columns x `rows` rows.
bool tc_make_map(CUtensorMap* m, const void* ptr, int heads, int L, int batch, int rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || ptr == nullptr) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)heads * 128, (cuuint64_t)L, (cuuint64_t)batch};
  cuuint64_t gstride[2] = {(cuuint64_t)heads * 128 * 2, (cuuint64_t)L * heads * 128 * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

namespace {
// ---------------------------------------------------------------- forward kernel
constexpr uint32_t IDESC_QK = make_idesc(128, 128, false, false);
constexpr uint32_t IDESC_PV = make_idesc(128, 128, false, true);
constexpr int TILE_BYTES = 2 * PANEL_BYTES;   // 128 x 128 bf16
#ifndef BDLM_P_IN_TMEM
#define BDLM_P_IN_TMEM 1
#endif
constexpr int FWD_SMEM = 6 * TILE_BYTES + 128 + 1024;   // Q, 2x(K,V), P, barriers, alignment slack

__global__ void __launch_bounds__(128, 1)
tc_fwd_kernel(const __grid_constant__ FwdMaps maps, const KArgs a, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base, sKV = base + TILE_BYTES, sP = base + 5 * TILE_BYTES;
  const uint32_t bars = base + 6 * TILE_BYTES;
  const uint32_t bar_q = bars, bar_kv0 = bars + 8, bar_s = bars + 24, bar_o = bars + 32;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + 6 * TILE_BYTES + 64);

  const int qs = blockIdx.z & 1, b = blockIdx.z >> 1;
  if (a.q[qs] == nullptr) return;
  const int h = blockIdx.y, hk = h / a.G;
  const int q0 = (gridDim.x - 1 - blockIdx.x) * TILE;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = q0 + tid;

  if (tid == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_kv0, 1); mbar_init(bar_kv0 + 8, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    fence_mbar_init();
    prefetch_tmap(&maps.q[qs]); prefetch_tmap(&maps.k[0]); prefetch_tmap(&maps.v[0]);
  }
  if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem + ((uint32_t)(warp * 32) << 16);   // columns 0..127: S
  const uint32_t tO = tS + 128;                               // columns 128..255: O

  // key segments visible from this query tile: clean keys first, then noisy keys
  int seg_lo[2], seg_hi[2], lo_last[2], hi_first[2], ntile[2];
  int rlo[2], rhi[2];
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    int lo_f, hi_f, lo_l, hi_l;
    visible_interval(qs, ks, q0, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, lo_f, hi_f);
    visible_interval(qs, ks, q0 + TILE - 1, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, lo_l, hi_l);
    seg_lo[ks] = lo_f; seg_hi[ks] = hi_l; lo_last[ks] = lo_l; hi_first[ks] = hi_f;
    ntile[ks] = seg_hi[ks] > seg_lo[ks] ? (seg_hi[ks] - seg_lo[ks] + TILE - 1) / TILE : 0;
    visible_interval(qs, ks, row, a.M, a.mode, a.kv_begin, a.kv_end, a.diag, rlo[ks], rhi[ks]);
  }
  const int nt = ntile[0] + ntile[1];

  auto issue_kv = [&](int t) {   // thread 0 only
    const int ks = t < ntile[0] ? 0 : 1;
    const int k0 = ks == 0 ? seg_lo[0] + t * TILE : seg_lo[1] + (t - ntile[0]) * TILE;
    const uint32_t bar = bar_kv0 + 8 * (t & 1);
    const uint32_t dK = sKV + (t & 1) * 2 * TILE_BYTES, dV = dK + TILE_BYTES;
    mbar_expect_tx(bar, 2 * TILE_BYTES);
    tma_load_3d(dK, &maps.k[ks], bar, hk * 128, k0, b);
    tma_load_3d(dK + PANEL_BYTES, &maps.k[ks], bar, hk * 128 + 64, k0, b);
    tma_load_3d(dV, &maps.v[ks], bar, hk * 128, k0, b);
    tma_load_3d(dV + PANEL_BYTES, &maps.v[ks], bar, hk * 128 + 64, k0, b);
  };

  if (tid == 0 && nt > 0) {
    mbar_expect_tx(bar_q, TILE_BYTES);
    tma_load_3d(sQ, &maps.q[qs], bar_q, h * 128, q0, b);
    tma_load_3d(sQ + PANEL_BYTES, &maps.q[qs], bar_q, h * 128 + 64, q0, b);
    issue_kv(0);
  }

  float m = -INFINITY, l = 0.f;
  bool fail = false;
  for (int t = 0; t < nt; ++t) {
    const int ks = t < ntile[0] ? 0 : 1;
    const int k0 = ks == 0 ? seg_lo[0] + t * TILE : seg_lo[1] + (t - ntile[0]) * TILE;
    const uint32_t sK = sKV + (t & 1) * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
    if (tid == 0 && t + 1 < nt) issue_kv(t + 1);   // stage (t+1)&1 was released by the PV MMA of tile t-1
    if (t == 0) fail |= !mbar_wait(bar_q, 0);
    fail |= !mbar_wait(bar_kv0 + 8 * (t & 1), (t >> 1) & 1);
    if (tid == 0 && !fail) {
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const uint32_t off = (kk >> 2) * PANEL_BYTES + (kk & 3) * 32;
        mma_ss(tmem, smem_desc(sQ + off, 16, 1024), smem_desc(sK + off, 16, 1024), IDESC_QK, kk > 0);
      }
      mma_commit(bar_s);
    }
    fail |= !mbar_wait(bar_s, t & 1);
    tc_fence_after();

    // ---- softmax on this thread's row -----------------------------------------------------
    uint32_t sr[128];
    {
      uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(sr);
      tmem_ld32(tS, c[0]); tmem_ld32(tS + 32, c[1]); tmem_ld32(tS + 64, c[2]); tmem_ld32(tS + 96, c[3]);
      tmem_wait_ld();
    }
    const bool need_mask = (k0 < lo_last[ks]) || (k0 + TILE > hi_first[ks]);
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < 128; ++c) {
      float x = __uint_as_float(sr[c]) * a.scale_log2;
      if (need_mask) {
        const int j = k0 + c;
        x = (j >= rlo[ks] && j < rhi[ks]) ? x : -INFINITY;
      }
      sr[c] = __float_as_uint(x);
      mx = fmaxf(mx, x);
    }
    const float m_new = fmaxf(m, mx);
    const float mb = (m_new == -INFINITY) ? 0.f : m_new;
    const float corr = exp2f(m - mb);
    m = m_new;
    float psum = 0.f;
#if BDLM_P_IN_TMEM
    // P (bf16 pairs) overwrites the first 64 columns of this row's S in tensor memory
#pragma unroll
    for (int c32 = 0; c32 < 2; ++c32) {
      uint32_t pk[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const float p0 = exp2f(__uint_as_float(sr[c32 * 64 + 2 * e]) - mb);
        const float p1 = exp2f(__uint_as_float(sr[c32 * 64 + 2 * e + 1]) - mb);
        psum += p0 + p1;
        pk[e] = pack_bf16(p0, p1);
      }
      tmem_st32(tS + c32 * 32, pk);
    }
#else
    uint8_t* prow = sm + (sP - base);
#pragma unroll
    for (int c8 = 0; c8 < 16; ++c8) {
      float p[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) { p[e] = exp2f(__uint_as_float(sr[c8 * 8 + e]) - mb); psum += p[e]; }
      uint4 v;
      v.x = pack_bf16(p[0], p[1]); v.y = pack_bf16(p[2], p[3]); v.z = pack_bf16(p[4], p[5]); v.w = pack_bf16(p[6], p[7]);
      *reinterpret_cast<uint4*>(prow + sw128_offset(tid, c8 * 8)) = v;
    }
#endif
    l = l * corr + psum;
    if (t > 0) {   // rescale the running output (the previous PV MMA has completed)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(tO + c * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * corr);
        tmem_st32(tO + c * 32, o);
      }
    }
    tmem_wait_st();
    tc_fence_before();
    fence_async_smem();
    if (__syncthreads_or(fail)) { fail = true; break; }
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
#if BDLM_P_IN_TMEM
        mma_ts(tmem + 128, tmem + kk * 8, smem_desc(sV + kk * 2048, PANEL_BYTES, 1024), IDESC_PV,
               (t > 0 || kk > 0) ? 1u : 0u);
#else
        const uint32_t aoff = (kk >> 2) * PANEL_BYTES + (kk & 3) * 32;
        mma_ss(tmem + 128, smem_desc(sP + aoff, 16, 1024), smem_desc(sV + kk * 2048, PANEL_BYTES, 1024), IDESC_PV,
               (t > 0 || kk > 0) ? 1u : 0u);
#endif
      }
      mma_commit(bar_o);
    }
    fail |= !mbar_wait(bar_o, t & 1);
    tc_fence_after();
  }

  // ---- epilogue: O / l -> bf16, LSE ------------------------------------------------------------
  if (!fail) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
    bf16* orow = a.o[qs] + (((int64_t)b * a.L + row) * a.H + h) * 128;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t o[32];
      if (nt > 0) { tmem_ld32(tO + c * 32, o); tmem_wait_ld(); }
#pragma unroll
      for (int e8 = 0; e8 < 4; ++e8) {
        uint4 v;
        uint32_t* pv = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float x0 = nt > 0 ? __uint_as_float(o[e8 * 8 + 2 * e]) * inv : 0.f;
          float x1 = nt > 0 ? __uint_as_float(o[e8 * 8 + 2 * e + 1]) * inv : 0.f;
          pv[e] = pack_bf16(x0, x1);
        }
        *reinterpret_cast<uint4*>(orow + c * 32 + e8 * 8) = v;
      }
    }
    a.lse[qs][((int64_t)b * a.H + h) * a.L + row] = l > 0.f ? (m + log2f(l)) * LN2 : -INFINITY;
  } else if (tid == 0) {
    atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

bool tc_fwd_supported(const KArgs& a) {
  return a.d == 128 && a.L % TILE == 0 && encode_fn() != nullptr;
}

cudaError_t launch_tc_fwd(const KArgs& a, cudaStream_t st) {
  FwdMaps maps;
  for (int s = 0; s < 2; ++s) {
    const void* q = a.q[s] ? (const void*)a.q[s] : (const void*)a.q[1 - s];
    if (!tc_make_map(&maps.q[s], q, a.H, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.k[s], a.k[s], a.Hkv, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
    if (!tc_make_map(&maps.v[s], a.v[s], a.Hkv, a.L, a.batch, TILE)) return cudaErrorInvalidValue;
  }
  int* status = device_status_ptr();
  if (status == nullptr) return cudaErrorUnknown;
  cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM);
  if (e != cudaSuccess) return e;
  dim3 grid(a.L / TILE, a.H, a.batch * 2);
  tc_fwd_kernel<<<grid, 128, FWD_SMEM, st>>>(maps, a, status);
  return cudaGetLastError();
}

}  // namespace bdlm
