// Bandwidth-bound kernels of the BDLM attention path: the LSE merge of partial outputs
// (Eq. csbp-lse-merge over n partials, final division included) and the
// backward preprocess D_i = sum_d dO_i,d * O_i,d.
#include <type_traits>

#include "bdlm_common.cuh"

namespace bdlm {
namespace {

using bf16 = __nv_bfloat16;
constexpr int MAX_PARTIALS = 16;

struct MergeArgs {
  const void* o[MAX_PARTIALS];
  const float* lse[MAX_PARTIALS];
  int n;
};

// Eq. csbp-lse-merge for n partials at once: with m = max_j z_j and w_j = exp(z_j - m),
//   O = sum_j w_j O_j / sum_j w_j,   z = m + log sum_j w_j.
// One thread owns EPT (8 or 16) consecutive head-dim elements of one (row, head).  It first reads the row's n LSEs
// (n <= 16: they stay in registers), takes their maximum and turns them into normalised weights w_j / sum w; an empty
// partial (z_j = -inf) gets weight 0, a row whose partials are all empty gets O = 0 and z = -inf.  Then the
// partial outputs are streamed through once, four partials' loads in flight at a time, and added up with their
// weights -- no running rescale and nothing another thread could overwrite.
// NP = the number of partials rounded up to a multiple of four: the weights are a register array of that length.
template <bool F32IN, int EPT, int NP>
__global__ void __launch_bounds__(256, 3) merge_kernel(MergeArgs ma, int64_t total_chunks, int L, int H, int d,
                                                    bf16* __restrict__ o_out, float* __restrict__ lse_out) {
  constexpr int NV = F32IN ? EPT / 4 : EPT / 8;   // 16-byte vectors per thread and partial
  const int cpr = d / EPT;   // chunks per (row, head)
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total_chunks;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx % cpr);
    const int64_t rh = idx / cpr;
    const int h = (int)(rh % H);
    const int64_t row = rh / H;
    const int64_t bidx = row / L;
    const int i = (int)(row % L);
    const int64_t lidx = (bidx * H + h) * L + i;
    // The partial outputs do not depend on the weights: the first four partials' loads go out together with the
    // LSE loads; each later group of four is requested once the group in hand has been added up.
    uint4 cur[4][NV];
    auto request = [&](int j0, uint4 (&buf)[4][NV]) {
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        if (j0 + jj < ma.n) {
          const uint4* p = F32IN ? reinterpret_cast<const uint4*>(static_cast<const float*>(ma.o[j0 + jj]) + idx * EPT)
                                 : reinterpret_cast<const uint4*>(static_cast<const bf16*>(ma.o[j0 + jj]) + idx * EPT);
#pragma unroll
          for (int v = 0; v < NV; ++v) buf[jj][v] = p[v];
        }
      }
    };
    request(0, cur);
    float wgt[NP];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < NP; ++j) {
      wgt[j] = j < ma.n ? ma.lse[j][lidx] : -INFINITY;
      m = fmaxf(m, wgt[j]);
    }
    const float m_ref = (m == -INFINITY) ? 0.f : m;   // all empty: every weight becomes exp(-inf) = 0
    float wsum = 0.f;
#pragma unroll
    for (int j = 0; j < NP; ++j) {
      wgt[j] = (wgt[j] == -INFINITY) ? 0.f : expf(wgt[j] - m_ref);
      wsum += wgt[j];
    }
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    float acc[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) acc[e] = 0.f;
#pragma unroll
    for (int j0 = 0; j0 < NP; j0 += 4) {
      if (j0 >= ma.n) break;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        if (j0 + jj >= ma.n) break;
        const float wj = wgt[j0 + jj] * inv;
        if (F32IN) {
          const float* pf = reinterpret_cast<const float*>(&cur[jj][0]);
#pragma unroll
          for (int e = 0; e < EPT; ++e) acc[e] = fmaf(wj, pf[e], acc[e]);
        } else {
          const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&cur[jj][0]);
#pragma unroll
          for (int e = 0; e < EPT / 2; ++e) {
            const float2 f = __bfloat1622float2(p2[e]);
            acc[2 * e] = fmaf(wj, f.x, acc[2 * e]);
            acc[2 * e + 1] = fmaf(wj, f.y, acc[2 * e + 1]);
          }
        }
      }
      if (j0 + 4 < ma.n) request(j0 + 4, cur);
    }
#pragma unroll
    for (int v = 0; v < EPT / 8; ++v) {
      uint4 outv;
      uint32_t* ow = reinterpret_cast<uint32_t*>(&outv);
#pragma unroll
      for (int e = 0; e < 4; ++e) ow[e] = pack_bf16(acc[8 * v + 2 * e], acc[8 * v + 2 * e + 1]);
      reinterpret_cast<uint4*>(o_out + idx * EPT)[v] = outv;
    }
    if (c == 0) lse_out[lidx] = wsum > 0.f ? m + logf(wsum) : -INFINITY;
  }
}

// D = sum over d of dO * O, fp32.  D / 8 lanes per (batch, row, head) with 16-byte loads, four rows per lane group in
// flight (the kernel is a pure stream over dO and O: enough bytes in flight per thread to keep HBM busy).
template <int D>
__global__ void __launch_bounds__(256) dsum_kernel(const bf16* __restrict__ dout, const bf16* __restrict__ o,
                                                   float* __restrict__ dsum, int64_t nrows, int L, int H) {
  constexpr int LPR = D / 8;            // lanes per row: 16 (d = 128) or 8 (d = 64)
  constexpr int RPW = 32 / LPR;         // rows per warp and pass
  constexpr int UNROLL = 4;
  const int lane = threadIdx.x & 31, sub = lane / LPR, c = lane % LPR;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t base = warp * (RPW * UNROLL);
  uint4 ua[UNROLL], ub[UNROLL];
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const int64_t w = base + j * RPW + sub;
    if (w < nrows) {
      ua[j] = *reinterpret_cast<const uint4*>(dout + w * D + c * 8);
      ub[j] = *reinterpret_cast<const uint4*>(o + w * D + c * 8);
    } else {
      ua[j] = make_uint4(0u, 0u, 0u, 0u); ub[j] = ua[j];
    }
  }
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const uint32_t* pa = reinterpret_cast<const uint32_t*>(&ua[j]);
    const uint32_t* pb = reinterpret_cast<const uint32_t*>(&ub[j]);
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pa[e]));
      const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pb[e]));
      acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
    }
#pragma unroll
    for (int sft = LPR / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    const int64_t w = base + j * RPW + sub;
    if (c == 0 && w < nrows) {
      // w indexes [batch, L, H]; D is stored [batch, H, L]
      const int h = (int)(w % H);
      const int64_t row = w / H;
      const int64_t bidx = row / L;
      const int i = (int)(row % L);
      dsum[(bidx * H + h) * L + i] = acc;
    }
  }
}

// The same sums for a tile of 32 consecutive rows x all H heads per block: dO and O are read as they lie
// ([batch, L, H, d]: the tile is one contiguous piece), the sums go through shared memory and leave as 128-byte runs
// along L of the [batch, H, L] result (written straight from the reading lanes they would be 4-byte stores H*4 apart).
constexpr int DS_LB = 32;
template <int D>
__global__ void __launch_bounds__(256) dsum_tile_kernel(const bf16* __restrict__ dout, const bf16* __restrict__ o,
                                                        float* __restrict__ dsum, int L, int H, int tiles_per_batch) {
  extern __shared__ float sums[];          // [H][DS_LB + 1]
  constexpr int LPR = D / 8;               // lanes per row
  constexpr int RPP = 256 / LPR;           // rows per pass of the block
  constexpr int UNROLL = 4;
  const int b = blockIdx.x / tiles_per_batch, l0 = (blockIdx.x % tiles_per_batch) * DS_LB;
  const int nl = min(DS_LB, L - l0);
  const int nrows = nl * H;                // rows of the tile: r = li * H + h
  const int64_t base = ((int64_t)b * L + l0) * H;
  const int sub = threadIdx.x / LPR, c = threadIdx.x % LPR;
  for (int r0 = 0; r0 < nrows; r0 += RPP * UNROLL) {
    uint4 ua[UNROLL], ub[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
      const int r = r0 + j * RPP + sub;
      if (r < nrows) {
        ua[j] = *reinterpret_cast<const uint4*>(dout + (base + r) * D + c * 8);
        ub[j] = *reinterpret_cast<const uint4*>(o + (base + r) * D + c * 8);
      } else {
        ua[j] = make_uint4(0u, 0u, 0u, 0u); ub[j] = ua[j];
      }
    }
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
      const uint32_t* pa = reinterpret_cast<const uint32_t*>(&ua[j]);
      const uint32_t* pb = reinterpret_cast<const uint32_t*>(&ub[j]);
      float acc = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pa[e]));
        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pb[e]));
        acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
      }
#pragma unroll
      for (int sft = LPR / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
      const int r = r0 + j * RPP + sub;
      if (c == 0 && r < nrows) sums[(r % H) * (DS_LB + 1) + r / H] = acc;
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < H * DS_LB; idx += 256) {
    const int h = idx / DS_LB, li = idx % DS_LB;
    if (li < nl) dsum[((int64_t)b * H + h) * L + l0 + li] = sums[h * (DS_LB + 1) + li];
  }
}

}  // namespace

cudaError_t launch_merge(int n, int batch, int L, int H, int d, const void* const* o_parts,
                         const float* const* lse_parts, int dtype, void* o_out, float* lse_out,
                         cudaStream_t st) {
  MergeArgs ma;
  ma.n = n;
  for (int j = 0; j < MAX_PARTIALS; ++j) {
    ma.o[j] = j < n ? o_parts[j] : nullptr;
    ma.lse[j] = j < n ? lse_parts[j] : nullptr;
  }
  // few partials: 16 elements per thread (more bytes in flight per thread); otherwise 8 (more warps per SM)
  const int ept = (d % 16 == 0 && n <= 3) ? 16 : 8;
  const int64_t total = (int64_t)batch * L * H * (d / ept);
  int64_t want = (total + 255) / 256;
  const int64_t cap = (int64_t)device_sm_count() * 16;
  int blocks = (int)(want < cap ? (want > 0 ? want : 1) : cap);
  bf16* oo = static_cast<bf16*>(o_out);
  auto go = [&](auto f32in, auto ept_c, auto np_c) {
    merge_kernel<decltype(f32in)::value, decltype(ept_c)::value, decltype(np_c)::value>
        <<<blocks, 256, 0, st>>>(ma, total, L, H, d, oo, lse_out);
  };
  auto by_np = [&](auto f32in, auto ept_c) {
    if (n <= 4) go(f32in, ept_c, std::integral_constant<int, 4>{});
    else if (n <= 8) go(f32in, ept_c, std::integral_constant<int, 8>{});
    else if (n <= 12) go(f32in, ept_c, std::integral_constant<int, 12>{});
    else go(f32in, ept_c, std::integral_constant<int, 16>{});
  };
  // (16 elements per thread only go with up to three partials, i.e. with four weights)
  if (dtype == 1) {
    if (ept == 16) go(std::true_type{}, std::integral_constant<int, 16>{}, std::integral_constant<int, 4>{});
    else by_np(std::true_type{}, std::integral_constant<int, 8>{});
  } else {
    if (ept == 16) go(std::false_type{}, std::integral_constant<int, 16>{}, std::integral_constant<int, 4>{});
    else by_np(std::false_type{}, std::integral_constant<int, 8>{});
  }
  return cudaGetLastError();
}

cudaError_t launch_dsum(const KArgs& a, float* dsum_clean, float* dsum_noisy, cudaStream_t st) {
  float* out[2] = {dsum_clean, dsum_noisy};
  for (int s = 0; s < 2; ++s) {
    if (a.q[s] == nullptr) continue;   // a stream without queries has no D rows
    const int rows = rows_q(a, s);
    const size_t tile_smem = (size_t)a.H * (DS_LB + 1) * sizeof(float);
    if (tile_smem <= 48 * 1024 && rows > 0) {   // the tiled form: coalesced on both sides
      const int tpb = (rows + DS_LB - 1) / DS_LB;
      const int64_t nblk = (int64_t)a.batch * tpb;
      if (nblk <= 0x7fffffff) {
        if (a.d == 128) dsum_tile_kernel<128><<<(int)nblk, 256, tile_smem, st>>>(a.dout[s], a.o[s], out[s], rows, a.H, tpb);
        else dsum_tile_kernel<64><<<(int)nblk, 256, tile_smem, st>>>(a.dout[s], a.o[s], out[s], rows, a.H, tpb);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        continue;
      }
    }
    const int64_t nrows = (int64_t)a.batch * rows * a.H;
    const int rows_per_block = 8 * (32 / (a.d / 8)) * 4;   // 8 warps, 32 / (d / 8) rows per warp and pass, 4 passes
    const int blocks = (int)((nrows + rows_per_block - 1) / rows_per_block);
    if (blocks == 0) continue;
    if (a.d == 128)
      dsum_kernel<128><<<blocks, 256, 0, st>>>(a.dout[s], a.o[s], out[s], nrows, rows, a.H);
    else
      dsum_kernel<64><<<blocks, 256, 0, st>>>(a.dout[s], a.o[s], out[s], nrows, rows, a.H);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace bdlm
