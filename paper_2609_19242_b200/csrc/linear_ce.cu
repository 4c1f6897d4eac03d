// Token-chunked linear cross-entropy on the 5th-generation tensor cores (paper section 5, "Implementation and
// metrics": vocabulary projection + softmax cross-entropy without the logits of the whole sequence; the loss of
// Eq. bdlm-training-objective as a weighted sum of per-token negative log-likelihoods).
//
// One persistent, warp-specialised GEMM kernel C[M x N] = A . B with a contraction of K serves every matrix product
// of the path; what differs is where the operands lie and what the epilogue does with an accumulator tile:
//
//   forward            z = H W^T            epilogue: running row maximum and sum of exponentials, target logit
//   backward, chunk    z = H_c W^T          epilogue: dz = g w_t (exp(z - lse) - onehot) as bf16 into the workspace
//                      dH_c = dz W          epilogue: bf16 store
//                      dW  += dz^T H_c      epilogue: bf16 store, or fp32 accumulation over the chunks
//
// Tiles are 128 x 256 with 64-deep contraction steps: TMA (128-byte swizzle) fills a 4-stage ring of A (16 KB) and
// B (32 KB) tiles, one warp issues tcgen05.mma (M = 128, N = 256, K = 16) into one of two 256-column accumulators in
// tensor memory, and four epilogue warps (one thread per accumulator row) drain the other one meanwhile.  An operand
// is either K-major (rows of the matrix = rows of the tile, contraction contiguous) or MN-major (rows of the matrix
// = contraction index, M/N contiguous), so W, H and dz are used as they lie in memory, never transposed.
// CTAs are persistent: work items (an M tile x a run of N tiles) are dealt round-robin in an order that keeps the
// operand shared by concurrently running CTAs in L2.  Every wait is bounded and abortable.
#include <math.h>

#include "../../include/bdlm_linear_ce.h"
#include "tc_common.cuh"
#include "tc_launch.h"

namespace bdlm {
namespace {

using namespace tc;
using bf16 = __nv_bfloat16;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int G_BARS = STAGES * STAGE_BYTES;
constexpr int G_SMEM = G_BARS + 256 + 1024;      // barriers, TMEM slot, abort flag; slack for 1024-byte alignment
constexpr int G_THREADS = 192;                   // warps 0-3 epilogue, warp 4 TMA, warp 5 MMA
constexpr int MN_PANEL = BK * 128;               // an MN-major panel: 64 contraction rows x 64 M/N elements

enum { EPI_LSE = 0, EPI_DZ = 1, EPI_STORE = 2 };
enum { C_BF16 = 0, C_F32_STORE = 1, C_F32_ADD = 2, C_F32_ADD_TO_BF16 = 3 };

struct GemmMaps { CUtensorMap a, b; };

struct GemmArgs {
  int M, N, K;
  int m_tiles, n_tiles, n_run, n_runs;   // an item = one M tile x n_run consecutive N tiles; n_runs = ceil(n_tiles / n_run)
  int m_inner;                           // item order: 1 = consecutive items share the N run, 0 = share the M tile
  int a_mn, b_mn;                        // operand layouts (0 = K-major, 1 = MN-major)
  // EPI_LSE / EPI_DZ: rows are tokens row0 .. row0 + M - 1
  int row0;
  const int* labels;
  const float* weight;
  const float* lse;
  float grad;
  float* part_m;   // [n_runs, ldp] running maxima (log2 units) per vocabulary run
  float* part_l;   // [n_runs, ldp] sums of exponentials relative to that maximum
  float* zlab;     // [ldp] logit of the target
  int ldp;
  bf16* dz;        // EPI_DZ: [M, N] row-major, ld = ldz
  int ldz;
  // EPI_STORE
  int c_mode;
  bf16* c16; float* c32; int ldc;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}

// Walks the CTA's tiles in the order every role uses.
struct TileWalk {
  int item, items, mt, nrun, nt, nt_end;
  const GemmArgs* a;
  __device__ __forceinline__ void start(const GemmArgs& args) {
    a = &args; items = args.m_tiles * args.n_runs; item = blockIdx.x; nt = 0; nt_end = 0;
    if (item < items) open();
  }
  __device__ __forceinline__ void open() {
    if (a->m_inner) { nrun = item / a->m_tiles; mt = item - nrun * a->m_tiles; }
    else { mt = item / a->n_runs; nrun = item - mt * a->n_runs; }
    nt = nrun * a->n_run;
    nt_end = min(a->n_tiles, nt + a->n_run);
  }
  __device__ __forceinline__ bool valid() const { return item < items; }
  __device__ __forceinline__ bool first_of_item() const { return nt == nrun * a->n_run; }
  __device__ __forceinline__ bool last_of_item() const { return nt + 1 == nt_end; }
  __device__ __forceinline__ void next() {
    if (++nt < nt_end) return;
    item += gridDim.x;
    if (item < items) open();
  }
};

template <int EPI>
__global__ void __launch_bounds__(G_THREADS, 1)
lce_gemm_kernel(const __grid_constant__ GemmMaps maps, const GemmArgs a, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + G_BARS;
  const uint32_t bar_full = bars /*[STAGES]*/, bar_empty = bars + 8 * STAGES /*[STAGES]*/,
                 bar_acc_full = bars + 16 * STAGES /*[2]*/, bar_acc_empty = bars + 16 * STAGES + 16 /*[2]*/;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + G_BARS + 16 * STAGES + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + G_BARS + 16 * STAGES + 40);
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_acc_full + 8 * i, 1); mbar_init(bar_acc_empty + 8 * i, 128); }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 4) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  const int nk = (a.K + BK - 1) / BK;

  if (warp == 4) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      TileWalk w;
      w.start(a);
      int ks = 0;
      bool ok = true;
      for (; w.valid() && ok; w.next()) {
        const int m0 = w.mt * BM, n0 = w.nt * BN;
        for (int k = 0; k < nk && ok; ++k, ++ks) {
          const int s = ks % STAGES;
          if (ks >= STAGES) ok = mbar_wait_abortable(bar_empty + 8 * s, ((ks / STAGES) - 1) & 1, abort_flag);
          if (!ok) break;
          const uint32_t sA = base + s * STAGE_BYTES, sB = sA + A_BYTES, bar = bar_full + 8 * s;
          mbar_expect_tx(bar, STAGE_BYTES);
          if (!a.a_mn) tma_load_2d(sA, &maps.a, bar, k * BK, m0);
          else {
#pragma unroll
            for (int p = 0; p < BM / 64; ++p) tma_load_2d(sA + p * MN_PANEL, &maps.a, bar, m0 + 64 * p, k * BK);
          }
          if (!a.b_mn) tma_load_2d(sB, &maps.b, bar, k * BK, n0);
          else {
#pragma unroll
            for (int p = 0; p < BN / 64; ++p) tma_load_2d(sB + p * MN_PANEL, &maps.b, bar, n0 + 64 * p, k * BK);
          }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop,
    // one elected lane issues
    const uint32_t el = elect_one();
    const uint32_t idesc = make_idesc(BM, BN, a.a_mn != 0, a.b_mn != 0);
    const uint32_t a_lo0 = a.a_mn ? (((base & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(MN_PANEL >> 4) << 16)) : desc_lo_k(base);
    const uint32_t b_lo0 = a.b_mn ? ((((base + A_BYTES) & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(MN_PANEL >> 4) << 16))
                                  : desc_lo_k(base + A_BYTES);
    const uint32_t a_step = a.a_mn ? 128u : 2u, b_step = a.b_mn ? 128u : 2u;   // low-word advance per 16-deep slice
    TileWalk w;
    w.start(a);
    int ks = 0, tcnt = 0;
    bool ok = true;
    for (; w.valid() && ok; w.next(), ++tcnt) {
      const int buf = tcnt & 1;
      if (tcnt >= 2) {
        ok = mbar_wait_abortable(bar_acc_empty + 8 * buf, ((tcnt >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      const uint32_t d = tmem + buf * BN;
      for (int k = 0; k < nk; ++k, ++ks) {
        const int s = ks % STAGES;
        ok = mbar_wait_lean(bar_full + 8 * s, (ks / STAGES) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_lo = a_lo0 + s * (STAGE_BYTES >> 4), b_lo = b_lo0 + s * (STAGE_BYTES >> 4);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk)
          mma_ss_e(d, desc64(a_lo + kk * a_step), desc64(b_lo + kk * b_step), idesc, (k > 0 || kk > 0) ? 1u : 0u, el);
        mma_commit_e(bar_empty + 8 * s, el);
      }
      if (!ok) break;
      mma_commit_e(bar_acc_full + 8 * buf, el);
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one thread per accumulator row
    const int r = warp * 32 + lane;
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    TileWalk w;
    w.start(a);
    int tcnt = 0;
    bool ok = true;
    // per-item row state of the forward
    float run_m = -INFINITY, run_l = 0.f;
    for (; w.valid() && ok; w.next(), ++tcnt) {
      const int buf = tcnt & 1;
      const int m0 = w.mt * BM, n0 = w.nt * BN;
      const int row = m0 + r;
      const bool row_ok = row < a.M;
      const int ncols = min(BN, a.N - n0);          // valid columns of this tile (a multiple of 8)
      int y = -1;
      float coef = 0.f, lse2 = 0.f;
      if (EPI != EPI_STORE && row_ok) {
        y = a.labels[a.row0 + row];
        if (EPI == EPI_DZ) {
          const float wt = a.weight != nullptr ? a.weight[a.row0 + row] : 1.f;
          coef = y >= 0 ? a.grad * wt : 0.f;
          lse2 = a.lse[a.row0 + row] * LOG2E;
        }
      }
      if (EPI == EPI_LSE && w.first_of_item()) { run_m = -INFINITY; run_l = 0.f; }
      ok = mbar_wait_abortable(bar_acc_full + 8 * buf, (tcnt >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t x[32];
        tmem_ld32(tl + buf * BN + c * 32, x);
        tmem_wait_ld();
        const int col0 = n0 + c * 32;
        const int cvalid = ncols - c * 32;           // columns of this chunk inside the matrix (may be <= 0 or >= 32)
        // (no `continue` below: the tensor-memory loads are warp-collective, every lane takes every iteration)
        if (EPI == EPI_LSE && cvalid > 0) {
          if (cvalid < 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (e >= cvalid) x[e] = 0xff800000u;   // -inf beyond the vocabulary
          }
          float mx = -INFINITY;
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(x[e]));
          mx *= LOG2E;
          if (mx > run_m) { run_l *= exp2f(run_m - mx); run_m = mx; }
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            s0 += exp2f(fmaf(__uint_as_float(x[e]), LOG2E, -run_m));
            s1 += exp2f(fmaf(__uint_as_float(x[e + 1]), LOG2E, -run_m));
          }
          run_l += s0 + s1;
          if ((unsigned)(y - col0) < 32u) {
            float z = 0.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) if (col0 + e == y) z = __uint_as_float(x[e]);
            a.zlab[a.row0 + row] = z;
          }
        } else if (EPI == EPI_DZ && cvalid > 0 && row_ok) {
          float p[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) p[e] = coef * exp2f(fmaf(__uint_as_float(x[e]), LOG2E, -lse2));
          if ((unsigned)(y - col0) < 32u) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (col0 + e == y) p[e] -= coef;
          }
          bf16* dst = a.dz + (int64_t)row * a.ldz + col0;
#pragma unroll
          for (int e8 = 0; e8 < 4; ++e8) {
            if (e8 * 8 < cvalid) {
              uint4 v;
              v.x = pack_bf16(p[e8 * 8 + 0], p[e8 * 8 + 1]); v.y = pack_bf16(p[e8 * 8 + 2], p[e8 * 8 + 3]);
              v.z = pack_bf16(p[e8 * 8 + 4], p[e8 * 8 + 5]); v.w = pack_bf16(p[e8 * 8 + 6], p[e8 * 8 + 7]);
              *reinterpret_cast<uint4*>(dst + e8 * 8) = v;
            }
          }
        } else if (EPI == EPI_STORE && cvalid > 0 && row_ok) {
          const int64_t off = (int64_t)row * a.ldc + col0;
#pragma unroll
          for (int e8 = 0; e8 < 4; ++e8) {
            if (e8 * 8 >= cvalid) break;
            float v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(x[e8 * 8 + e]);
            if (a.c_mode == C_F32_ADD || a.c_mode == C_F32_ADD_TO_BF16) {
              const float4 u0 = *reinterpret_cast<const float4*>(a.c32 + off + e8 * 8);
              const float4 u1 = *reinterpret_cast<const float4*>(a.c32 + off + e8 * 8 + 4);
              v[0] += u0.x; v[1] += u0.y; v[2] += u0.z; v[3] += u0.w; v[4] += u1.x; v[5] += u1.y; v[6] += u1.z; v[7] += u1.w;
            }
            if (a.c_mode == C_F32_STORE || a.c_mode == C_F32_ADD) {
              *reinterpret_cast<float4*>(a.c32 + off + e8 * 8) = make_float4(v[0], v[1], v[2], v[3]);
              *reinterpret_cast<float4*>(a.c32 + off + e8 * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
            } else {
              uint4 o;
              o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]); o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
              *reinterpret_cast<uint4*>(a.c16 + off + e8 * 8) = o;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty + 8 * buf);
      if (EPI == EPI_LSE && w.last_of_item() && row_ok) {
        a.part_m[(int64_t)w.nrun * a.ldp + a.row0 + row] = run_m;
        a.part_l[(int64_t)w.nrun * a.ldp + a.row0 + row] = run_l;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
  if (warp == 4) tmem_dealloc(tmem, 512);
}

// Combines the per-run partial (maximum, sum) pairs of every token (Eq. csbp-lse-merge's rule, in log2 units),
// writes lse and nll, and leaves one weighted partial sum of the loss per block (fixed order: reproducible).
__global__ void __launch_bounds__(256) lce_finish_kernel(const float* __restrict__ part_m, const float* __restrict__ part_l,
                                                         const float* __restrict__ zlab, const int* __restrict__ labels,
                                                         const float* __restrict__ weight, int T, int n_runs, int ldp,
                                                         float* __restrict__ lse, float* __restrict__ nll,
                                                         float* __restrict__ block_sums) {
  __shared__ float red[256];
  const int t = blockIdx.x * 256 + threadIdx.x;
  float contrib = 0.f;
  if (t < T) {
    float m = -INFINITY;
    for (int c = 0; c < n_runs; ++c) m = fmaxf(m, part_m[(int64_t)c * ldp + t]);
    float l = 0.f;
    for (int c = 0; c < n_runs; ++c) l += part_l[(int64_t)c * ldp + t] * exp2f(part_m[(int64_t)c * ldp + t] - m);
    const float z = (m + log2f(l)) * LN2;
    const int y = labels[t];
    const float n = y >= 0 ? z - zlab[t] : 0.f;
    lse[t] = z;
    if (nll != nullptr) nll[t] = n;
    contrib = (weight != nullptr ? weight[t] : 1.f) * n;
  }
  red[threadIdx.x] = contrib;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) block_sums[blockIdx.x] = red[0];
}

__global__ void __launch_bounds__(256) lce_sum_kernel(const float* __restrict__ block_sums, int n, float* __restrict__ loss) {
  __shared__ float red[256];
  float acc = 0.f;
  for (int i = threadIdx.x; i < n; i += 256) acc += block_sums[i];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *loss = red[0];
}

// ------------------------------------------------------------------------------------------ host
// Operand descriptions of one product: A is [M x K] (K-major) or [K x M] (MN-major) in memory, B likewise with N.
struct Operand { const void* ptr; int64_t ld; int mn; };

template <int EPI>
cudaError_t launch_gemm(GemmArgs a, const Operand& A, const Operand& B, cudaStream_t st) {
  GemmMaps maps;
  a.a_mn = A.mn; a.b_mn = B.mn;
  const bool okA = A.mn ? tc_make_map_2d(&maps.a, A.ptr, a.K, a.M, A.ld, 64) : tc_make_map_2d(&maps.a, A.ptr, a.M, a.K, A.ld, BM);
  const bool okB = B.mn ? tc_make_map_2d(&maps.b, B.ptr, a.K, a.N, B.ld, 64) : tc_make_map_2d(&maps.b, B.ptr, a.N, a.K, B.ld, BN);
  if (!okA || !okB) return cudaErrorInvalidValue;
  a.m_tiles = (a.M + BM - 1) / BM;
  a.n_tiles = (a.N + BN - 1) / BN;
  a.n_runs = (a.n_tiles + a.n_run - 1) / a.n_run;
  int* status = device_status_ptr();
  if (status == nullptr) return cudaErrorUnknown;
  auto kern = lce_gemm_kernel<EPI>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM);
  if (e != cudaSuccess) return e;
  const int items = a.m_tiles * a.n_runs;
  const int grid = items < device_sm_count() ? items : device_sm_count();
  kern<<<grid, G_THREADS, G_SMEM, st>>>(maps, a, status);
  return cudaGetLastError();
}

constexpr int FWD_N_RUN = 8;   // vocabulary tiles per forward work item: 2048 logits per partial (maximum, sum) pair

int fwd_runs(int V) { const int nt = (V + BN - 1) / BN; return (nt + FWD_N_RUN - 1) / FWD_N_RUN; }
size_t align256(size_t x) { return (x + 255) / 256 * 256; }
int default_chunk(const bdlm_lce_params* p) {
  if (p->token_chunk > 0) return p->token_chunk;
  const int up = (p->T + 127) / 128 * 128;
  return up < 4096 ? up : 4096;
}

int check(const bdlm_lce_params* p) {
  if (p == nullptr) return BDLM_ERR_INVALID_ARG;
  if (p->T <= 0 || p->D <= 0 || p->V <= 0 || p->D % 8 != 0 || p->V % 8 != 0) return BDLM_ERR_INVALID_ARG;
  if (p->token_chunk < 0 || p->token_chunk % 128 != 0) return BDLM_ERR_INVALID_ARG;
  if (!(p->grad_loss == p->grad_loss) || isinf(p->grad_loss)) return BDLM_ERR_INVALID_ARG;
  return BDLM_OK;
}
bool al16(const void* x) { return (reinterpret_cast<uintptr_t>(x) & 15u) == 0; }
bool sm100() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  return major == 10;
}

}  // namespace
}  // namespace bdlm

using namespace bdlm;

extern "C" {

size_t bdlm_linear_ce_workspace_bytes(const bdlm_lce_params* p, int32_t which) {
  if (check(p) != BDLM_OK) return 0;
  if (which == BDLM_LCE_WS_FWD) {
    const size_t per = align256((size_t)p->T * sizeof(float));
    return (2 * (size_t)fwd_runs(p->V) + 1) * per + align256(((size_t)p->T + 255) / 256 * sizeof(float));
  }
  if (which == BDLM_LCE_WS_BWD) {
    const int tc_ = default_chunk(p);
    const int chunks = (p->T + tc_ - 1) / tc_;
    size_t bytes = align256((size_t)tc_ * p->V * 2);
    if (chunks > 1) bytes += align256((size_t)p->V * p->D * sizeof(float));
    return bytes;
  }
  return 0;
}

int bdlm_linear_ce_fwd(const bdlm_lce_params* p, const void* h, const void* w, const int32_t* labels,
                       const float* token_weight, float* loss, float* nll, float* lse,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check(p);
  if (rc != BDLM_OK) return rc;
  const void* need[] = {h, w, labels, loss, lse, workspace};
  for (const void* x : need) if (x == nullptr) return BDLM_ERR_INVALID_ARG;
  if (!al16(h) || !al16(w) || !al16(workspace) || (reinterpret_cast<uintptr_t>(labels) & 3u) ||
      (reinterpret_cast<uintptr_t>(loss) & 3u) || (reinterpret_cast<uintptr_t>(lse) & 3u) ||
      (reinterpret_cast<uintptr_t>(nll) & 3u) || (reinterpret_cast<uintptr_t>(token_weight) & 3u))
    return BDLM_ERR_INVALID_ARG;
  if (workspace_bytes < bdlm_linear_ce_workspace_bytes(p, BDLM_LCE_WS_FWD)) return BDLM_ERR_WORKSPACE_TOO_SMALL;
  if (!sm100() || !tc_encoder_available()) return BDLM_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int runs = fwd_runs(p->V);
  const size_t per = align256((size_t)p->T * sizeof(float));
  char* ws = static_cast<char*>(workspace);
  GemmArgs a = {};
  a.M = p->T; a.N = p->V; a.K = p->D; a.n_run = FWD_N_RUN; a.m_inner = 1;
  a.row0 = 0; a.labels = labels; a.weight = token_weight; a.ldp = (int)(per / sizeof(float));
  a.part_m = reinterpret_cast<float*>(ws);
  a.part_l = reinterpret_cast<float*>(ws + (size_t)runs * per);
  a.zlab = reinterpret_cast<float*>(ws + 2 * (size_t)runs * per);
  float* block_sums = reinterpret_cast<float*>(ws + (2 * (size_t)runs + 1) * per);
  if (launch_gemm<EPI_LSE>(a, Operand{h, p->D, 0}, Operand{w, p->D, 0}, st) != cudaSuccess) return BDLM_ERR_CUDA;
  const int blocks = (p->T + 255) / 256;
  lce_finish_kernel<<<blocks, 256, 0, st>>>(a.part_m, a.part_l, a.zlab, labels, token_weight, p->T, runs, a.ldp, lse, nll, block_sums);
  if (cudaGetLastError() != cudaSuccess) return BDLM_ERR_CUDA;
  lce_sum_kernel<<<1, 256, 0, st>>>(block_sums, blocks, loss);
  return cudaGetLastError() == cudaSuccess ? BDLM_OK : BDLM_ERR_CUDA;
}

int bdlm_linear_ce_bwd(const bdlm_lce_params* p, const void* h, const void* w, const int32_t* labels,
                       const float* token_weight, const float* lse, void* dh, void* dw,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check(p);
  if (rc != BDLM_OK) return rc;
  const void* need[] = {h, w, labels, lse, dh, dw, workspace};
  for (const void* x : need) if (x == nullptr) return BDLM_ERR_INVALID_ARG;
  if (!al16(h) || !al16(w) || !al16(dh) || !al16(dw) || !al16(workspace) || (reinterpret_cast<uintptr_t>(labels) & 3u) ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) || (reinterpret_cast<uintptr_t>(token_weight) & 3u))
    return BDLM_ERR_INVALID_ARG;
  if (workspace_bytes < bdlm_linear_ce_workspace_bytes(p, BDLM_LCE_WS_BWD)) return BDLM_ERR_WORKSPACE_TOO_SMALL;
  if (!sm100() || !tc_encoder_available()) return BDLM_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int T = p->T, D = p->D, V = p->V;
  const int tc_ = default_chunk(p);
  const int chunks = (T + tc_ - 1) / tc_;
  bf16* dz = static_cast<bf16*>(workspace);
  float* dw32 = reinterpret_cast<float*>(static_cast<char*>(workspace) + align256((size_t)tc_ * V * 2));
  const bf16* hb = static_cast<const bf16*>(h);
  for (int ci = 0; ci < chunks; ++ci) {
    const int t0 = ci * tc_, rows = (T - t0) < tc_ ? (T - t0) : tc_;
    // dz of the chunk: logits again, softmax minus one-hot in the epilogue
    GemmArgs a = {};
    a.M = rows; a.N = V; a.K = D; a.n_run = FWD_N_RUN; a.m_inner = 1;
    a.row0 = t0; a.labels = labels; a.weight = token_weight; a.lse = lse; a.grad = p->grad_loss;
    a.dz = dz; a.ldz = V;
    if (launch_gemm<EPI_DZ>(a, Operand{hb + (size_t)t0 * D, D, 0}, Operand{w, D, 0}, st) != cudaSuccess) return BDLM_ERR_CUDA;
    // dH of the chunk = dz W   (contraction over the vocabulary; W as it lies is the MN-major B operand)
    GemmArgs b = {};
    b.M = rows; b.N = D; b.K = V; b.n_run = 1; b.m_inner = 1;
    b.c_mode = C_BF16; b.c16 = static_cast<bf16*>(dh) + (size_t)t0 * D; b.ldc = D;
    if (launch_gemm<EPI_STORE>(b, Operand{dz, V, 0}, Operand{w, D, 1}, st) != cudaSuccess) return BDLM_ERR_CUDA;
    // dW += dz^T H_c   (contraction over the chunk's tokens; both operands MN-major)
    GemmArgs c = {};
    c.M = V; c.N = D; c.K = rows; c.n_run = 1; c.m_inner = 0;
    c.c16 = static_cast<bf16*>(dw); c.c32 = dw32; c.ldc = D;
    c.c_mode = chunks == 1 ? C_BF16 : (ci == 0 ? C_F32_STORE : (ci + 1 < chunks ? C_F32_ADD : C_F32_ADD_TO_BF16));
    if (launch_gemm<EPI_STORE>(c, Operand{dz, V, 1}, Operand{hb + (size_t)t0 * D, D, 1}, st) != cudaSuccess) return BDLM_ERR_CUDA;
  }
  return BDLM_OK;
}

}  // extern "C"
