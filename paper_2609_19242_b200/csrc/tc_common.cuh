// Blackwell (sm_100a) primitives used by the tensor-memory kernels: mbarriers with bounded
// waits, TMA tile loads, tcgen05 MMA / commit / TMEM load-store, shared-memory and
// instruction descriptors.  Everything is inline PTX; no library templates.
#pragma once
#include <cuda.h>   // CUtensorMap (types only; the encoder is fetched at run time)
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bdlm {
namespace tc {

constexpr int TILE = 128;                // query rows / keys per tile
constexpr int PANEL_BYTES = TILE * 128;  // one 128-row x 64-column bf16 panel, 128-byte rows, swizzled

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait of the warp-specialised kernels: gives up after ~2^31 clock ticks (about a second), so a
// protocol slip ends the kernel with an error status instead of hanging the device; it also gives up as soon
// as another role has raised the CTA's abort flag, and raises it itself on a timeout, so every role leaves its loop.
constexpr long long WAIT_LIMIT_TICKS = 1ll << 31;
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                    long long limit_ticks = WAIT_LIMIT_TICKS) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit_ticks) { *abort_flag = 1; return false; }
    }
  }
  return true;
}

// Lean wait for the MMA-issuing thread: its instruction stream is the critical path, so the common case
// (barrier already complete) must cost a single try_wait.
__device__ __forceinline__ bool mbar_wait_lean(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_abortable(bar, parity, abort_flag);
}

// Reading the clock costs tens of cycles on a path that is otherwise a handful of instructions, so the cycle
// accounting is compiled in only for the traced instantiation of a kernel (TR = true).
template <bool TR>
__device__ __forceinline__ long long tick() {
  if constexpr (TR) return clock64(); else return 0;
}
template <bool TR>
__device__ __forceinline__ bool mbar_wait_timed(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long& acc) {
  if constexpr (TR) {
    const long long t0 = clock64();
    const bool ok = mbar_wait_abortable(bar, parity, abort_flag);
    acc += clock64() - t0;
    return ok;
  } else {
    return mbar_wait_lean(bar, parity, abort_flag);
  }
}

// Cycle accounting for the optional trace buffer: a role keeps a few local counters and adds
// them to the global slots once, when it leaves its loop.
template <bool TR>
struct Stopwatch {
  long long t;
  __device__ __forceinline__ void start() { if constexpr (TR) t = clock64(); }
  __device__ __forceinline__ void lap(long long& acc) {
    if constexpr (TR) { const long long n = clock64(); acc += n - t; t = n; }
  }
};
__device__ __forceinline__ void trace_add(unsigned long long* trace, int slot, long long v) {
  if (trace != nullptr) atomicAdd(trace + slot, static_cast<unsigned long long>(v));
}

// ---------------------------------------------------------------- fences
__device__ __forceinline__ void fence_async_smem() {   // generic-proxy smem writes -> async proxy (MMA / TMA)
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// Shared -> global add-reduction of `bytes` contiguous fp32 bytes by the TMA engine (both addresses 16-byte
// aligned, bytes a multiple of 16), tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_reduce_add_f32(float* gdst, uint32_t ssrc, uint32_t bytes) {
  asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
               ::"l"(__cvta_generic_to_global(gdst)), "r"(ssrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }   // all but the last one
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }          // reductions performed

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {   // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {    // one full warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// tcgen05.mma: D[tmem] (+)= A * B, bf16 inputs, fp32 accumulate (ss: A and B from shared memory; ts: A from tensor
// memory), and tcgen05.commit: mbarrier arrive once all MMAs issued so far by the thread have completed.
// Warp-uniform issue: when a whole warp walks the MMA loop (waits, descriptor arithmetic) and only the
// instruction itself is predicated on one elected lane, the loop stays convergent and the compiler can keep
// the descriptors in the uniform datapath; with the loop inside `if (lane == 0)` every operand is moved over
// from a vector register per instruction, and issuing one MMA costs more than the 64 clocks it runs.
__device__ __forceinline__ uint32_t elect_one() {   // 1 in exactly one lane of the (converged) warp, 0 elsewhere
  uint32_t r;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r));
  return r;
}
__device__ __forceinline__ void mma_ss_e(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate,
                                         uint32_t elected) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.ne.b32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(elected) : "memory");
}
__device__ __forceinline__ void mma_ts_e(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate,
                                         uint32_t elected) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.ne.b32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(elected) : "memory");
}
__device__ __forceinline__ void mma_commit_e(uint32_t bar, uint32_t elected) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar), "r"(elected) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (taddr.lane + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
        "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, tile base 1024-byte aligned.
//   K-major operand  (rows of 64 bf16 along the contraction dim): SBO = 1024 (8 rows), LBO unused.
//   MN-major operand (rows of 64 bf16 along M/N, one row per contraction index): LBO = stride between
//   64-element groups along M/N (one panel), SBO = 1024 (8 contraction rows).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;   // descriptor version (Blackwell)
  d |= 2ull << 61;   // SWIZZLE_128B
  return d;
}
// Instruction descriptor for kind::f16 with bf16 A/B and fp32 D.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// The MMA-issuing thread is a single scalar instruction stream: a 128x128x16 MMA occupies the
// tensor pipe for 64 clocks, so the issue path must cost well under that per instruction.
// Descriptors are therefore kept as a precomputed low word per tile (address field + LBO) plus a
// constant high word, and the k-slice offsets are compile-time constants added to the low word.
constexpr uint32_t DESC_HI = 0x40004040u;   // SBO = 1024 B (>>4 = 0x40), version 1 (bit 46), SWIZZLE_128B (2 << 61)
__device__ __forceinline__ uint32_t desc_lo_k(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t desc_lo_mn(uint32_t addr) {
  return ((addr & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(PANEL_BYTES >> 4) << 16);
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return (static_cast<uint64_t>(DESC_HI) << 32) | lo; }
__host__ __device__ constexpr uint32_t koff(int kk) { return (kk >> 2) * (PANEL_BYTES >> 4) + (kk & 3) * 2; }   // K-major slice
__host__ __device__ constexpr uint32_t moff(int kk) { return kk * 128; }                                        // MN-major slice (16 rows)
constexpr uint32_t TILE_LO = (2 * PANEL_BYTES) >> 4;   // low-word stride between consecutive 32 KB tiles

// GEMMs over a 128-deep contraction (8 k-slices of 16), issued by the elected lane of a converged warp (see
// elect_one).  Suffixes: ss = both operands in shared memory, ts = A as bf16 pairs in tensor memory; operands
// are K-major unless the name says mn/km/mm (B MN-major; A K-major and B MN-major; both MN-major).
// KS = number of 16-deep slices of the contraction: 8 for a contraction over 128 keys / queries or a head dimension of
// 128, 4 for a head dimension of 64 (the tile's second 64-column panel is then neither loaded nor read).
template <int KS = 8>
__device__ __forceinline__ void gemm_ss_e(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first, uint32_t el) {
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) mma_ss_e(d, desc64(a_lo + koff(kk)), desc64(b_lo + koff(kk)), idesc, kk == 0 ? acc_first : 1u, el);
}
template <int KS = 8>
__device__ __forceinline__ void gemm_ts_e(uint32_t d, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t acc_first, uint32_t el) {
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) mma_ts_e(d, a_tmem + kk * 8, desc64(b_lo + koff(kk)), idesc, kk == 0 ? acc_first : 1u, el);
}
template <int CW>
__device__ __forceinline__ void gemm_ts_mn_cw_e(uint32_t d, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t acc_first, uint32_t el) {
#pragma unroll
  for (int kk = 0; kk < 8; ++kk)
    mma_ts_e(d, a_tmem + ((kk * 16) / CW) * CW + ((kk * 16) % CW) / 2, desc64(b_lo + moff(kk)), idesc, kk == 0 ? acc_first : 1u, el);
}
__device__ __forceinline__ void gemm_ss_km_e(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first, uint32_t el) {
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) mma_ss_e(d, desc64(a_lo + koff(kk)), desc64(b_lo + moff(kk)), idesc, kk == 0 ? acc_first : 1u, el);
}

__device__ __forceinline__ void gemm_ss_mm_e(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first, uint32_t el) {
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) mma_ss_e(d, desc64(a_lo + moff(kk)), desc64(b_lo + moff(kk)), idesc, kk == 0 ? acc_first : 1u, el);
}

// Byte offset of element (row, col) inside a [128 x 128] bf16 tile stored as two swizzled panels
// (panel = 64 columns): the layout TMA writes with SWIZZLE_128B and the MMA reads.
__device__ __forceinline__ uint32_t sw128_offset(int row, int col) {
  const int panel = col >> 6, chunk = (col & 63) >> 3;
  return panel * PANEL_BYTES + row * 128 + (((chunk ^ (row & 7)) << 4) | ((col & 7) << 1));
}

}  // namespace tc
}  // namespace bdlm
