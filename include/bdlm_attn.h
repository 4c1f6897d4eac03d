/*
 * bdlm_attn.h -- C ABI of the block-diffusion (BDLM) attention layer for B200 (sm_100a).
 *
 * The layer (paper section 3.2; appendix A, Eqs. correctness-clean-attention and
 * correctness-corrupted-attention): a length-L clean stream and a length-L corrupted
 * ("noisy") stream, cut into blocks of `block_size` tokens.
 *   - clean query i      sees clean keys 0..i                     (clean_mask_mode 0)
 *   - noisy query i      sees noisy keys of its own block (bidirectional) and the clean
 *                        keys of all earlier blocks: j < floor(i/block_size)*block_size
 *   - sliding-window layers (appendix K of the paper mentions 1,024-token windows) restrict the clean keys
 *     further to i - j < window (`window` parameter; the paper does not spell this mask out)
 * Scores are q.k * scale (scale = 1/sqrt(d), Eq. context-parallel-attention), softmax is
 * taken over the visible keys, LSE is the natural-log row log-sum-exp of the scaled scores.
 * Partials over disjoint key sets are combined exactly by Eq. csbp-lse-merge.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers, contiguous, 16-byte aligned, owned by the
 *     caller.  The library allocates and frees nothing; work is enqueued on `cuda_stream`
 *     (a cudaStream_t passed as void*, NULL = default stream) and the call returns without
 *     synchronising.  Outputs are overwritten.
 *   - Layouts: q, o, do, dq  [batch, L, H, d]      bf16
 *              k, v, dk, dv  [batch, L, H_kv, d]   bf16   (query head h reads KV head h/(H/H_kv))
 *              lse           [batch, H, L]         fp32
 *   - Return value: 0 on success, a negative bdlm_status otherwise.  Arguments are
 *     checked before anything is launched; a failed check launches nothing.  The library
 *     never aborts, traps or prints.
 */
#ifndef BDLM_ATTN_H_
#define BDLM_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BDLM_OK = 0,
  BDLM_ERR_INVALID_ARG = -1,        /* null/misaligned pointer, bad size, H % H_kv, L % block_size, bad shard range */
  BDLM_ERR_UNSUPPORTED = -2,        /* d not in {64,128}; device is not sm_100; sharded backward */
  BDLM_ERR_WORKSPACE_TOO_SMALL = -3,
  BDLM_ERR_CUDA = -4,               /* a CUDA runtime/driver call or a launch failed */
  BDLM_ERR_DEVICE_TIMEOUT = -5,     /* a bounded device-side wait expired (see bdlm_get_device_status) */
  BDLM_ERR_STATIC_SCRATCH_TOO_SMALL = -6   /* batch*H*L exceeds BDLM_STATIC_SCRATCH_ROWS (bdlm_attn_bwd_static_scratch) */
} bdlm_status;

typedef struct {
  int32_t batch, L, block_size, H, H_kv, d;
  float   scale;               /* 0 => 1/sqrt(d) */
  int32_t clean_mask_mode;     /* 0: clean query i sees clean keys <= i (the paper's block-causal mask);
                                  1: clean query sees its whole own clean block as well */
  int32_t kv_begin, kv_end;    /* clean key positions [kv_begin, kv_end) present in this call (one context
                                  shard C_r, Eq. correctness-clean-partition).  kv_end == 0 with kv_begin == 0
                                  means 0..L unless kv_range_set != 0.  k_clean/v_clean still point at
                                  position 0 of the full [batch, L, H_kv, d] tensors. */
  int32_t kv_range_set;        /* 0: ignore kv_begin/kv_end (full range); 1: use them (may be empty) */
  int32_t include_noisy_diag;  /* 1: noisy queries also attend their own noisy block; 0: clean-shard partial only */
  int32_t impl;                /* 0: automatic (the tcgen05 kernels: head dimension 64 or 128, any length); 1: force the
                                  portable mma.sync kernels (a slow cross-check); 2: force the tcgen05 kernels */
  int32_t bwd_passes;          /* backward only: 0 = all passes; otherwise a bit set of BDLM_BWD_PASS_* to run
                                  (lets a caller time the passes separately; each pass needs the earlier ones'
                                  results from a previous call with the same workspace) */
  int32_t bwd_single_pass;     /* backward only: which kernels form the gradients (BDLM_BWD_AUTO / _FUSED / _TWO_PASS).
                                  BDLM_BWD_FUSED (1): one kernel produces dK, dV and dQ (5 GEMMs per tile pair instead of 7).
                                  Each CTA adds its dQ tiles into an fp32 accumulator in the workspace (bulk add-reductions),
                                  so dQ is reproducible only up to fp32 summation order; dK and dV are bitwise reproducible
                                  (fixed order).  Needs the workspace bdlm_workspace_bytes[_packed] reports for this setting
                                  (BDLM_ERR_WORKSPACE_TOO_SMALL otherwise); with impl = 1 (the mma.sync kernels) the
                                  two-pass path runs.
                                  BDLM_BWD_TWO_PASS (2): dK/dV pass + dQ pass, fixed summation order, every gradient
                                  bitwise reproducible; needs only the D rows in the workspace.
                                  BDLM_BWD_AUTO (0, the default of a zeroed struct): the fused kernel when the workspace
                                  passed to the call is at least the size bdlm_workspace_bytes[_packed] reports for this
                                  setting (the fused size), the two-pass path when it is smaller (it must still hold the
                                  D rows: the size reported for BDLM_BWD_TWO_PASS).
                                  With bwd_passes the fused kernel runs under BDLM_BWD_PASS_DKDV; BDLM_BWD_PASS_DQ is then
                                  a no-op. */
  int32_t window;              /* sliding-window layers: > 0 = a clean key j is visible to the query at position i (of either
                                  stream) only if additionally i - j < window; the noisy own block is unaffected.  0 = none. */
  int32_t reserved[2];
} bdlm_params;

enum { BDLM_BWD_PASS_DSUM = 1, BDLM_BWD_PASS_DKDV = 2, BDLM_BWD_PASS_DQ = 4 };
enum { BDLM_BWD_AUTO = 0, BDLM_BWD_FUSED = 1, BDLM_BWD_TWO_PASS = 2 };   /* values of bdlm_params.bwd_single_pass */

enum { BDLM_WS_FWD = 0, BDLM_WS_BWD = 1 };

/* Scratch bytes a call needs for these parameters (`which` = BDLM_WS_FWD or BDLM_WS_BWD).
 * Returns 0 when none is needed or the parameters are invalid. */
size_t bdlm_workspace_bytes(const bdlm_params* p, int32_t which);

/*
 * Forward (Algorithm 1 without the all-gather; Eq. csbp-block-attention).  For every clean
 * and noisy query row writes the normalised output and its LSE.  A stream is skipped when
 * its q pointer is NULL (its o/lse may then be NULL too).  A row whose visible key set is
 * empty in this call (possible only with a shard range or include_noisy_diag = 0) gets
 * O = 0 and LSE = -inf.
 */
int bdlm_attn_fwd(const bdlm_params* p,
                  const void* q_clean, const void* k_clean, const void* v_clean,
                  const void* q_noisy, const void* k_noisy, const void* v_noisy,
                  void* o_clean, void* o_noisy,
                  float* lse_clean, float* lse_noisy,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward (Algorithm 2 without the reduce-scatter; Eqs. correctness-corrupted-gradient,
 * correctness-clean-gradient, correctness-query-gradient).  Inputs are the forward's inputs,
 * its saved O and LSE, and the upstream gradient dO of both streams.  dK/dV of a KV head are
 * summed over the query heads of its group; clean dK/dV are summed over clean and noisy
 * queries; noisy dK/dV only over the queries of the same block.  The summation order of dK and dV
 * is fixed, so they are bitwise reproducible; dQ is too on the two-pass path, and reproducible up to
 * fp32 summation order when the fused kernel runs (see bdlm_params.bwd_single_pass for which one
 * does).  Requires the full clean key range.
 * The workspace holds D_i = sum_d dO_i,d * O_i,d and, for the fused kernel, an fp32 dQ accumulator
 * [batch, H, rows rounded up to 64, 128] per query stream; nothing in it has to be initialised or kept between calls.
 * bdlm_workspace_bytes(p, BDLM_WS_BWD) reports the size for p->bwd_single_pass; with the default
 * (BDLM_BWD_AUTO) that is the fused kernel's size, and a call given less than that -- but at least
 * the BDLM_BWD_TWO_PASS size -- runs the two-pass kernels.
 */
int bdlm_attn_bwd(const bdlm_params* p,
                  const void* q_clean, const void* k_clean, const void* v_clean,
                  const void* q_noisy, const void* k_noisy, const void* v_noisy,
                  const void* o_clean, const void* o_noisy,
                  const float* lse_clean, const float* lse_noisy,
                  const void* do_clean, const void* do_noisy,
                  void* dq_clean, void* dk_clean, void* dv_clean,
                  void* dq_noisy, void* dk_noisy, void* dv_noisy,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * LSE merge (Eq. csbp-lse-merge folded left to right; the final division and LSE write of
 * Implementation 1 are part of the same kernel).  Combines n_partials (1..16) normalised
 * partial outputs over disjoint key sets.  `o_partials` / `lse_partials` are HOST arrays of
 * device pointers: o_partials[j] is [rows, H, d] (bf16 if partial_dtype == 0, fp32 if 1),
 * lse_partials[j] is [batch, H, L] fp32 with rows = batch * L.  A partial row with a
 * non-finite LSE has weight 0; if all are empty the row gets O = 0, LSE = -inf.
 * o_out is bf16 [rows, H, d]; lse_out fp32 [batch, H, L].  o_out may be one of the bf16 partials;
 * lse_out must not be any of the partial LSE buffers (rejected with BDLM_ERR_INVALID_ARG).
 */
int bdlm_lse_merge(int32_t n_partials, int32_t batch, int32_t L, int32_t H, int32_t d,
                   const void* const* o_partials, const float* const* lse_partials,
                   int32_t partial_dtype,
                   void* o_out, float* lse_out, void* cuda_stream);

/*
 * Packed form: what one rank of the CSBP schedule launches (Algorithm 1 and Algorithm 2 of the paper), and
 * DFlash2-style blocks (appendix E, Eq. dflash2-block-attention).
 *
 *   - Clean K/V are complete and addressed by position: k_clean, v_clean, dk_clean, dv_clean are
 *     [batch, L, H_kv, d] with L = p->L (L need not be a multiple of block_size here).
 *   - Clean queries are one run of consecutive positions: q_clean, o_clean, do_clean, dq_clean are
 *     [batch, Lq_clean, H, d], lse_clean [batch, H, Lq_clean]; row i is the clean token at position
 *     clean_q_pos0 + i and sees clean keys 0 .. clean_q_pos0 + i (one piece of the rank's context shard).
 *   - Corrupted blocks are packed one after the other: every noisy tensor has n_blocks * block_size rows
 *     (queries [batch, n_blocks*block_size, H, d], K/V [batch, n_blocks*block_size, H_kv, d], lse_noisy
 *     [batch, H, n_blocks*block_size]).  Packed block b sees its own block_size noisy keys (bidirectional) and
 *     the clean keys at positions j < block_prefix[b]: block_prefix[b] = (block index) * block_size for a
 *     block of the BDLM layer, the anchor position a_b for a DFlash2 block.  block_prefix is a DEVICE array
 *     of n_blocks int32 shared by all batch elements; it must be non-decreasing (sort the blocks); NULL means
 *     b * block_size.  Row i of packed block b stands at position block_prefix[b] + i for the sliding
 *     window; with window > 0 the blocks must not overlap in position (block_prefix[b+1] >= block_prefix[b]
 *     + block_size).  Values are not validated by the library (it never reads device memory on the host).
 *   - Clean K/V in gathered order (Algorithm 1 and the paper's paragraph on its fused operator: the kernels read
 *     the all-gather's output where it lies and mask every key by the position it came from).  With kv_chunk_len > 0 the clean K/V tensors (and dK/dV)
 *     are a sequence of chunks of kv_chunk_len rows; memory chunk m holds the keys at positions
 *     kv_chunk_pos[m] .. kv_chunk_pos[m] + kv_chunk_len - 1 (for zigzag shards gathered rank by rank: chunks
 *     r and 2P-1-r of rank r, one after the other).  kv_pos_chunk is the inverse permutation.  Requirements:
 *     kv_chunk_len a multiple of 128 that divides L, chunk positions multiples of kv_chunk_len, window = 0,
 *     kv_begin a multiple of 128; otherwise BDLM_ERR_UNSUPPORTED / BDLM_ERR_INVALID_ARG.  Masks, block_prefix,
 *     clean_q_pos0 and kv_begin/kv_end are always in positions.
 *   - A query stream is left out by passing its q pointer as NULL; in the backward every tensor of that
 *     stream (for the noisy stream also K/V and dK/dV) may then be NULL.
 *   - Backward: dq_* and dk_noisy/dv_noisy are complete for the rows of this call; dk_clean/dv_clean
 *     [batch, L, H_kv, d] are THIS CALL'S contribution for every clean key (overwritten, zero where no query
 *     of the call sees the key): the reduce-scatter of Algorithm 2 adds them over the ranks' calls.
 *   - Everything else (checks, statuses, layouts, stream semantics, reproducibility) is as for
 *     bdlm_attn_fwd / bdlm_attn_bwd, bwd_single_pass included; kv_begin/kv_end select a clean shard in the
 *     forward.  Workspace of the backward: bdlm_workspace_bytes_packed(p, g, BDLM_WS_BWD).
 */
typedef struct {
  int32_t Lq_clean;             /* rows of the clean query tensors (ignored when q_clean is NULL) */
  int32_t clean_q_pos0;         /* position of clean query row 0; clean_q_pos0 + Lq_clean <= L */
  int32_t n_blocks;             /* packed corrupted blocks (ignored when q_noisy is NULL) */
  int32_t kv_chunk_len;         /* 0: clean K/V stored by position; > 0: stored as chunks of this many rows (see above) */
  const int32_t* block_prefix;  /* device, [n_blocks], non-decreasing; NULL = b * block_size */
  const int32_t* kv_chunk_pos;  /* device, [L / kv_chunk_len]: position of the first key of memory chunk m */
  const int32_t* kv_pos_chunk;  /* device, [L / kv_chunk_len]: memory chunk that holds positions c*kv_chunk_len .. (the inverse) */
} bdlm_packed_geometry;

size_t bdlm_workspace_bytes_packed(const bdlm_params* p, const bdlm_packed_geometry* g, int32_t which);

int bdlm_attn_fwd_packed(const bdlm_params* p, const bdlm_packed_geometry* g,
                         const void* q_clean, const void* k_clean, const void* v_clean,
                         const void* q_noisy, const void* k_noisy, const void* v_noisy,
                         void* o_clean, void* o_noisy, float* lse_clean, float* lse_noisy,
                         void* cuda_stream);

int bdlm_attn_bwd_packed(const bdlm_params* p, const bdlm_packed_geometry* g,
                         const void* q_clean, const void* k_clean, const void* v_clean,
                         const void* q_noisy, const void* k_noisy, const void* v_noisy,
                         const void* o_clean, const void* o_noisy,
                         const float* lse_clean, const float* lse_noisy,
                         const void* do_clean, const void* do_noisy,
                         void* dq_clean, void* dk_clean, void* dv_clean,
                         void* dq_noisy, void* dk_noisy, void* dv_noisy,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Human-readable name of a status code (static storage). */
const char* bdlm_status_string(int status);

/*
 * Synchronises `cuda_stream` and returns the device-side status word of the current
 * device: BDLM_OK, or BDLM_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded wait since the
 * last call (the word is cleared).  BDLM_ERR_CUDA if the synchronise itself failed.
 */
int bdlm_get_device_status(void* cuda_stream);

/*
 * Backward without a workspace argument (the paper has no counterpart; this exists for callers
 * that are not allowed to allocate device memory: a plug-in inside a host framework whose pool
 * already owns the whole GPU, or a latency-critical loop that cannot accept the device-wide
 * synchronisation an allocator call implies).  Same inputs, outputs, checks and kernels as
 * bdlm_attn_bwd; the D_i scratch lives in a fixed device array inside the library
 * (2 * BDLM_STATIC_SCRATCH_ROWS floats = 8 MiB, resident on every GPU that loads the library
 * until the process exits).  The call allocates and frees nothing.
 *   - It always runs the two-pass kernels (as bdlm_attn_bwd with BDLM_BWD_TWO_PASS; p->bwd_single_pass
 *     is ignored): the fused kernel's fp32 dQ accumulators would need 512 bytes per query row and head,
 *     far more than a fixed array can reasonably hold.  Every gradient is therefore bitwise reproducible.
 *   - Limit: batch * H * L <= BDLM_STATIC_SCRATCH_ROWS, otherwise
 *     BDLM_ERR_STATIC_SCRATCH_TOO_SMALL is returned and nothing is launched.  Other errors are
 *     those of bdlm_attn_bwd (an unsupported head dimension is BDLM_ERR_UNSUPPORTED here too).
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.  The address is remembered per
 *     device ordinal for the life of the device's primary context: after cudaDeviceReset (or any
 *     other teardown of that context) the library must be reloaded before this entry point is
 *     used on that device again.
 *   - All calls on a device share the one array and it keeps the previous call's contents.
 *     Nothing in it has to start at zero (each call rewrites D in full before reading it), but
 *     two calls that overlap on the GPU -- different streams, or different host threads -- race
 *     on it: serialise them.
 */
enum { BDLM_STATIC_SCRATCH_ROWS = 1 << 20 };
int bdlm_attn_bwd_static_scratch(const bdlm_params* p,
                                 const void* q_clean, const void* k_clean, const void* v_clean,
                                 const void* q_noisy, const void* k_noisy, const void* v_noisy,
                                 const void* o_clean, const void* o_noisy,
                                 const float* lse_clean, const float* lse_noisy,
                                 const void* do_clean, const void* do_noisy,
                                 void* dq_clean, void* dk_clean, void* dv_clean,
                                 void* dq_noisy, void* dk_noisy, void* dv_noisy,
                                 void* cuda_stream);

/*
 * Tracing (no counterpart in the paper; the paper reports GPU spans in its appendix K only).
 * When a device buffer of at least BDLM_TRACE_SLOTS 64-bit counters is set, the tensor-core
 * kernels add, per CTA and role, the clock cycles spent waiting and computing:
 *   slot = kernel * 16 + counter, kernel 0 = forward, 1 = dK/dV pass or the fused backward (whichever
 *   runs), 2 = dQ pass;
 *   counters 0..7 belong to compute warp 0 (0 steps, 1..5 waits/compute phases in kernel order,
 *   6 total; 7 in the fused backward: the MMA warp's wait for Q tiles), 8..11 to the MMA warp (8 total,
 *   9..11 waits), 12..13 to the producer (12 total or, fused, the MMA warp's wait for dO tiles; 13 wait
 *   for a free stage), 14..15 kernel-specific (dK/dV pass: S^T load and exponent arithmetic; fused: the
 *   read-out warpgroup's wait for dQ^T and its busy time).
 * The buffer is set per device (the device current at the call) and applies to every later launch on
 * that device from any thread.  Pass NULL to switch tracing off (the default).  The caller zeroes and
 * reads the buffer.
 */
enum { BDLM_TRACE_SLOTS = 256 };
int bdlm_set_trace_buffer(void* device_counters, size_t bytes);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait inside the
 * kernels gives up after a limit of clock ticks, raises its CTA's abort flag so that the other roles
 * leave their loops too, and the kernel reports BDLM_ERR_DEVICE_TIMEOUT through the device status
 * word instead of hanging the GPU.  This call launches a one-CTA kernel without any copy or
 * tensor-core work in which one warp waits, with a limit of `limit_ticks` clock ticks (1 .. 2^31), on
 * a barrier that nothing will ever complete, and a second warp waits on the same barrier with the
 * kernels' regular limit (about a second) and leaves as soon as the first warp has raised the flag.  Afterwards bdlm_get_device_status returns
 * BDLM_ERR_DEVICE_TIMEOUT once, and BDLM_OK on the next call.  The kernel always terminates.
 */
int bdlm_selftest_wait_timeout(int64_t limit_ticks, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* BDLM_ATTN_H_ */
