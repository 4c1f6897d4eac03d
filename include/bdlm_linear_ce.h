/*
 * bdlm_linear_ce.h -- C ABI of the token-chunked linear cross-entropy loss for B200 (sm_100a).
 *
 * The step after the last transformer layer of BDLM training (paper section 5, "Experimental setup",
 * paragraph "Implementation and metrics": a token-chunked linear cross-entropy -- vocabulary projection
 * plus softmax cross-entropy -- that never holds the logits of the whole sequence; the loss it serves is
 * Eq. bdlm-training-objective, a weighted sum of per-token negative log-likelihoods).  For T token
 * positions with hidden states h_t, output-embedding rows W_v, targets y_t and weights w_t:
 *
 *     z_tv = h_t . W_v      lse_t = log sum_v exp(z_tv)      nll_t = lse_t - z_t,y_t   (0 if y_t < 0)
 *     loss = sum_t w_t nll_t
 *     dz_tv = grad_loss * w_t * (exp(z_tv - lse_t) - [v == y_t])     (0 for positions with y_t < 0)
 *     dH_t = sum_v dz_tv W_v        dW_v = sum_t dz_tv h_t
 *
 * Forward: one tensor-core GEMM whose epilogue keeps a running row maximum and sum of exponentials, so no
 * logit is ever written to memory.  Backward: per chunk of tokens the logits are recomputed by the same
 * GEMM, its epilogue writes dz (bf16) for that chunk into the workspace, and two more GEMMs form dH of
 * the chunk and add the chunk's share to dW; only one chunk of dz exists at a time.
 *
 * Conventions: as in bdlm_attn.h -- device pointers, contiguous, 16-byte aligned, owned by the caller;
 * nothing is allocated or freed; work is enqueued on `cuda_stream` without synchronising; outputs are
 * overwritten; the return value is 0 or a negative bdlm_status; arguments are checked before any launch.
 *   h      [T, D]  bf16        w   [V, D]  bf16 (row v = output embedding of token id v)
 *   labels [T]     int32 (negative = position ignored; otherwise < V, not checked on the host)
 *   token_weight [T] fp32 or NULL (= 1 everywhere)
 * Requirements: T >= 1, D and V multiples of 8 (rows 16-byte aligned).
 */
#ifndef BDLM_LINEAR_CE_H_
#define BDLM_LINEAR_CE_H_

#include <stddef.h>
#include <stdint.h>

#include "bdlm_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t T, D, V;
  int32_t token_chunk;   /* backward: tokens per chunk, a multiple of 128; 0 = min(T rounded up to 128, 4096).
                            A call whose workspace is too small for this chunk returns BDLM_ERR_WORKSPACE_TOO_SMALL. */
  float   grad_loss;     /* backward: upstream gradient of the scalar loss */
  int32_t reserved[3];
} bdlm_lce_params;

enum { BDLM_LCE_WS_FWD = 0, BDLM_LCE_WS_BWD = 1 };

/* Scratch bytes of a call (0 for invalid parameters).  Forward: partial (maximum, sum) pairs per token and
 * vocabulary chunk.  Backward: one chunk of dz, bf16 [token_chunk, V], plus -- when T needs more than one
 * chunk -- an fp32 dW accumulator [V, D]. */
size_t bdlm_linear_ce_workspace_bytes(const bdlm_lce_params* p, int32_t which);

/*
 * Forward.  Writes lse [T] (natural log), nll [T] (may be NULL) and the scalar loss (one float in device
 * memory; summed in a fixed order, so bitwise reproducible).
 */
int bdlm_linear_ce_fwd(const bdlm_lce_params* p, const void* h, const void* w, const int32_t* labels,
                       const float* token_weight, float* loss, float* nll, float* lse,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward.  `lse` is the forward's.  Writes dh [T, D] bf16 and dw [V, D] bf16.  dz is rounded to bf16
 * before the two gradient GEMMs; sums over the vocabulary (dH) and over the tokens of a chunk (dW) are
 * accumulated in fp32, chunks are added in fp32 in a fixed order (bitwise reproducible).
 */
int bdlm_linear_ce_bwd(const bdlm_lce_params* p, const void* h, const void* w, const int32_t* labels,
                       const float* token_weight, const float* lse, void* dh, void* dw,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* BDLM_LINEAR_CE_H_ */
