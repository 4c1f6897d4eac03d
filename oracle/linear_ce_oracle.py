"""CPU oracle for the token-chunked linear cross-entropy loss: forward and backward.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 statement of what the loss head computes.  It shares no
code with the CUDA path and must never be imported by it; only tests, the smoke check and the
benchmark's CPU-baseline leg call it.

What is computed.  The paper (section 5, "Experimental setup", paragraph "Implementation and
metrics") names a token-chunked linear cross-entropy -- the vocabulary projection followed by
softmax cross-entropy, evaluated chunk of tokens by chunk of tokens so that the logits of the
whole sequence never exist at once -- and gives no formula beyond the training objective
(Eq. bdlm-training-objective): a sum over target blocks of -w(t_b) log p(x^(b) | ...), i.e. a
weighted sum of per-token negative log-likelihoods.  Written out for T token positions with
hidden states h_t (length D), output embedding rows W_v (V rows of length D), target ids y_t and
per-token weights w_t (w(t_b) of the token's block, including any token normalisation; 0 for a
position that is not a target):

    z_tv   = h_t . W_v                                   logits
    lse_t  = log sum_v exp(z_tv)                          natural log
    nll_t  = lse_t - z_t,y_t                              0 when y_t < 0 (position ignored)
    loss   = sum_t w_t nll_t

and for an upstream scalar gradient g of the loss

    dz_tv  = g w_t (exp(z_tv - lse_t) - [v = y_t])        0 for ignored positions
    dH_t   = sum_v dz_tv W_v
    dW_v   = sum_t dz_tv h_t.

The token chunking changes nothing in these values (sums over t are split, nothing else); the
oracle takes the chunk loop as the paper states it so that a reader can see that, and the pins
check the invariance.  Pinned by tests/test_oracle_linear_ce_pins.py: torch's cross_entropy and
autograd in fp64, a pure-Python brute force, central differences, the uniform-logit closed form
and chunk-count invariance.
"""
from __future__ import annotations

import numpy as np


def _chunks(T, token_chunk):
    step = T if not token_chunk or token_chunk <= 0 else int(token_chunk)
    return [(t0, min(T, t0 + step)) for t0 in range(0, T, max(step, 1))]


def linear_ce_forward(h, W, labels, weights=None, token_chunk=None):
    """h [T, D], W [V, D], labels [T] (int; negative = ignored), weights [T] or None (= 1).
    Returns (loss scalar, nll [T], lse [T]).  One chunk of tokens at a time: logits of the chunk,
    row log-sum-exp with the maximum subtracted, the target's logit picked out."""
    h = np.asarray(h, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    y = np.asarray(labels, dtype=np.int64)
    T = h.shape[0]
    w = np.ones(T) if weights is None else np.asarray(weights, dtype=np.float64)
    nll = np.zeros(T)
    lse = np.zeros(T)
    loss = 0.0
    for t0, t1 in _chunks(T, token_chunk):
        z = h[t0:t1] @ W.T
        m = z.max(axis=1)
        lse_c = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
        yc = y[t0:t1]
        valid = yc >= 0
        picked = z[np.arange(t1 - t0), np.where(valid, yc, 0)]
        nll_c = np.where(valid, lse_c - picked, 0.0)
        lse[t0:t1] = lse_c
        nll[t0:t1] = nll_c
        loss += float((w[t0:t1] * nll_c).sum())
    return loss, nll, lse


def linear_ce_backward(h, W, labels, weights=None, grad_loss=1.0, token_chunk=None):
    """Gradients of `loss` (see linear_ce_forward) times the upstream scalar `grad_loss`.
    Returns (dH [T, D], dW [V, D]).  dW adds up over the token chunks; dH is per chunk."""
    h = np.asarray(h, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    y = np.asarray(labels, dtype=np.int64)
    T = h.shape[0]
    w = np.ones(T) if weights is None else np.asarray(weights, dtype=np.float64)
    dH = np.zeros_like(h)
    dW = np.zeros_like(W)
    for t0, t1 in _chunks(T, token_chunk):
        z = h[t0:t1] @ W.T
        m = z.max(axis=1)
        e = np.exp(z - m[:, None])
        p = e / e.sum(axis=1, keepdims=True)
        yc = y[t0:t1]
        valid = yc >= 0
        dz = p.copy()
        dz[np.nonzero(valid)[0], yc[valid]] -= 1.0
        dz *= (grad_loss * w[t0:t1] * valid)[:, None]
        dH[t0:t1] = dz @ W
        dW += dz.T @ h[t0:t1]
    return dH, dW


def linear_ce_rows(h_rows, W, labels_rows):
    """lse and nll of selected token rows only (for sizes where only a sample is checked)."""
    _, nll, lse = linear_ce_forward(h_rows, W, labels_rows, token_chunk=256)
    return nll, lse
