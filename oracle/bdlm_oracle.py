"""CPU oracle for the block-diffusion (BDLM) attention layer: forward, backward, LSE merge.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, fp64 statement of what the
attention layer computes.  It shares no code with the CUDA path and must never be
imported by it; only tests, the smoke check and the benchmark's CPU-baseline leg call it.

What is computed (paper section 3.2, "Block diffusion language models"; appendix A,
Eqs. correctness-clean-attention / correctness-corrupted-attention):

* A length-L clean stream and a length-L corrupted ("noisy") stream sit side by side as
  one length-2L sequence, cut into blocks of M = block_size tokens.
* Clean query at position i sees clean keys 0..i (preceding clean blocks plus causal
  access inside its own block).  `clean_mask_mode=1` is the alternative reading of
  "block-causal" (whole own block visible); mode 0 is the paper's.
* Noisy query of block b sees every noisy key of block b (bidirectional) and the clean
  keys of blocks < b; nothing else.
* Attention is softmax(q.k / sqrt(d_h)) over the visible keys (Eq.
  context-parallel-attention); LSE is the natural-log row log-sum-exp of the scaled
  scores.
* Partials over disjoint key sets combine exactly by the log-sum-exp rule
  (Eq. csbp-lse-merge, Eq. correctness-online-softmax-merge).
* The backward pass is the analytic derivative of the above for the scalar
  sum(O * dO); clean K/V gradients add up over clean and noisy queries
  (Eq. correctness-clean-gradient), noisy K/V gradients only over the own block
  (Eq. correctness-corrupted-gradient).  With grouped-query attention (not in the paper;
  query head h reads KV head h // (H / H_kv)) K/V gradients add over the group.

Array conventions: q/o/do are [batch, L, H, d]; k/v/dk/dv are [batch, L, H_kv, d];
lse is [batch, H, L]; everything float64.  Rows and keys are 0-indexed.

All functions here are pinned by tests/test_oracle_*.py against closed forms, the
paper's mask-count formulas (appendix B), library attention in special cases, finite
differences and an independent per-row brute force.  The packed form at the end of the file
(one rank's launches under Algorithms 1 and 2; DFlash2-style blocks of appendix E) is pinned
by tests/test_oracle_packed_pins.py: per-row brute force, finite differences, the identity
"ranks' results add up to the unsharded layer" and the work-balance counts of appendix B.
"""
from __future__ import annotations

import numpy as np

CLEAN = 0
NOISY = 1


# --------------------------------------------------------------------------------------
# visibility (the mask, written out)
# --------------------------------------------------------------------------------------
def visible_rows(stream, rows, L, M, clean_mask_mode=0, kv_begin=0, kv_end=None,
                 include_noisy_diag=True, window=0):
    """Boolean visibility [len(rows), 2L] of the concatenated key axis (clean keys 0..L-1
    then noisy keys L..2L-1) for the given query rows of one stream.

    Section 3.2 / Eqs. correctness-clean-attention, correctness-corrupted-attention.
    `kv_begin:kv_end` restricts the clean keys to one context shard (set C_r of Eq.
    correctness-clean-partition); `include_noisy_diag=False` drops the noisy keys, which
    leaves the clean-shard partial of a noisy query.  `window` = W > 0 is the sliding-window
    variant of a layer (appendix K mentions 1,024-token windows; the paper does not spell the
    mask out, so this is a reading): a clean key j is visible to a query at position i of either
    stream only if additionally i - j < W; the noisy keys of the own block are unaffected.
    """
    if kv_end is None:
        kv_end = L
    i = np.asarray(rows, dtype=np.int64)[:, None]
    j = np.arange(L, dtype=np.int64)[None, :]
    in_shard = (j >= kv_begin) & (j < kv_end)
    if window and window > 0:
        in_shard = in_shard & (i - j < window)
    if stream == CLEAN:
        if clean_mask_mode == 0:
            to_clean = j <= i
        else:
            to_clean = (j // M) <= (i // M)
        to_noisy = np.zeros((i.shape[0], L), dtype=bool)
    else:
        to_clean = j < (i // M) * M
        to_noisy = (j // M) == (i // M)
        if not include_noisy_diag:
            to_noisy = np.zeros_like(to_noisy)
    return np.concatenate([to_clean & in_shard, to_noisy], axis=1)


def visibility_2L(L, M, clean_mask_mode=0, kv_begin=0, kv_end=None, include_noisy_diag=True, window=0):
    """The explicit 2L x 2L mask: rows 0..L-1 clean queries, rows L..2L-1 noisy queries."""
    allrows = np.arange(L)
    top = visible_rows(CLEAN, allrows, L, M, clean_mask_mode, kv_begin, kv_end, include_noisy_diag, window)
    bot = visible_rows(NOISY, allrows, L, M, clean_mask_mode, kv_begin, kv_end, include_noisy_diag, window)
    return np.concatenate([top, bot], axis=0)


# --------------------------------------------------------------------------------------
# masked softmax attention on explicit matrices (one head)
# --------------------------------------------------------------------------------------
def _masked_attention(q, k, v, vis, scale):
    """softmax over visible keys.  q [n,d], k/v [m,d], vis [n,m] bool.
    Returns (O [n,d], LSE [n], P [n,m]).  A row with no visible key gives O = 0,
    LSE = -inf, P = 0 (empty clean prefix of the first block, appendix A step 2)."""
    s = (q @ k.T) * scale
    s = np.where(vis, s, -np.inf)
    a_max = s.max(axis=1)
    safe_max = np.where(np.isfinite(a_max), a_max, 0.0)
    e = np.exp(s - safe_max[:, None])          # exp(-inf) = 0 on hidden keys
    denom = e.sum(axis=1)
    with np.errstate(divide="ignore"):
        lse = np.where(denom > 0, safe_max + np.log(denom), -np.inf)
    p = e / np.where(denom > 0, denom, 1.0)[:, None]
    return p @ v, lse, p


def _masked_attention_grad(q, k, v, p, do, scale):
    """Derivative of sum(O*dO) for O = P V, P = softmax(scale q k^T) on the visible set.
    dV = P^T dO; dP = dO V^T; dS = P * (dP - rowsum(P*dP)); dQ = scale dS K; dK = scale dS^T Q."""
    dv = p.T @ do
    dp = do @ v.T
    ds = p * (dp - (p * dp).sum(axis=1, keepdims=True))
    dq = scale * (ds @ k)
    dk = scale * (ds.T @ q)
    return dq, dk, dv


def _check_shapes(q_clean, k_clean, q_noisy, k_noisy, M):
    B, L, H, d = q_clean.shape
    Hkv = k_clean.shape[2]
    assert q_noisy.shape == (B, L, H, d) and k_clean.shape == (B, L, Hkv, d)
    assert k_noisy.shape == (B, L, Hkv, d)
    assert H % Hkv == 0 and L % M == 0
    return B, L, H, Hkv, d


# --------------------------------------------------------------------------------------
# full-size forward / backward (explicit 2L x 2L mask per head)
# --------------------------------------------------------------------------------------
def attn_forward(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, block_size,
                 scale=None, clean_mask_mode=0, kv_begin=0, kv_end=None,
                 include_noisy_diag=True, row_chunk=2048, window=0):
    """Forward of the BDLM attention layer (Eqs. correctness-clean-attention,
    correctness-corrupted-attention; scale 1/sqrt(d_h) per Eq. context-parallel-attention).
    Returns (o_clean, lse_clean, o_noisy, lse_noisy)."""
    M = block_size
    B, L, H, Hkv, d = _check_shapes(q_clean, k_clean, q_noisy, k_noisy, M)
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    o = [np.zeros((B, L, H, d)), np.zeros((B, L, H, d))]
    lse = [np.zeros((B, H, L)), np.zeros((B, H, L))]
    qs = [q_clean, q_noisy]
    for b in range(B):
        for h in range(H):
            hk = h // G
            k2 = np.concatenate([k_clean[b, :, hk], k_noisy[b, :, hk]], axis=0)
            v2 = np.concatenate([v_clean[b, :, hk], v_noisy[b, :, hk]], axis=0)
            for stream in (CLEAN, NOISY):
                for r0 in range(0, L, row_chunk):
                    rows = np.arange(r0, min(L, r0 + row_chunk))
                    vis = visible_rows(stream, rows, L, M, clean_mask_mode, kv_begin, kv_end,
                                       include_noisy_diag, window)
                    oo, ll, _ = _masked_attention(qs[stream][b, rows, h], k2, v2, vis, scale)
                    o[stream][b, rows, h] = oo
                    lse[stream][b, h, rows] = ll
    return o[CLEAN], lse[CLEAN], o[NOISY], lse[NOISY]


def attn_backward(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, do_clean, do_noisy,
                  block_size, scale=None, clean_mask_mode=0, row_chunk=2048, window=0):
    """Backward of the layer for the scalar sum(O*dO) (Algorithm 2; Eqs.
    correctness-corrupted-gradient, correctness-clean-gradient, correctness-query-gradient).
    Returns (dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy)."""
    M = block_size
    B, L, H, Hkv, d = _check_shapes(q_clean, k_clean, q_noisy, k_noisy, M)
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    dq = [np.zeros((B, L, H, d)), np.zeros((B, L, H, d))]
    dk2 = np.zeros((B, 2 * L, Hkv, d))
    dv2 = np.zeros((B, 2 * L, Hkv, d))
    qs = [q_clean, q_noisy]
    dos = [do_clean, do_noisy]
    for b in range(B):
        for h in range(H):
            hk = h // G
            k2 = np.concatenate([k_clean[b, :, hk], k_noisy[b, :, hk]], axis=0)
            v2 = np.concatenate([v_clean[b, :, hk], v_noisy[b, :, hk]], axis=0)
            for stream in (CLEAN, NOISY):
                for r0 in range(0, L, row_chunk):
                    rows = np.arange(r0, min(L, r0 + row_chunk))
                    vis = visible_rows(stream, rows, L, M, clean_mask_mode, window=window)
                    qq = qs[stream][b, rows, h]
                    _, _, p = _masked_attention(qq, k2, v2, vis, scale)
                    gq, gk, gv = _masked_attention_grad(qq, k2, v2, p, dos[stream][b, rows, h], scale)
                    dq[stream][b, rows, h] = gq
                    dk2[b, :, hk] += gk          # sums over heads of the group and both streams
                    dv2[b, :, hk] += gv
    return dq[CLEAN], dk2[:, :L], dv2[:, :L], dq[NOISY], dk2[:, L:], dv2[:, L:]


# --------------------------------------------------------------------------------------
# LSE merge of partials over disjoint key sets
# --------------------------------------------------------------------------------------
def lse_merge(o_partials, lse_partials):
    """Combine normalised partial outputs O_j [batch, L, H, d] with row LSEs z_j
    [batch, H, L] computed over disjoint key sets (Eq. csbp-lse-merge applied left to
    right; a partial whose LSE is not finite carries weight 0, as in the guards of
    Implementation 1).  Running state is (numerator, m, normaliser); the final step is
    O = numerator / normaliser, LSE = m + log(normaliser).  All partials empty gives
    O = 0, LSE = -inf."""
    num = np.zeros_like(np.asarray(o_partials[0], dtype=np.float64))
    m = np.full(np.asarray(lse_partials[0]).shape, -np.inf)
    norm = np.zeros_like(m)
    for o_j, z_j in zip(o_partials, lse_partials):
        o_j = np.asarray(o_j, dtype=np.float64)
        z_j = np.asarray(z_j, dtype=np.float64)
        m_new = np.maximum(m, z_j)
        ref = np.where(np.isfinite(m_new), m_new, 0.0)
        w_acc = np.where(np.isfinite(m), np.exp(m - ref), 0.0)
        w_j = np.where(np.isfinite(z_j), np.exp(z_j - ref), 0.0)
        # [batch, H, L] weights against [batch, L, H, d] values
        num = np.swapaxes(w_acc, 1, 2)[..., None] * num + np.swapaxes(w_j, 1, 2)[..., None] * o_j
        norm = w_acc * norm + w_j
        m = m_new
    nz = norm > 0
    o = num / np.swapaxes(np.where(nz, norm, 1.0), 1, 2)[..., None]
    with np.errstate(divide="ignore"):
        lse = np.where(nz, m + np.log(np.where(nz, norm, 1.0)), -np.inf)
    return o, lse


# --------------------------------------------------------------------------------------
# sampled query rows (one batch element, one query head) for sizes where the full
# 2L x 2L computation does not fit
# --------------------------------------------------------------------------------------
def attn_rows(stream, rows, q_rows, k_clean, v_clean, k_noisy, v_noisy, block_size,
              do_rows=None, scale=None, clean_mask_mode=0, kv_begin=0, kv_end=None,
              include_noisy_diag=True, row_chunk=128, window=0):
    """The same definition evaluated for selected query rows of one (batch, head).

    q_rows/do_rows [n, d] belong to `rows` of `stream`; k_*/v_* are that head's KV head,
    [L, d].  Key columns hidden from every row of a chunk are dropped before the matrix
    products (they contribute exact zeros).  Returns a dict with `o` [n,d], `lse` [n] and,
    when do_rows is given, `dq` [n,d] and the rows' contributions `dk_clean`, `dv_clean`,
    `dk_noisy`, `dv_noisy` [L,d] to the K/V gradients."""
    M = block_size
    L, d = k_clean.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    rows = np.asarray(rows, dtype=np.int64)
    n = rows.shape[0]
    out = {"o": np.zeros((n, d)), "lse": np.zeros(n)}
    want_grad = do_rows is not None
    if want_grad:
        out["dq"] = np.zeros((n, d))
        dk2 = np.zeros((2 * L, d))
        dv2 = np.zeros((2 * L, d))
    order = np.argsort(rows, kind="stable")
    for c0 in range(0, n, row_chunk):
        sel = order[c0:c0 + row_chunk]
        vis = visible_rows(stream, rows[sel], L, M, clean_mask_mode, kv_begin, kv_end,
                           include_noisy_diag, window)
        cols = np.nonzero(vis.any(axis=0))[0]
        kc = np.concatenate([k_clean[cols[cols < L]], k_noisy[cols[cols >= L] - L]], axis=0)
        vc = np.concatenate([v_clean[cols[cols < L]], v_noisy[cols[cols >= L] - L]], axis=0)
        visc = vis[:, cols]
        oo, ll, p = _masked_attention(q_rows[sel], kc, vc, visc, scale)
        out["o"][sel] = oo
        out["lse"][sel] = ll
        if want_grad:
            gq, gk, gv = _masked_attention_grad(q_rows[sel], kc, vc, p, do_rows[sel], scale)
            out["dq"][sel] = gq
            dk2[cols] += gk
            dv2[cols] += gv
    if want_grad:
        out["dk_clean"], out["dk_noisy"] = dk2[:L], dk2[L:]
        out["dv_clean"], out["dv_noisy"] = dv2[:L], dv2[L:]
    return out


# --------------------------------------------------------------------------------------
# counting (used for FLOP accounting and the appendix-B pins)
# --------------------------------------------------------------------------------------
def visible_pair_counts(L, M, clean_mask_mode=0, window=0):
    """(clean pairs, noisy pairs) counted from the explicit mask, per (batch, head)."""
    vis = visibility_2L(L, M, clean_mask_mode, window=window)
    return int(vis[:L].sum()), int(vis[L:].sum())


# --------------------------------------------------------------------------------------
# packed form: what one rank of the CSBP schedule launches, and DFlash2-style blocks
# --------------------------------------------------------------------------------------
# Algorithm 1 / Algorithm 2 give a rank (a) a run of consecutive clean query positions
# (one piece of its context shard) and (b) a list of complete corrupted blocks, packed one
# after the other; both attend the full gathered clean K/V, whose keys keep their original
# positions.  Appendix E (Eq. dflash2-block-attention) has the same shape with sampled
# blocks: block b is the token at position a_b followed by M-1 masked tokens, attends its own
# M keys bidirectionally and the clean ("target-feature") keys at positions < a_b.  Both are
# described by one table: block_prefix[b] = number of leading clean keys block b sees
# (b_index * M for a BDLM block, a_b for a DFlash2 block).  Packed row i belongs to packed
# block i // M and stands at position block_prefix[i // M] + i % M (used by the window only).
def visible_rows_packed(stream, rows, Lk, M, n_blocks, block_prefix=None, clean_q_pos0=0,
                        clean_mask_mode=0, kv_begin=0, kv_end=None, include_noisy_diag=True,
                        window=0):
    """Boolean visibility [len(rows), Lk + n_blocks*M]: clean keys 0..Lk-1 (by position), then
    the packed noisy keys.  `rows` index the packed query tensor of `stream`: clean row i is
    the clean token at position clean_q_pos0 + i; noisy row i is token i % M of packed block
    i // M."""
    if kv_end is None:
        kv_end = Lk
    Ln = n_blocks * M
    if block_prefix is None:
        block_prefix = np.arange(n_blocks, dtype=np.int64) * M
    block_prefix = np.asarray(block_prefix, dtype=np.int64)
    i = np.asarray(rows, dtype=np.int64)[:, None]
    j = np.arange(Lk, dtype=np.int64)[None, :]
    in_shard = (j >= kv_begin) & (j < kv_end)
    if stream == CLEAN:
        pos = clean_q_pos0 + i
        to_clean = (j <= pos) if clean_mask_mode == 0 else ((j // M) <= (pos // M))
        to_noisy = np.zeros((i.shape[0], Ln), dtype=bool)
    else:
        pfx = block_prefix[i // M]
        pos = pfx + i % M
        to_clean = j < pfx
        jj = np.arange(Ln, dtype=np.int64)[None, :]
        to_noisy = (jj // M) == (i // M)
        if not include_noisy_diag:
            to_noisy = np.zeros_like(to_noisy)
    if window and window > 0:
        in_shard = in_shard & (pos - j < window)
    return np.concatenate([to_clean & in_shard, to_noisy], axis=1)


def attn_packed(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, block_size,
                do_clean=None, do_noisy=None, block_prefix=None, clean_q_pos0=0, scale=None,
                clean_mask_mode=0, kv_begin=0, kv_end=None, include_noisy_diag=True, window=0,
                row_chunk=1024):
    """Forward (and, when a dO is given, backward for sum(O*dO)) of the packed form.

    q_clean [B, Lq, H, d] or None: clean queries at positions clean_q_pos0 .. +Lq-1.
    q_noisy [B, n_blocks*M, H, d] or None: packed blocks; k_noisy/v_noisy [B, n_blocks*M, Hkv, d].
    k_clean/v_clean [B, Lk, Hkv, d]: every clean key, by position.
    Returns a dict: o_clean, lse_clean, o_noisy, lse_noisy (present when that q is given) and,
    with gradients, dq_clean, dq_noisy, dk_clean, dv_clean (this call's contribution for every
    clean key: Algorithm 2 reduce-scatters exactly these), dk_noisy, dv_noisy."""
    M = block_size
    B, Lk, Hkv, d = k_clean.shape
    Ln = k_noisy.shape[1]
    assert Ln % M == 0
    nb = Ln // M
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    qs = [q_clean, q_noisy]
    dos = [do_clean, do_noisy]
    names = ["clean", "noisy"]
    out = {}
    want_grad = do_clean is not None or do_noisy is not None
    if want_grad:
        dk2 = np.zeros((B, Lk + Ln, Hkv, d))
        dv2 = np.zeros((B, Lk + Ln, Hkv, d))
    for stream in (CLEAN, NOISY):
        q = qs[stream]
        if q is None:
            continue
        _, Lq, H, _ = q.shape
        G = H // Hkv
        o = np.zeros((B, Lq, H, d))
        lse = np.zeros((B, H, Lq))
        dq = np.zeros((B, Lq, H, d)) if dos[stream] is not None else None
        for b in range(B):
            for h in range(H):
                hk = h // G
                k2 = np.concatenate([k_clean[b, :, hk], k_noisy[b, :, hk]], axis=0)
                v2 = np.concatenate([v_clean[b, :, hk], v_noisy[b, :, hk]], axis=0)
                for r0 in range(0, Lq, row_chunk):
                    rows = np.arange(r0, min(Lq, r0 + row_chunk))
                    vis = visible_rows_packed(stream, rows, Lk, M, nb, block_prefix, clean_q_pos0,
                                              clean_mask_mode, kv_begin, kv_end, include_noisy_diag, window)
                    qq = q[b, rows, h]
                    oo, ll, p = _masked_attention(qq, k2, v2, vis, scale)
                    o[b, rows, h] = oo
                    lse[b, h, rows] = ll
                    if dq is not None:
                        gq, gk, gv = _masked_attention_grad(qq, k2, v2, p, dos[stream][b, rows, h], scale)
                        dq[b, rows, h] = gq
                        dk2[b, :, hk] += gk
                        dv2[b, :, hk] += gv
        out["o_" + names[stream]] = o
        out["lse_" + names[stream]] = lse
        if dq is not None:
            out["dq_" + names[stream]] = dq
    if want_grad:
        out["dk_clean"], out["dk_noisy"] = dk2[:, :Lk], dk2[:, Lk:]
        out["dv_clean"], out["dv_noisy"] = dv2[:, :Lk], dv2[:, Lk:]
    return out


def attn_rows_packed(stream, rows, q_rows, k_clean, v_clean, k_noisy, v_noisy, block_size,
                     do_rows=None, block_prefix=None, clean_q_pos0=0, scale=None, clean_mask_mode=0,
                     window=0, row_chunk=128):
    """Packed form for selected query rows of one (batch, head): the counterpart of `attn_rows`.
    k_clean/v_clean [Lk, d], k_noisy/v_noisy [n_blocks*M, d] are that head's KV head.  Returns `o`,
    `lse` and, with do_rows, `dq` and the rows' contributions dk_clean/dv_clean [Lk, d],
    dk_noisy/dv_noisy [n_blocks*M, d]."""
    M = block_size
    Lk, d = k_clean.shape
    Ln = k_noisy.shape[0]
    nb = Ln // M
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    rows = np.asarray(rows, dtype=np.int64)
    n = rows.shape[0]
    out = {"o": np.zeros((n, d)), "lse": np.zeros(n)}
    want_grad = do_rows is not None
    if want_grad:
        out["dq"] = np.zeros((n, d))
        dk2 = np.zeros((Lk + Ln, d))
        dv2 = np.zeros((Lk + Ln, d))
    order = np.argsort(rows, kind="stable")
    for c0 in range(0, n, row_chunk):
        sel = order[c0:c0 + row_chunk]
        vis = visible_rows_packed(stream, rows[sel], Lk, M, nb, block_prefix, clean_q_pos0,
                                  clean_mask_mode, window=window)
        cols = np.nonzero(vis.any(axis=0))[0]
        kc = np.concatenate([k_clean[cols[cols < Lk]], k_noisy[cols[cols >= Lk] - Lk]], axis=0)
        vc = np.concatenate([v_clean[cols[cols < Lk]], v_noisy[cols[cols >= Lk] - Lk]], axis=0)
        oo, ll, p = _masked_attention(q_rows[sel], kc, vc, vis[:, cols], scale)
        out["o"][sel] = oo
        out["lse"][sel] = ll
        if want_grad:
            gq, gk, gv = _masked_attention_grad(q_rows[sel], kc, vc, p, do_rows[sel], scale)
            out["dq"][sel] = gq
            dk2[cols] += gk
            dv2[cols] += gv
    if want_grad:
        out["dk_clean"], out["dk_noisy"] = dk2[:Lk], dk2[Lk:]
        out["dv_clean"], out["dv_noisy"] = dv2[:Lk], dv2[Lk:]
    return out
