"""Pins for the CPU oracle: everything here checks `oracle/` against something other than
itself -- the paper's mask-count formulas (appendix B), a hand-derived micro-case, closed
forms for uniform scores, library attention in the special cases where the layer reduces
to it, an independent per-row brute force, finite differences and the invariants of the
exactness proposition (appendix A).  No GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import bdlm_oracle as orc


def _rand(shape, seed, sigma=0.5):
    return np.random.default_rng(seed).normal(size=shape) * sigma


def _inputs(B, L, H, Hkv, d, seed=0):
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    heads = [H, Hkv, Hkv, H, Hkv, Hkv]
    t = {n: _rand((B, L, h, d), seed + i) for i, (n, h) in enumerate(zip(names, heads))}
    t["doc"] = _rand((B, L, H, d), seed + 10, 1.0)
    t["don"] = _rand((B, L, H, d), seed + 11, 1.0)
    return t


# ----------------------------------------------------------------------------- masks
@pytest.mark.parametrize("L,M", [(4, 2), (16, 1), (16, 16), (48, 8), (96, 32), (60, 12), (128, 64)])
def test_mask_counts_match_appendix_B(L, M):
    """Eq. block-work-by-position: noisy block b has b*M^2 visible pairs, clean block b has
    (b-1)M^2 + M(M+1)/2; Eq. aligned-pair-work: pair sums (B+1)M^2 and B*M^2 + M;
    Eq. aligned-rank-work (P=1): totals B(B+1)M^2/2 and L(L+1)/2."""
    vis = orc.visibility_2L(L, M)
    B = L // M
    clean_per_block = vis[:L].reshape(B, M, 2 * L).sum(axis=(1, 2))
    noisy_per_block = vis[L:].reshape(B, M, 2 * L).sum(axis=(1, 2))
    for b in range(1, B + 1):
        assert noisy_per_block[b - 1] == b * M * M
        assert clean_per_block[b - 1] == (b - 1) * M * M + M * (M + 1) // 2
        assert noisy_per_block[b - 1] + noisy_per_block[B - b] == (B + 1) * M * M
        assert clean_per_block[b - 1] + clean_per_block[B - b] == B * M * M + M
    assert noisy_per_block.sum() == B * (B + 1) * M * M // 2 == L * (L + M) // 2
    assert clean_per_block.sum() == L * (L + 1) // 2
    assert orc.visible_pair_counts(L, M) == (L * (L + 1) // 2, L * (L + M) // 2)
    # every noisy row of block b sees exactly b*M keys; clean row i sees i+1
    assert (vis[L:].sum(axis=1) == (np.arange(L) // M + 1) * M).all()
    assert (vis[:L].sum(axis=1) == np.arange(L) + 1).all()


def test_mask_micro_case_L4_M2():
    """Section 3.2 written out for L=4, M=2 (keys c0..c3 then n0..n3)."""
    vis = orc.visibility_2L(4, 2).astype(int)
    expect = np.array([
        # c0 c1 c2 c3 n0 n1 n2 n3
        [1, 0, 0, 0, 0, 0, 0, 0],   # clean 0
        [1, 1, 0, 0, 0, 0, 0, 0],   # clean 1
        [1, 1, 1, 0, 0, 0, 0, 0],   # clean 2
        [1, 1, 1, 1, 0, 0, 0, 0],   # clean 3
        [0, 0, 0, 0, 1, 1, 0, 0],   # noisy 0 (block 0: empty prefix)
        [0, 0, 0, 0, 1, 1, 0, 0],   # noisy 1
        [1, 1, 0, 0, 0, 0, 1, 1],   # noisy 2 (block 1: clean block 0 + own block)
        [1, 1, 0, 0, 0, 0, 1, 1],   # noisy 3
    ])
    assert (vis == expect).all()
    assert expect[:4].sum() == 10 and expect[4:].sum() == 12


def test_clean_never_sees_noisy_and_noisy_never_sees_own_clean_block():
    L, M = 32, 8
    vis = orc.visibility_2L(L, M)
    assert not vis[:L, L:].any()
    for i in range(L):
        b = i // M
        assert not vis[L + i, b * M:L].any()           # own and later clean blocks hidden
        assert vis[L + i, :b * M].all()
        assert vis[L + i, L + b * M:L + (b + 1) * M].all()
        assert vis[L + i, L:].sum() == M


def test_mask_mode1_whole_own_clean_block():
    L, M = 24, 6
    vis = orc.visibility_2L(L, M, clean_mask_mode=1)
    for i in range(L):
        assert vis[i, :L].sum() == (i // M + 1) * M


def test_shard_masks_partition_the_full_mask():
    """Eq. correctness-clean-partition: shard masks plus the diagonal-only mask are
    disjoint and their union is the full mask."""
    L, M = 48, 8
    full = orc.visibility_2L(L, M)
    parts = [orc.visibility_2L(L, M, kv_begin=a, kv_end=b, include_noisy_diag=False)
             for a, b in [(0, 16), (16, 20), (20, 48)]]
    parts.append(orc.visibility_2L(L, M, kv_begin=0, kv_end=0))
    assert (sum(p.astype(int) for p in parts) == full.astype(int)).all()


# ---------------------------------------------------------------- uniform-score closed form
def test_uniform_scores_closed_form():
    """With q = 0 every visible key has weight 1/n: LSE = ln(n), O = mean of visible v,
    dV_j = sum over rows that see j of dO_i / n_i, dQ = dK = 0 when dP - D vanishes is not
    assumed: dQ is checked to be scale * sum_j P_ij (dP_ij - D_i) k_j by direct loops."""
    B, L, H, Hkv, d, M = 1, 24, 2, 1, 4, 6
    t = _inputs(B, L, H, Hkv, d, seed=3)
    t["qc"][:] = 0
    t["qn"][:] = 0
    oc, lc, on, ln = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M)
    for i in range(L):
        b = i // M
        assert np.allclose(lc[0, :, i], math.log(i + 1), atol=1e-12)
        assert np.allclose(ln[0, :, i], math.log((b + 1) * M), atol=1e-12)   # bM visible keys
        assert np.allclose(oc[0, i, 0], t["vc"][0, :i + 1, 0].mean(axis=0), atol=1e-12)
        vis_v = np.concatenate([t["vc"][0, :b * M, 0], t["vn"][0, b * M:(b + 1) * M, 0]])
        assert np.allclose(on[0, i, 1], vis_v.mean(axis=0), atol=1e-12)
    g = orc.attn_backward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], t["doc"], t["don"], M)
    dvc_expect = np.zeros((L, d))
    dvn_expect = np.zeros((L, d))
    for h in range(H):
        for i in range(L):
            b = i // M
            dvc_expect[:i + 1] += t["doc"][0, i, h] / (i + 1)
            dvc_expect[:b * M] += t["don"][0, i, h] / ((b + 1) * M)
            dvn_expect[b * M:(b + 1) * M] += t["don"][0, i, h] / ((b + 1) * M)
    assert np.allclose(g[2][0, :, 0], dvc_expect, atol=1e-12)
    assert np.allclose(g[5][0, :, 0], dvn_expect, atol=1e-12)
    # q = 0 => dK = scale * dS^T q = 0
    assert np.abs(g[1]).max() == 0 and np.abs(g[4]).max() == 0


def test_softmax_rows_sum_to_one():
    """With V = 1 the output is the row sum of P."""
    B, L, H, Hkv, d, M = 2, 32, 4, 2, 8, 4
    t = _inputs(B, L, H, Hkv, d, seed=5)
    t["vc"][:] = 1.0
    t["vn"][:] = 1.0
    oc, _, on, _ = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M)
    assert np.allclose(oc, 1.0, atol=1e-13) and np.allclose(on, 1.0, atol=1e-13)


# ---------------------------------------------------------- reduction to library attention
def _sdpa(q, k, v, causal):
    """torch scaled_dot_product_attention in fp64 on [L, H, d] arrays, with autograd."""
    tq, tk, tv = (torch.tensor(np.moveaxis(x, 1, 0)[None], dtype=torch.float64, requires_grad=True)
                  for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal)
    return o, (tq, tk, tv)


def test_block_size_1_clean_stream_is_causal_attention():
    B, L, H, d, M = 1, 40, 3, 16, 1
    t = _inputs(B, L, H, H, d, seed=7)
    oc, lc, on, ln = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M)
    o_ref, (tq, tk, tv) = _sdpa(t["qc"][0], t["kc"][0], t["vc"][0], causal=True)
    assert np.allclose(oc[0], np.moveaxis(o_ref[0].detach().numpy(), 0, 1), atol=1e-12)
    # gradient of the clean stream alone: zero dO on the noisy stream
    g = orc.attn_backward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"],
                          t["doc"], np.zeros_like(t["don"]), M)
    (o_ref * torch.tensor(np.moveaxis(t["doc"][0], 1, 0)[None])).sum().backward()
    for got, ref in zip(g[:3], (tq, tk, tv)):
        assert np.allclose(got[0], np.moveaxis(ref.grad[0].numpy(), 0, 1), atol=1e-11)
    assert np.abs(g[3]).max() == 0      # no dO on noisy rows => no noisy dQ


def test_block_size_L_noisy_stream_is_full_bidirectional_attention():
    B, L, H, d = 1, 24, 2, 8
    M = L
    t = _inputs(B, L, H, H, d, seed=9)
    oc, lc, on, ln = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M)
    o_ref, (tq, tk, tv) = _sdpa(t["qn"][0], t["kn"][0], t["vn"][0], causal=False)
    assert np.allclose(on[0], np.moveaxis(o_ref[0].detach().numpy(), 0, 1), atol=1e-12)
    s = np.einsum("ihd,jhd->hij", t["qn"][0], t["kn"][0]) / math.sqrt(d)
    assert np.allclose(ln[0], torch.logsumexp(torch.tensor(s), dim=-1).numpy(), atol=1e-12)
    g = orc.attn_backward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"],
                          np.zeros_like(t["doc"]), t["don"], M)
    (o_ref * torch.tensor(np.moveaxis(t["don"][0], 1, 0)[None])).sum().backward()
    for got, ref in zip(g[3:], (tq, tk, tv)):
        assert np.allclose(got[0], np.moveaxis(ref.grad[0].numpy(), 0, 1), atol=1e-11)
    assert np.abs(g[1]).max() == 0 and np.abs(g[2]).max() == 0   # empty prefix: clean K/V untouched


def test_matches_library_masked_attention_with_autograd_gqa():
    """General case against torch: additive mask built here by loops (not by the oracle),
    GQA by repeating KV heads, gradients by autograd."""
    B, L, H, Hkv, d, M = 2, 24, 4, 2, 8, 6
    G = H // Hkv
    t = _inputs(B, L, H, Hkv, d, seed=11)
    mask = torch.full((2 * L, 2 * L), -float("inf"), dtype=torch.float64)
    for i in range(L):
        for j in range(L):
            if j <= i:
                mask[i, j] = 0
            if j < (i // M) * M:
                mask[L + i, j] = 0
            if j // M == i // M:
                mask[L + i, L + j] = 0
    tt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in t.items()
          if k in ("qc", "kc", "vc", "qn", "kn", "vn")}
    q2 = torch.cat([tt["qc"], tt["qn"]], dim=1).permute(0, 2, 1, 3)
    k2 = torch.cat([tt["kc"], tt["kn"]], dim=1).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    v2 = torch.cat([tt["vc"], tt["vn"]], dim=1).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    s = q2 @ k2.transpose(-1, -2) / math.sqrt(d) + mask
    o2 = torch.softmax(s, dim=-1) @ v2
    lse2 = torch.logsumexp(s, dim=-1)
    do2 = torch.tensor(np.concatenate([t["doc"], t["don"]], axis=1)).permute(0, 2, 1, 3)
    (o2 * do2).sum().backward()
    oc, lc, on, ln = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M)
    o2n = o2.detach().permute(0, 2, 1, 3).numpy()
    assert np.allclose(oc, o2n[:, :L], atol=1e-12) and np.allclose(on, o2n[:, L:], atol=1e-12)
    assert np.allclose(lc, lse2[:, :, :L].detach().numpy(), atol=1e-12)
    assert np.allclose(ln, lse2[:, :, L:].detach().numpy(), atol=1e-12)
    g = orc.attn_backward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], t["doc"], t["don"], M)
    for got, name in zip(g, ["qc", "kc", "vc", "qn", "kn", "vn"]):
        assert np.allclose(got, tt[name].grad.numpy(), atol=1e-11), name


# ------------------------------------------------------------ independent brute force
def _brute(t, M, mode=0):
    """Per-row Python loops over the visible set; no matrix code, no oracle code."""
    B, L, H, d = t["qc"].shape
    Hkv = t["kc"].shape[2]
    G = H // Hkv
    sc = 1 / math.sqrt(d)
    out = {n: np.zeros_like(t[s]) for n, s in
           [("oc", "qc"), ("on", "qn"), ("dqc", "qc"), ("dqn", "qn"), ("dkc", "kc"),
            ("dvc", "vc"), ("dkn", "kn"), ("dvn", "vn")]}
    out["lc"] = np.zeros((B, H, L))
    out["ln"] = np.zeros((B, H, L))
    for b in range(B):
        for h in range(H):
            hk = h // G
            for stream in ("c", "n"):
                for i in range(L):
                    blk = i // M
                    if stream == "c":
                        hi = i + 1 if mode == 0 else (blk + 1) * M
                        keys = [("c", j) for j in range(hi)]
                    else:
                        keys = [("c", j) for j in range(blk * M)] + \
                               [("n", j) for j in range(blk * M, (blk + 1) * M)]
                    q = t["q" + stream][b, i, h]
                    do = t["do" + stream][b, i, h]
                    a = [sc * float(np.dot(q, t["k" + s][b, j, hk])) for s, j in keys]
                    amax = max(a)
                    w = [math.exp(x - amax) for x in a]
                    z = sum(w)
                    p = [x / z for x in w]
                    o = sum(pj * t["v" + s][b, j, hk] for pj, (s, j) in zip(p, keys))
                    out["o" + stream][b, i, h] = o
                    out["l" + stream][b, h, i] = amax + math.log(z)
                    dp = [float(np.dot(do, t["v" + s][b, j, hk])) for s, j in keys]
                    dsum = sum(pj * dpj for pj, dpj in zip(p, dp))
                    for pj, dpj, (s, j) in zip(p, dp, keys):
                        ds = pj * (dpj - dsum)
                        out["dq" + stream][b, i, h] += sc * ds * t["k" + s][b, j, hk]
                        out["dk" + s][b, j, hk] += sc * ds * q
                        out["dv" + s][b, j, hk] += pj * do
    return out


@pytest.mark.parametrize("L,M,H,Hkv,mode", [(16, 4, 4, 2, 0), (12, 3, 2, 2, 0), (8, 8, 2, 1, 0),
                                             (8, 1, 2, 2, 0), (12, 4, 2, 1, 1)])
def test_against_brute_force(L, M, H, Hkv, mode):
    t = _inputs(2, L, H, Hkv, 4, seed=13)
    ref = _brute(t, M, mode)
    oc, lc, on, ln = orc.attn_forward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M,
                                      clean_mask_mode=mode)
    g = orc.attn_backward(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], t["doc"], t["don"],
                          M, clean_mask_mode=mode)
    for got, name in zip((oc, lc, on, ln) + g,
                         ["oc", "lc", "on", "ln", "dqc", "dkc", "dvc", "dqn", "dkn", "dvn"]):
        assert np.allclose(got, ref[name], atol=1e-12), name


# ---------------------------------------------------------------- finite differences
def test_gradients_by_central_differences():
    B, L, H, Hkv, d, M = 1, 12, 2, 1, 4, 4
    t = _inputs(B, L, H, Hkv, d, seed=17)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]

    def loss(tt):
        oc, _, on, _ = orc.attn_forward(*[tt[n] for n in names], M)
        return (oc * t["doc"]).sum() + (on * t["don"]).sum()

    g = orc.attn_backward(*[t[n] for n in names], t["doc"], t["don"], M)
    rng = np.random.default_rng(0)
    eps = 1e-5
    for name, grad in zip(names, g):
        for _ in range(12):
            idx = tuple(int(rng.integers(0, s)) for s in t[name].shape)
            tp = {k: v.copy() for k, v in t.items()}
            tm = {k: v.copy() for k, v in t.items()}
            tp[name][idx] += eps
            tm[name][idx] -= eps
            fd = (loss(tp) - loss(tm)) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


# ------------------------------------------------- exactness-proposition invariants
def test_block_independence():
    """Eq. correctness-block-dependency: noisy Q/K/V of block b' do not reach any other
    block's output nor any clean output; Eq. correctness-corrupted-gradient: noisy dK/dV of
    block b ignore dO outside block b."""
    B, L, H, Hkv, d, M = 1, 32, 2, 1, 8, 8
    t = _inputs(B, L, H, Hkv, d, seed=19)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    base = orc.attn_forward(*[t[n] for n in names], M)
    t2 = {k: v.copy() for k, v in t.items()}
    blk = slice(8, 16)
    for n in ("qn", "kn", "vn"):
        t2[n][:, blk] += 1.0
    pert = orc.attn_forward(*[t2[n] for n in names], M)
    assert np.array_equal(base[0], pert[0]) and np.array_equal(base[1], pert[1])
    keep = np.ones(L, bool)
    keep[blk] = False
    assert np.array_equal(base[2][:, keep], pert[2][:, keep])
    assert not np.allclose(base[2][:, blk], pert[2][:, blk])
    g1 = orc.attn_backward(*[t[n] for n in names], t["doc"], t["don"], M)
    don2 = t["don"].copy()
    don2[:, keep] *= -3.0
    g2 = orc.attn_backward(*[t[n] for n in names], t["doc"] * 2, don2, M)
    assert np.allclose(g1[4][:, blk], g2[4][:, blk], atol=1e-14)
    assert np.allclose(g1[5][:, blk], g2[5][:, blk], atol=1e-14)


def test_clean_stream_independent_of_block_size():
    B, L, H, Hkv, d = 1, 24, 2, 2, 8
    t = _inputs(B, L, H, Hkv, d, seed=23)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    ref = orc.attn_forward(*[t[n] for n in names], 1)
    for M in (2, 3, 4, 6, 8, 12, 24):
        got = orc.attn_forward(*[t[n] for n in names], M)
        assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


@pytest.mark.parametrize("cuts", [[0, 48], [0, 8, 48], [0, 5, 17, 32, 48], [0, 16, 16, 48]])
def test_shard_partials_merge_to_unsharded(cuts):
    """Eq. correctness-online-softmax-merge: partials over any partition of the clean keys,
    plus the noisy-diagonal partial, merge to the unsharded result."""
    B, L, H, Hkv, d, M = 2, 48, 4, 2, 8, 8
    t = _inputs(B, L, H, Hkv, d, seed=29)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    full = orc.attn_forward(*[t[n] for n in names], M)
    parts = [orc.attn_forward(*[t[n] for n in names], M, kv_begin=a, kv_end=b,
                              include_noisy_diag=False) for a, b in zip(cuts[:-1], cuts[1:])]
    diag = orc.attn_forward(*[t[n] for n in names], M, kv_begin=0, kv_end=0)
    assert np.isneginf(diag[1]).all() and np.abs(diag[0]).max() == 0   # clean rows: empty set
    oc, lc = orc.lse_merge([p[0] for p in parts], [p[1] for p in parts])
    on, ln = orc.lse_merge([p[2] for p in parts] + [diag[2]], [p[3] for p in parts] + [diag[3]])
    for got, ref in zip((oc, lc, on, ln), full):
        assert np.allclose(got, ref, atol=1e-12)
    # first noisy block has an empty clean prefix in every shard partial
    assert np.isneginf(parts[0][3][:, :, :M]).all()


def test_merge_special_cases():
    """Eq. csbp-lse-merge: equal LSEs average the outputs and add ln 2; an empty side
    (-inf) leaves the other unchanged; all empty gives O = 0, LSE = -inf; order-free."""
    rng = np.random.default_rng(31)
    o1, o2, o3 = (rng.normal(size=(1, 5, 2, 3)) for _ in range(3))
    z = rng.normal(size=(1, 2, 5))
    o, l = orc.lse_merge([o1, o2], [z, z])
    assert np.allclose(o, (o1 + o2) / 2, atol=1e-15) and np.allclose(l, z + math.log(2), atol=1e-15)
    ninf = np.full_like(z, -np.inf)
    o, l = orc.lse_merge([o1, o2], [z, ninf])
    assert np.array_equal(o, o1) and np.array_equal(l, z)
    o, l = orc.lse_merge([o1, o2], [ninf, z])
    assert np.array_equal(o, o2) and np.array_equal(l, z)
    o, l = orc.lse_merge([o1, o2], [ninf, ninf])
    assert np.abs(o).max() == 0 and np.isneginf(l).all()
    z2, z3 = rng.normal(size=z.shape) * 5, rng.normal(size=z.shape) * 5
    a = orc.lse_merge([o1, o2, o3], [z, z2, z3])
    b = orc.lse_merge([o3, o1, o2], [z3, z, z2])
    assert np.allclose(a[0], b[0], atol=1e-14) and np.allclose(a[1], b[1], atol=1e-14)
    # two-set formula typed out: w_j = exp(z_j - m)
    m = np.maximum(z, z2)
    w1, w2 = np.exp(z - m), np.exp(z2 - m)
    o, l = orc.lse_merge([o1, o2], [z, z2])
    w1b, w2b = np.swapaxes(w1, 1, 2)[..., None], np.swapaxes(w2, 1, 2)[..., None]
    assert np.allclose(o, (w1b * o1 + w2b * o2) / (w1b + w2b), atol=1e-15)
    assert np.allclose(l, m + np.log(w1 + w2), atol=1e-15)


# --------------------------------------------------------- sampled rows = full oracle
@pytest.mark.parametrize("mode", [0, 1])
def test_sampled_rows_equal_full_oracle(mode):
    B, L, H, Hkv, d, M = 1, 64, 2, 1, 8, 8
    t = _inputs(B, L, H, Hkv, d, seed=37)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    full = orc.attn_forward(*[t[n] for n in names], M, clean_mask_mode=mode)
    rows = np.array([0, 1, 7, 8, 9, 31, 40, 63])
    for h in range(H):
        # gradients with dO zero outside the sampled rows of this one head
        doc = np.zeros_like(t["doc"])
        don = np.zeros_like(t["don"])
        doc[0, rows, h] = t["doc"][0, rows, h]
        don[0, rows, h] = t["don"][0, rows, h]
        g = orc.attn_backward(*[t[n] for n in names], doc, don, M, clean_mask_mode=mode)
        rc = orc.attn_rows(orc.CLEAN, rows, t["qc"][0, rows, h], t["kc"][0, :, 0], t["vc"][0, :, 0],
                           t["kn"][0, :, 0], t["vn"][0, :, 0], M, do_rows=t["doc"][0, rows, h],
                           clean_mask_mode=mode, row_chunk=3)
        rn = orc.attn_rows(orc.NOISY, rows, t["qn"][0, rows, h], t["kc"][0, :, 0], t["vc"][0, :, 0],
                           t["kn"][0, :, 0], t["vn"][0, :, 0], M, do_rows=t["don"][0, rows, h],
                           clean_mask_mode=mode, row_chunk=3)
        assert np.allclose(rc["o"], full[0][0, rows, h], atol=1e-13)
        assert np.allclose(rc["lse"], full[1][0, h, rows], atol=1e-13)
        assert np.allclose(rn["o"], full[2][0, rows, h], atol=1e-13)
        assert np.allclose(rn["lse"], full[3][0, h, rows], atol=1e-13)
        assert np.allclose(rc["dq"], g[0][0, rows, h], atol=1e-13)
        assert np.allclose(rn["dq"], g[3][0, rows, h], atol=1e-13)
        assert np.allclose(rc["dk_clean"] + rn["dk_clean"], g[1][0, :, 0], atol=1e-13)
        assert np.allclose(rc["dv_clean"] + rn["dv_clean"], g[2][0, :, 0], atol=1e-13)
        assert np.allclose(rn["dk_noisy"], g[4][0, :, 0], atol=1e-13)
        assert np.allclose(rn["dv_noisy"], g[5][0, :, 0], atol=1e-13)
        assert np.abs(rc["dk_noisy"]).max() == 0


# ------------------------------------------------------------------ sliding-window variant
@pytest.mark.parametrize("L,M,W", [(32, 4, 8), (48, 8, 5), (24, 6, 6), (32, 8, 100), (40, 1, 7)])
def test_window_mask_counts_and_shape(L, M, W):
    """Reading of the sliding-window layers (appendix K): clean key j visible to position i only if i - j < W.
    Clean row i then sees min(i+1, W) keys; noisy row i of block b sees its M noisy keys plus the clean keys
    of (i-W, bM); with W >= L the mask is the unwindowed one."""
    vis = orc.visibility_2L(L, M, window=W)
    for i in range(L):
        b = i // M
        assert vis[i, :L].sum() == min(i + 1, W)
        lo = max(0, i - W + 1)
        assert vis[L + i, :L].sum() == max(0, b * M - lo)
        if b * M > lo:
            assert vis[L + i, lo:b * M].all()
        assert vis[L + i, L:].sum() == M
        assert not vis[i, L:].any()
    if W >= L:
        assert (vis == orc.visibility_2L(L, M)).all()
    c, n = orc.visible_pair_counts(L, M, window=W)
    assert c == sum(min(i + 1, W) for i in range(L))


def test_window_clean_stream_is_library_sliding_window_attention():
    """M = 1: the clean stream under a window is ordinary causal sliding-window attention; compared with
    torch SDPA given a band mask built here by loops, values and autograd gradients."""
    B, L, H, d, M, W = 1, 40, 2, 8, 1, 6
    t = _inputs(B, L, H, H, d, seed=41)
    band = torch.zeros(L, L, dtype=torch.bool)
    for i in range(L):
        for j in range(L):
            band[i, j] = (j <= i) and (i - j < W)
    tq, tk, tv = (torch.tensor(np.moveaxis(x[0], 1, 0)[None], dtype=torch.float64, requires_grad=True)
                  for x in (t["qc"], t["kc"], t["vc"]))
    o_ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=band)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    oc, lc, on, ln = orc.attn_forward(*[t[n] for n in names], M, window=W)
    assert np.allclose(oc[0], np.moveaxis(o_ref[0].detach().numpy(), 0, 1), atol=1e-12)
    g = orc.attn_backward(*[t[n] for n in names], t["doc"], np.zeros_like(t["don"]), M, window=W)
    (o_ref * torch.tensor(np.moveaxis(t["doc"][0], 1, 0)[None])).sum().backward()
    for got, ref in zip(g[:3], (tq, tk, tv)):
        assert np.allclose(got[0], np.moveaxis(ref.grad[0].numpy(), 0, 1), atol=1e-11)


def test_window_against_brute_force_and_rows():
    """General windowed case against per-row loops over the visible set, and the sampled-row path."""
    B, L, H, Hkv, d, M, W = 1, 24, 2, 1, 4, 6, 9
    t = _inputs(B, L, H, Hkv, d, seed=43)
    names = ["qc", "kc", "vc", "qn", "kn", "vn"]
    oc, lc, on, ln = orc.attn_forward(*[t[n] for n in names], M, window=W)
    sc = 1 / math.sqrt(d)
    for h in range(H):
        for i in range(L):
            blk = i // M
            for stream, q, o_got, l_got in (("c", t["qc"], oc, lc), ("n", t["qn"], on, ln)):
                if stream == "c":
                    keys = [("c", j) for j in range(max(0, i - W + 1), i + 1)]
                else:
                    keys = [("c", j) for j in range(max(0, i - W + 1), blk * M)] + [("n", j) for j in range(blk * M, (blk + 1) * M)]
                a = np.array([sc * np.dot(q[0, i, h], t["k" + s][0, j, 0]) for s, j in keys])
                w_ = np.exp(a - a.max())
                o = sum(wj * t["v" + s][0, j, 0] for wj, (s, j) in zip(w_ / w_.sum(), keys))
                assert np.allclose(o_got[0, i, h], o, atol=1e-12)
                assert abs(l_got[0, h, i] - (a.max() + math.log(w_.sum()))) < 1e-12
    rows = np.array([0, 5, 6, 13, 23])
    full_g = None
    for h in range(H):
        r = orc.attn_rows(orc.NOISY, rows, t["qn"][0, rows, h], t["kc"][0, :, 0], t["vc"][0, :, 0],
                          t["kn"][0, :, 0], t["vn"][0, :, 0], M, window=W)
        assert np.allclose(r["o"], on[0, rows, h], atol=1e-13) and np.allclose(r["lse"], ln[0, h, rows], atol=1e-13)
    # gradients by central differences under the window
    g = orc.attn_backward(*[t[n] for n in names], t["doc"], t["don"], M, window=W)

    def loss(tt):
        a_, _, b_, _ = orc.attn_forward(*[tt[n] for n in names], M, window=W)
        return (a_ * t["doc"]).sum() + (b_ * t["don"]).sum()
    rng = np.random.default_rng(1)
    for name, grad in zip(names, g):
        for _ in range(6):
            idx = tuple(int(rng.integers(0, s_)) for s_ in t[name].shape)
            tp = {k: v.copy() for k, v in t.items()}
            tm = {k: v.copy() for k, v in t.items()}
            tp[name][idx] += 1e-5
            tm[name][idx] -= 1e-5
            fd = (loss(tp) - loss(tm)) / 2e-5
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd))
