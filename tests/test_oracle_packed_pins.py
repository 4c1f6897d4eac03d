"""Pins for the oracle's packed form (rank-local CSBP launches, DFlash2-style blocks) and for the
host-side CSBP partition: per-row brute force, finite differences, the rank-sum identities of
Algorithm 2 / Eq. dflash2-gradient-decomposition, and the work-balance formulas of appendix B."""
import math

import numpy as np
import pytest

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import schedule


def _rand(rng, *shape):
    return rng.standard_normal(shape) * 0.7


def _brute_row(q, keys, vals, scale):
    """softmax attention of one query over an explicit key list, written with Python loops."""
    if len(keys) == 0:
        return np.zeros_like(q), -math.inf
    s = [scale * sum(q[t] * k[t] for t in range(len(q))) for k in keys]
    m = max(s)
    w = [math.exp(x - m) for x in s]
    z = sum(w)
    o = np.zeros_like(q)
    for wi, v in zip(w, vals):
        o += (wi / z) * v
    return o, m + math.log(z)


def test_dflash2_blocks_match_per_row_brute_force():
    """Eq. dflash2-block-attention: block b sees its own M keys and the clean keys at positions < a_b."""
    rng = np.random.default_rng(5)
    B, Lk, H, Hkv, d, M = 1, 23, 2, 1, 4, 3
    anchors = [0, 4, 4, 11, 23]                     # includes an empty prefix, a repeat, the full prefix
    nb = len(anchors)
    kc, vc = _rand(rng, B, Lk, Hkv, d), _rand(rng, B, Lk, Hkv, d)
    qn, kn, vn = _rand(rng, B, nb * M, H, d), _rand(rng, B, nb * M, Hkv, d), _rand(rng, B, nb * M, Hkv, d)
    out = orc.attn_packed(None, kc, vc, qn, kn, vn, M, block_prefix=anchors)
    assert "o_clean" not in out
    scale = 1.0 / math.sqrt(d)
    for h in range(H):
        for b, a_b in enumerate(anchors):
            keys = [kn[0, b * M + t, 0] for t in range(M)] + [kc[0, j, 0] for j in range(a_b)]
            vals = [vn[0, b * M + t, 0] for t in range(M)] + [vc[0, j, 0] for j in range(a_b)]
            for t in range(M):
                o, z = _brute_row(qn[0, b * M + t, h], keys, vals, scale)
                assert np.allclose(out["o_noisy"][0, b * M + t, h], o, atol=1e-12)
                assert abs(out["lse_noisy"][0, h, b * M + t] - z) < 1e-12


def test_clean_segment_matches_per_row_brute_force():
    """A run of clean queries at positions pos0.. sees clean keys 0..position (Algorithm 1, clean part)."""
    rng = np.random.default_rng(6)
    Lk, d, M, pos0, Lq = 20, 4, 4, 8, 7
    kc, vc = _rand(rng, 1, Lk, 1, d), _rand(rng, 1, Lk, 1, d)
    kn, vn = _rand(rng, 1, M, 1, d), _rand(rng, 1, M, 1, d)
    qc = _rand(rng, 1, Lq, 1, d)
    out = orc.attn_packed(qc, kc, vc, None, kn, vn, M, clean_q_pos0=pos0)
    for i in range(Lq):
        keys = [kc[0, j, 0] for j in range(pos0 + i + 1)]
        vals = [vc[0, j, 0] for j in range(pos0 + i + 1)]
        o, z = _brute_row(qc[0, i, 0], keys, vals, 0.5)
        assert np.allclose(out["o_clean"][0, i, 0], o, atol=1e-12)
        assert abs(out["lse_clean"][0, 0, i] - z) < 1e-12


def test_packed_window_uses_token_positions():
    """Window W: packed row i of a block with prefix a stands at position a + i % M; it sees clean key j
    only if j < a and (a + i % M) - j < W."""
    M, Lk = 4, 32
    prefix = [8, 20]
    vis = orc.visible_rows_packed(orc.NOISY, np.arange(8), Lk, M, 2, prefix, window=6)
    for i in range(8):
        a = prefix[i // M]
        pos = a + i % M
        want = [j for j in range(Lk) if j < a and pos - j < 6]
        assert list(np.nonzero(vis[i, :Lk])[0]) == want
        assert list(np.nonzero(vis[i, Lk:])[0]) == list(range((i // M) * M, (i // M) * M + M))


def test_packed_gradients_match_finite_differences():
    rng = np.random.default_rng(7)
    B, Lk, H, Hkv, d, M = 1, 12, 2, 1, 3, 2
    prefix = [1, 5, 12]
    nb = len(prefix)
    t = {"kc": _rand(rng, B, Lk, Hkv, d), "vc": _rand(rng, B, Lk, Hkv, d),
         "qc": _rand(rng, B, 5, H, d), "qn": _rand(rng, B, nb * M, H, d),
         "kn": _rand(rng, B, nb * M, Hkv, d), "vn": _rand(rng, B, nb * M, Hkv, d)}
    doc, don = _rand(rng, B, 5, H, d), _rand(rng, B, nb * M, H, d)

    def loss(x):
        o = orc.attn_packed(x["qc"], x["kc"], x["vc"], x["qn"], x["kn"], x["vn"], M, block_prefix=prefix, clean_q_pos0=4)
        return float((o["o_clean"] * doc).sum() + (o["o_noisy"] * don).sum())

    g = orc.attn_packed(t["qc"], t["kc"], t["vc"], t["qn"], t["kn"], t["vn"], M, do_clean=doc, do_noisy=don,
                        block_prefix=prefix, clean_q_pos0=4)
    names = {"qc": "dq_clean", "kc": "dk_clean", "vc": "dv_clean", "qn": "dq_noisy", "kn": "dk_noisy", "vn": "dv_noisy"}
    eps = 1e-6
    for key, gname in names.items():
        flat = t[key].reshape(-1)
        for idx in rng.choice(flat.size, size=6, replace=False):
            old = flat[idx]
            flat[idx] = old + eps
            up = loss(t)
            flat[idx] = old - eps
            dn = loss(t)
            flat[idx] = old
            assert abs((up - dn) / (2 * eps) - g[gname].reshape(-1)[idx]) < 1e-6, (key, idx)


@pytest.mark.parametrize("L,M,P", [(48, 4, 2), (64, 8, 4), (42, 6, 2), (40, 8, 2)])
def test_rank_local_launches_add_up_to_the_unsharded_layer(L, M, P):
    """Algorithm 1: each rank's outputs are the unsharded outputs of its rows.  Algorithm 2: dQ and the
    corrupted K/V gradients stay local, the clean K/V gradient is the sum of the ranks' contributions."""
    rng = np.random.default_rng(L + M + P)
    B, H, Hkv, d = 1, 2, 1, 4
    qc, qn = _rand(rng, B, L, H, d), _rand(rng, B, L, H, d)
    kc, vc, kn, vn = (_rand(rng, B, L, Hkv, d) for _ in range(4))
    doc, don = _rand(rng, B, L, H, d), _rand(rng, B, L, H, d)
    full_o = orc.attn_forward(qc, kc, vc, qn, kn, vn, M)
    full_g = orc.attn_backward(qc, kc, vc, qn, kn, vn, doc, don, M)
    if L % (2 * P) == 0:
        clean_ranges = schedule.zigzag_chunks(L, P)
    else:                                   # zigzag needs 2P | L; any contiguous cut shows the same identity
        cut = (L // P // M) * M
        clean_ranges = [[(r * cut, (r + 1) * cut if r < P - 1 else L)] for r in range(P)]
    blocks = schedule.dual_end_blocks(L // M, P, M)
    assert sorted(b for bl in blocks for b in bl) == list(range(L // M))
    dk_sum, dv_sum = np.zeros_like(kc), np.zeros_like(vc)
    for r in range(P):
        rows_n = np.concatenate([np.arange(b * M, (b + 1) * M) for b in blocks[r]])
        prefix = [b * M for b in blocks[r]]
        res = orc.attn_packed(None, kc, vc, qn[:, rows_n], kn[:, rows_n], vn[:, rows_n], M,
                              do_noisy=don[:, rows_n], block_prefix=prefix)
        assert np.allclose(res["o_noisy"], full_o[2][:, rows_n], atol=1e-12)
        assert np.allclose(res["lse_noisy"], full_o[3][:, :, rows_n], atol=1e-12)
        assert np.allclose(res["dq_noisy"], full_g[3][:, rows_n], atol=1e-12)
        assert np.allclose(res["dk_noisy"], full_g[4][:, rows_n], atol=1e-12)
        assert np.allclose(res["dv_noisy"], full_g[5][:, rows_n], atol=1e-12)
        dk_sum += res["dk_clean"]
        dv_sum += res["dv_clean"]
        for (p0, p1) in clean_ranges[r]:
            res = orc.attn_packed(qc[:, p0:p1], kc, vc, None, kn[:, :M], vn[:, :M], M, do_clean=doc[:, p0:p1],
                                  clean_q_pos0=p0)
            assert np.allclose(res["o_clean"], full_o[0][:, p0:p1], atol=1e-12)
            assert np.allclose(res["lse_clean"], full_o[1][:, :, p0:p1], atol=1e-12)
            assert np.allclose(res["dq_clean"], full_g[0][:, p0:p1], atol=1e-12)
            dk_sum += res["dk_clean"]
            dv_sum += res["dv_clean"]
    assert np.allclose(dk_sum, full_g[1], atol=1e-11)
    assert np.allclose(dv_sum, full_g[2], atol=1e-11)


@pytest.mark.parametrize("L,M,P", [(64, 4, 2), (96, 4, 4), (128, 8, 2)])
def test_work_balance_formulas(L, M, P):
    """Eq. aligned-rank-work: with 2P | B every rank gets B(B+1)M^2/(2P) corrupted-query pairs and
    L(L+1)/(2P) clean pairs, counted here from the explicit packed masks of the rank's launches."""
    B = L // M
    assert B % (2 * P) == 0
    plans = schedule.csbp_plan(L, M, P)
    for plan in plans:
        nb = len(plan.blocks)
        vis = orc.visible_rows_packed(orc.NOISY, np.arange(nb * M), L, M, nb, plan.block_prefix)
        assert int(vis.sum()) == B * (B + 1) * M * M // (2 * P)
        clean = 0
        for (p0, p1) in plan.clean_ranges:
            clean += int(orc.visible_rows_packed(orc.CLEAN, np.arange(p1 - p0), L, M, 1, clean_q_pos0=p0).sum())
        assert clean == L * (L + 1) // (2 * P)
    # pair sums of Eq. aligned-pair-work, 0-indexed block b paired with B-1-b
    for b in range(B // 2):
        assert schedule.block_work(b, M) + schedule.block_work(B - 1 - b, M) == (B + 1) * M * M


def test_partition_covers_everything_once_and_handles_odd_counts():
    for B, P in [(8, 2), (7, 2), (9, 4), (5, 8), (1, 3)]:
        owned = schedule.dual_end_blocks(B, P, 4)
        flat = sorted(b for x in owned for b in x)
        assert flat == list(range(B))
        loads = [sum(schedule.block_work(b, 4) for b in x) for x in owned]
        pair = (B + 1) * 16
        assert max(loads) - min(loads) <= pair          # never worse than one pair of imbalance
    chunks = schedule.zigzag_chunks(48, 3)
    seen = sorted(p for c in chunks for (a, b) in c for p in range(a, b))
    assert seen == list(range(48))
    with pytest.raises(ValueError):
        schedule.zigzag_chunks(50, 3)


@pytest.mark.parametrize("mode,window,row_chunk", [(0, 0, 3), (1, 0, 2), (0, 5, 3), (0, 0, 64)])
def test_sampled_rows_packed_equal_full_packed_oracle(mode, window, row_chunk):
    """`attn_rows_packed` (the checker of the full-size packed parity tests) against `attn_packed`, which the
    brute-force and finite-difference pins above fix: same rows -> same O, LSE, dQ; and, because dK/dV are
    linear in dO, its per-row K/V contributions equal the full backward with dO zeroed outside the sample.
    The prefix table holds an empty prefix, a repeat, non-multiples of M and the full prefix (Eq.
    dflash2-block-attention); the clean run starts at an offset; the sample is larger than a row chunk."""
    rng = np.random.default_rng(41 + mode + window)
    B, Lk, H, Hkv, d, M = 1, 40, 2, 1, 4, 4
    prefix = [0, 6, 6, 17, 28, 40] if window == 0 else [0, 4, 9, 17, 28, 36]   # with a window blocks may not overlap
    nb = len(prefix)
    pos0, Lq = 9, 22
    kc, vc = _rand(rng, B, Lk, Hkv, d), _rand(rng, B, Lk, Hkv, d)
    qc, qn = _rand(rng, B, Lq, H, d), _rand(rng, B, nb * M, H, d)
    kn, vn = _rand(rng, B, nb * M, Hkv, d), _rand(rng, B, nb * M, Hkv, d)
    doc, don = _rand(rng, B, Lq, H, d), _rand(rng, B, nb * M, H, d)
    rows_c = np.array([0, 1, 3, 4, 10, 11, 20, 21])
    rows_n = np.array([0, 3, 4, 7, 9, 12, 15, 16, 22, 23])
    kw = dict(block_prefix=prefix, clean_q_pos0=pos0, clean_mask_mode=mode, window=window)
    full = orc.attn_packed(qc, kc, vc, qn, kn, vn, M, **kw)
    for h in range(H):
        doc_s, don_s = np.zeros_like(doc), np.zeros_like(don)
        doc_s[0, rows_c, h] = doc[0, rows_c, h]
        don_s[0, rows_n, h] = don[0, rows_n, h]
        g = orc.attn_packed(qc, kc, vc, qn, kn, vn, M, do_clean=doc_s, do_noisy=don_s, **kw)
        rc = orc.attn_rows_packed(orc.CLEAN, rows_c, qc[0, rows_c, h], kc[0, :, 0], vc[0, :, 0], kn[0, :, 0],
                                  vn[0, :, 0], M, do_rows=doc[0, rows_c, h], row_chunk=row_chunk, **kw)
        rn = orc.attn_rows_packed(orc.NOISY, rows_n, qn[0, rows_n, h], kc[0, :, 0], vc[0, :, 0], kn[0, :, 0],
                                  vn[0, :, 0], M, do_rows=don[0, rows_n, h], row_chunk=row_chunk, **kw)
        assert np.allclose(rc["o"], full["o_clean"][0, rows_c, h], atol=1e-13)
        assert np.allclose(rc["lse"], full["lse_clean"][0, h, rows_c], atol=1e-13)
        assert np.allclose(rn["o"], full["o_noisy"][0, rows_n, h], atol=1e-13)
        assert np.allclose(rn["lse"], full["lse_noisy"][0, h, rows_n], atol=1e-13)
        assert np.allclose(rc["dq"], g["dq_clean"][0, rows_c, h], atol=1e-13)
        assert np.allclose(rn["dq"], g["dq_noisy"][0, rows_n, h], atol=1e-13)
        assert np.allclose(rc["dk_clean"] + rn["dk_clean"], g["dk_clean"][0, :, 0], atol=1e-13)
        assert np.allclose(rc["dv_clean"] + rn["dv_clean"], g["dv_clean"][0, :, 0], atol=1e-13)
        assert np.allclose(rn["dk_noisy"], g["dk_noisy"][0, :, 0], atol=1e-13)
        assert np.allclose(rn["dv_noisy"], g["dv_noisy"][0, :, 0], atol=1e-13)
        assert np.abs(rc["dk_noisy"]).max() == 0 and np.abs(rc["dv_noisy"]).max() == 0
        # unsorted, repeated-free sample order must not matter
        perm = rng.permutation(len(rows_n))
        rp = orc.attn_rows_packed(orc.NOISY, rows_n[perm], qn[0, rows_n[perm], h], kc[0, :, 0], vc[0, :, 0],
                                  kn[0, :, 0], vn[0, :, 0], M, do_rows=don[0, rows_n[perm], h], row_chunk=row_chunk, **kw)
        assert np.allclose(rp["o"], rn["o"][perm], atol=1e-13) and np.allclose(rp["dq"], rn["dq"][perm], atol=1e-13)


def test_sampled_rows_packed_reduce_to_plain_sampled_rows():
    """With the table b*M, no offset and every block present, the packed sampled-row oracle is the plain one."""
    rng = np.random.default_rng(77)
    L, d, M = 24, 4, 4
    kc, vc, kn, vn = (_rand(rng, L, d) for _ in range(4))
    rows = np.array([0, 3, 4, 9, 23])
    q, do = _rand(rng, len(rows), d), _rand(rng, len(rows), d)
    for stream in (orc.CLEAN, orc.NOISY):
        a = orc.attn_rows(stream, rows, q, kc, vc, kn, vn, M, do_rows=do)
        b = orc.attn_rows_packed(stream, rows, q, kc, vc, kn, vn, M, do_rows=do)
        for key in a:
            assert np.allclose(a[key], b[key], atol=1e-14), key


def test_workload_pair_counts_equal_explicit_mask_counts():
    """The FLOP denominators of the benchmark (`Workload.pairs_per_head`: closed forms of appendix B, the
    windowed and the packed variants) against pairs counted from the oracle's explicit masks."""
    from paper_2609_19242_b200 import synth
    for L, M, W in [(64, 8, 0), (96, 4, 0), (64, 8, 20), (64, 8, 8), (48, 16, 5), (60, 6, 7), (64, 4, 1000), (32, 1, 3)]:
        w = synth.Workload("t", 1, 2, 1, 8, L, M, window=W)
        assert w.pairs_per_head() == orc.visible_pair_counts(L, M, window=W), (L, M, W)
    for L, M, nb, seed in [(64, 4, 9, 0), (80, 8, 5, 3), (33, 3, 12, 5)]:
        w = synth.Workload("p", 1, 2, 1, 8, L, M, n_blocks=nb, seed=seed)
        vis = orc.visible_rows_packed(orc.NOISY, np.arange(nb * M), L, M, nb, w.anchors())
        assert w.pairs_per_head() == (0, int(vis.sum()))
    # appendix B totals (Eq. aligned-rank-work with P = 1) for the headline shapes, without building their masks
    for name in ("32k", "csbp128k", "256k"):
        w = synth.WORKLOADS[name]
        assert w.pairs_per_head() == (w.L * (w.L + 1) // 2, w.L * (w.L + w.block_size) // 2)
