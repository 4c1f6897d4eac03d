"""GPU-vs-oracle parity of the packed form: one rank's launches of the CSBP schedule (Algorithms 1, 2)
and DFlash2-style blocks (appendix E), through the C ABI, both kernel families."""
import numpy as np
import pytest
import torch

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import binding, schedule, synth

import parity_util as pu

pytestmark = pytest.mark.gpu

IMPLS = [binding.IMPL_PORTABLE, binding.IMPL_AUTO]


def _draw(seed, batch, Lk, Lq, Ln, H, Hkv, d):
    """Seeded bf16 inputs of a packed call (host tensors; None where a stream has no rows)."""
    g = torch.Generator().manual_seed(seed)
    mk = lambda rows, heads, sigma: (torch.randn(batch, rows, heads, d, generator=g) * sigma).to(torch.bfloat16)
    t = {"k_clean": mk(Lk, Hkv, 0.5), "v_clean": mk(Lk, Hkv, 0.5)}
    t["q_clean"] = mk(Lq, H, 0.5) if Lq else None
    t["do_clean"] = mk(Lq, H, 1.0) if Lq else None
    for n, heads, sigma in (("q_noisy", H, 0.5), ("k_noisy", Hkv, 0.5), ("v_noisy", Hkv, 0.5), ("do_noisy", H, 1.0)):
        t[n] = mk(Ln, heads, sigma) if Ln else None
    return t


def _cuda(t):
    return {k: (None if v is None else v.cuda()) for k, v in t.items()}


def _f64(t):
    return {k: (None if v is None else synth.to_f64(v)) for k, v in t.items()}


def _run_and_check(t, M, impl, prefix=None, pos0=0, window=0, mode=0, single_pass=False):
    g, x = _cuda(t), _f64(t)
    pfx_dev = None if prefix is None else torch.tensor(prefix, dtype=torch.int32, device="cuda")
    kw = dict(block_prefix=pfx_dev, clean_q_pos0=pos0, impl=impl, window=window, clean_mask_mode=mode)
    out = binding.bdlm_attn_fwd_packed(g["q_clean"], g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"],
                                       g["v_noisy"], M, **kw)
    grads = binding.bdlm_attn_bwd_packed(g["q_clean"], g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"],
                                         g["v_noisy"], out[0], out[1], out[2], out[3], g["do_clean"],
                                         g["do_noisy"], M, single_pass=single_pass, **kw)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    kn = x["k_noisy"] if x["k_noisy"] is not None else np.zeros((x["k_clean"].shape[0], M) + x["k_clean"].shape[2:])
    vn = x["v_noisy"] if x["v_noisy"] is not None else np.zeros_like(kn)
    ref = orc.attn_packed(x["q_clean"], x["k_clean"], x["v_clean"], x["q_noisy"], kn, vn, M,
                          do_clean=x["do_clean"], do_noisy=x["do_noisy"], block_prefix=prefix, clean_q_pos0=pos0,
                          window=window, clean_mask_mode=mode)
    for name, got in zip(["o_clean", "lse_clean", "o_noisy", "lse_noisy"], out):
        if got is None:
            assert name not in ref
            continue
        gotn, want = synth.to_f64(got), ref[name]
        assert not np.isnan(gotn).any(), name
        assert (np.isneginf(gotn) == np.isneginf(want)).all(), name
        fin = np.isfinite(want)
        assert np.abs(gotn[fin] - want[fin]).max() <= (pu.TOL_LSE if "lse" in name else pu.TOL_O), name
    names = ["dq_clean", "dk_clean", "dv_clean", "dq_noisy", "dk_noisy", "dv_noisy"]
    for name, got in zip(names, grads):
        if got is None:
            continue
        gotn = synth.to_f64(got)
        assert np.isfinite(gotn).all(), name
        want = ref[name]
        if np.abs(want).max() == 0:
            assert np.abs(gotn).max() == 0, name
        else:
            assert pu.rel_l2(gotn, want) <= pu.TOL_GRAD, (name, pu.rel_l2(gotn, want))
    return out, grads


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("case", [
    dict(Lk=512, M=16, anchors="random", nb=16, H=4, Hkv=2),
    dict(Lk=384, M=32, anchors=[0, 0, 5, 128, 129, 300, 384, 384], nb=8, H=2, Hkv=1),
    dict(Lk=256, M=128, anchors=[17, 256], nb=2, H=2, Hkv=2),
    dict(Lk=640, M=8, anchors="random", nb=48, H=2, Hkv=1),
], ids=["m16", "m32_edges", "m128", "m8"])
def test_dflash2_blocks_match_oracle(case, impl):
    """Sampled blocks with arbitrary anchors, no clean-query stream (Eq. dflash2-block-attention)."""
    M, nb, Lk = case["M"], case["nb"], case["Lk"]
    if case["anchors"] == "random":
        rng = np.random.default_rng(nb + M)
        anchors = sorted(int(v) for v in rng.integers(0, Lk + 1, size=nb))
    else:
        anchors = case["anchors"]
    t = _draw(11, 1, Lk, 0, nb * M, case["H"], case["Hkv"], 128)
    _run_and_check(t, M, impl, prefix=anchors)


@pytest.mark.parametrize("impl", IMPLS)
def test_clean_segment_and_both_streams(impl):
    """A run of clean queries at an offset; then both streams in one call with a prefix table."""
    t = _draw(12, 2, 512, 128, 0, 4, 2, 128)
    _run_and_check(t, 32, impl, pos0=256)
    t = _draw(13, 1, 512, 256, 256, 2, 1, 128)
    _run_and_check(t, 32, impl, prefix=[b * 32 for b in (0, 3, 4, 9, 10, 12, 14, 15)], pos0=128)
    _run_and_check(t, 32, impl, prefix=[b * 32 for b in (0, 3, 4, 9, 10, 12, 14, 15)], pos0=128, mode=1)


@pytest.mark.parametrize("impl", IMPLS)
def test_packed_with_sliding_window(impl):
    t = _draw(14, 1, 768, 128, 256, 2, 1, 128)
    prefix = [b * 64 for b in (1, 5, 8, 11)]
    _run_and_check(t, 64, impl, prefix=prefix, pos0=640, window=200)
    _run_and_check(t, 64, impl, prefix=prefix, pos0=0, window=33)


def test_fused_backward_on_packed_forms():
    """The fused one-kernel backward on the packed forms: sampled blocks alone, a clean run at an offset, both
    streams with a prefix table (both mask modes), a sliding window."""
    rng = np.random.default_rng(5)
    t = _draw(21, 1, 512, 0, 16 * 16, 4, 2, 128)
    _run_and_check(t, 16, binding.IMPL_AUTO, prefix=sorted(int(v) for v in rng.integers(0, 513, size=16)), single_pass=True)
    t = _draw(22, 2, 512, 128, 0, 4, 2, 128)
    _run_and_check(t, 32, binding.IMPL_AUTO, pos0=256, single_pass=True)
    t = _draw(23, 1, 512, 256, 256, 2, 1, 128)
    for mode in (0, 1):
        _run_and_check(t, 32, binding.IMPL_AUTO, prefix=[b * 32 for b in (0, 3, 4, 9, 10, 12, 14, 15)], pos0=128, mode=mode,
                       single_pass=True)
    t = _draw(24, 1, 768, 128, 256, 2, 1, 128)
    _run_and_check(t, 64, binding.IMPL_AUTO, prefix=[b * 64 for b in (1, 5, 8, 11)], pos0=640, window=200, single_pass=True)


def test_packed_forms_with_odd_group_sizes():
    """MHA and G = 3 on the packed forms: a single clean query tile (the forward's tile pair is half empty), three
    tiles of sampled blocks, both streams."""
    t = _draw(31, 1, 512, 128, 384, 3, 3, 128)
    _run_and_check(t, 32, binding.IMPL_TCGEN05, prefix=[b * 32 for b in (0, 1, 2, 5, 6, 7, 9, 11, 12, 13, 14, 15)], pos0=256)
    t = _draw(32, 1, 384, 0, 3 * 128, 3, 1, 128)
    _run_and_check(t, 128, binding.IMPL_TCGEN05, prefix=[0, 130, 384], single_pass=True)
    t = _draw(33, 2, 640, 384, 128, 2, 2, 128)
    _run_and_check(t, 64, binding.IMPL_TCGEN05, prefix=[64, 500], pos0=128, window=150, single_pass=True)


def test_portable_kernels_take_ragged_packed_shapes():
    """d = 64, a clean length that is no multiple of anything, a short clean run."""
    t = _draw(15, 1, 203, 37, 5 * 24, 2, 2, 64)
    _run_and_check(t, 24, binding.IMPL_PORTABLE, prefix=[0, 24, 100, 203, 203], pos0=150)


def _close(a, b, atol):
    assert (a.double() - b.double()).abs().max().item() <= atol


def _rel(a, b, tol=5e-3):
    assert pu.rel_l2(synth.to_f64(a), synth.to_f64(b)) <= tol


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("P", [2, 4])
def test_rank_local_launches_add_up(P, impl):
    """CSBP schedule emulation: every rank runs its clean position ranges and its packed blocks against the
    complete clean K/V; outputs and local gradients equal the unsharded layer's rows, and the ranks' clean
    K/V gradient contributions add up to the unsharded clean K/V gradient (Algorithm 2)."""
    w = synth.Workload("csbp_local", 1, 4, 2, 128, 2048, 64)
    inp = synth.make_inputs(w, "cpu")
    g = pu.to_cuda(inp)
    M, L = w.block_size, w.L
    full_o = pu.gpu_fwd(g, M, impl=impl)
    full_g = pu.gpu_bwd(g, full_o, M, impl=impl)
    torch.cuda.synchronize()
    dk_sum = torch.zeros_like(g["k_clean"], dtype=torch.float64)
    dv_sum = torch.zeros_like(g["v_clean"], dtype=torch.float64)
    for plan in schedule.csbp_plan(L, M, P):
        rows = torch.cat([torch.arange(b * M, (b + 1) * M) for b in plan.blocks]).cuda()
        pfx = torch.tensor(plan.block_prefix, dtype=torch.int32, device="cuda")
        sub = {n: g[n][:, rows].contiguous() for n in ("q_noisy", "k_noisy", "v_noisy", "do_noisy")}
        o = binding.bdlm_attn_fwd_packed(None, g["k_clean"], g["v_clean"], sub["q_noisy"], sub["k_noisy"],
                                         sub["v_noisy"], M, block_prefix=pfx, impl=impl)
        gr = binding.bdlm_attn_bwd_packed(None, g["k_clean"], g["v_clean"], sub["q_noisy"], sub["k_noisy"],
                                          sub["v_noisy"], None, None, o[2], o[3], None, sub["do_noisy"], M,
                                          block_prefix=pfx, impl=impl)
        # the packed tiles cut a row's keys at other places than the unsharded launch, so results agree to
        # rounding, not bitwise
        _close(o[2], full_o[2][:, rows], 2e-2); _close(o[3], full_o[3][:, :, rows], 1e-4)
        _rel(gr[3], full_g[3][:, rows]); _rel(gr[4], full_g[4][:, rows]); _rel(gr[5], full_g[5][:, rows])
        dk_sum += gr[1].double()
        dv_sum += gr[2].double()
        for (p0, p1) in plan.clean_ranges:
            qc, doc = g["q_clean"][:, p0:p1].contiguous(), g["do_clean"][:, p0:p1].contiguous()
            o = binding.bdlm_attn_fwd_packed(qc, g["k_clean"], g["v_clean"], None, None, None, M,
                                             clean_q_pos0=p0, impl=impl)
            gr = binding.bdlm_attn_bwd_packed(qc, g["k_clean"], g["v_clean"], None, None, None, o[0], o[1], None,
                                              None, doc, None, M, clean_q_pos0=p0, impl=impl)
            _close(o[0], full_o[0][:, p0:p1], 2e-2); _close(o[1], full_o[1][:, :, p0:p1], 1e-4)
            _rel(gr[0], full_g[0][:, p0:p1])
            dk_sum += gr[1].double()
            dv_sum += gr[2].double()
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    # each contribution is rounded to bf16 once, so the sum of 3P contributions differs from the single
    # rounding of the unsharded result by rounding noise only
    assert pu.rel_l2(dk_sum.cpu().numpy(), synth.to_f64(full_g[1])) <= 1e-2
    assert pu.rel_l2(dv_sum.cpu().numpy(), synth.to_f64(full_g[2])) <= 1e-2
    x = pu.f64(inp)
    ref = orc.attn_backward(*[x[n] for n in pu.NAMES6], x["do_clean"], x["do_noisy"], M)
    assert pu.rel_l2(dk_sum.cpu().numpy(), ref[1]) <= pu.TOL_GRAD
    assert pu.rel_l2(dv_sum.cpu().numpy(), ref[2]) <= pu.TOL_GRAD


def test_binding_rejects_bad_prefix_tables():
    t = _cuda(_draw(16, 1, 256, 0, 128, 2, 1, 128))
    args = (None, t["k_clean"], t["v_clean"], t["q_noisy"], t["k_noisy"], t["v_noisy"], 32)
    mk = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, block_prefix=mk([0, 64, 32, 128]))        # not sorted
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, block_prefix=mk([0, 64, 300, 400]))       # beyond the clean length
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, block_prefix=mk([0, 16, 64, 128]), window=64)   # overlapping blocks
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, block_prefix=mk([0, 64, 128]))            # wrong length


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("P", [2, 4])
def test_clean_kv_in_gathered_order(P, impl):
    """The all-gathered clean K/V used without a reordering copy: ranks' zigzag shards one after the other in
    memory, every key addressed by its original position.  Same tiles, same arithmetic: results are bitwise
    those of the position-ordered call (dK/dV come back in the gathered order)."""
    w = synth.Workload("gathered", 1, 4, 2, 128, 2048, 64)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    M, L = w.block_size, w.L
    Lc = L // (2 * P)
    order = [c for r in range(P) for c in (r, 2 * P - 1 - r)]           # memory chunk m holds position chunk order[m]
    positions = [c * Lc for c in order]
    gather = torch.cat([torch.arange(c * Lc, (c + 1) * Lc) for c in order]).cuda()
    kg, vg = g["k_clean"][:, gather].contiguous(), g["v_clean"][:, gather].contiguous()
    plan = schedule.csbp_plan(L, M, P)[P - 1]
    rows = torch.cat([torch.arange(b * M, (b + 1) * M) for b in plan.blocks]).cuda()
    pfx = torch.tensor(plan.block_prefix, dtype=torch.int32, device="cuda")
    sub = {n: g[n][:, rows].contiguous() for n in ("q_noisy", "k_noisy", "v_noisy", "do_noisy")}
    p0, p1 = plan.clean_ranges[1]
    qc, doc = g["q_clean"][:, p0:p1].contiguous(), g["do_clean"][:, p0:p1].contiguous()
    res = {}
    for name, (kc, vc, kw) in {"by_position": (g["k_clean"], g["v_clean"], {}),
                               "gathered": (kg, vg, {"kv_chunks": (Lc, positions)})}.items():
        o = binding.bdlm_attn_fwd_packed(qc, kc, vc, sub["q_noisy"], sub["k_noisy"], sub["v_noisy"], M,
                                         block_prefix=pfx, clean_q_pos0=p0, impl=impl, **kw)
        gr = binding.bdlm_attn_bwd_packed(qc, kc, vc, sub["q_noisy"], sub["k_noisy"], sub["v_noisy"], o[0], o[1], o[2],
                                          o[3], doc, sub["do_noisy"], M, block_prefix=pfx, clean_q_pos0=p0, impl=impl,
                                          single_pass=False, **kw)   # two-pass: dQ is compared bitwise below
        res[name] = (o, gr)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    (o_a, g_a), (o_b, g_b) = res["by_position"], res["gathered"]
    for x, y in zip(o_a, o_b):
        assert torch.equal(x, y)
    for i in (0, 3, 4, 5):
        assert torch.equal(g_a[i], g_b[i])
    assert torch.equal(g_a[1][:, gather], g_b[1]) and torch.equal(g_a[2][:, gather], g_b[2])
    # a shard of the gathered keys by position range, forward only
    o_s = binding.bdlm_attn_fwd_packed(qc, kg, vg, None, None, None, M, clean_q_pos0=p0, impl=impl,
                                       kv_range=(256, 1024), include_noisy_diag=False, kv_chunks=(Lc, positions))
    o_r = binding.bdlm_attn_fwd_packed(qc, g["k_clean"], g["v_clean"], None, None, None, M, clean_q_pos0=p0, impl=impl,
                                       kv_range=(256, 1024), include_noisy_diag=False)
    assert torch.equal(o_s[0], o_r[0]) and torch.equal(o_s[1], o_r[1])


def test_gathered_order_is_validated():
    t = _cuda(_draw(17, 1, 512, 128, 0, 2, 1, 128))
    args = (t["q_clean"], t["k_clean"], t["v_clean"], None, None, None, 32)
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, kv_chunks=(128, [0, 128, 128, 384]))     # not a permutation
    with pytest.raises(ValueError):
        binding.bdlm_attn_fwd_packed(*args, kv_chunks=(100, [0, 100, 200, 300, 400]))   # does not divide L
    with pytest.raises(binding.BdlmError):
        binding.bdlm_attn_fwd_packed(*args, kv_chunks=(64, [c * 64 for c in range(8)]))  # chunks must be multiples of 128
    with pytest.raises(binding.BdlmError):
        binding.bdlm_attn_fwd_packed(*args, kv_chunks=(128, [0, 128, 256, 384]), window=64)  # no window with chunks


@pytest.mark.parametrize("single_pass", [False, True])
def test_clean_key_tiles_that_no_query_sees(single_pass):
    """Sampled blocks with low anchors over a long clean sequence: most clean key tiles are seen by no query of the
    call (their CTAs write zeros and must leave without a copy in flight), with seen tiles before and between
    them.  dK/dV of the clean keys: zero beyond the last anchor, equal to the oracle, and -- for the keys that are
    seen -- bitwise those of the same call on a clean sequence cut off after the last seen tile."""
    M, L, H, Hkv = 32, 2048, 4, 2
    prefix = [0, 40, 130, 130, 600, 610, 900, 1000]              # last seen clean key: 999 -> key tiles 8..15 unseen
    nb = len(prefix)
    t = _draw(23, 1, L, 0, nb * M, H, Hkv, 128)
    g = _cuda(t)
    pfx = torch.tensor(prefix, dtype=torch.int32, device="cuda")

    def run(Lk):
        kc, vc = g["k_clean"][:, :Lk].contiguous(), g["v_clean"][:, :Lk].contiguous()
        o = binding.bdlm_attn_fwd_packed(None, kc, vc, g["q_noisy"], g["k_noisy"], g["v_noisy"], M, block_prefix=pfx,
                                         impl=binding.IMPL_TCGEN05)
        gr = binding.bdlm_attn_bwd_packed(None, kc, vc, g["q_noisy"], g["k_noisy"], g["v_noisy"], None, None, o[2], o[3],
                                          None, g["do_noisy"], M, block_prefix=pfx, impl=binding.IMPL_TCGEN05,
                                          single_pass=single_pass)
        return o, gr

    for rep in range(3):   # repeated: a copy left in flight by a retired CTA would land in its successor's tiles
        o_full, g_full = run(L)
        o_cut, g_cut = run(1024)
        torch.cuda.synchronize()
        assert binding.bdlm_get_device_status() == 0
        assert torch.equal(o_full[2], o_cut[2]) and torch.equal(o_full[3], o_cut[3])
        for i in (1, 2):
            assert torch.equal(g_full[i][:, :1024], g_cut[i])
            assert float(g_full[i][:, 1000:].float().abs().max()) == 0.0
        for i in (4, 5):
            assert torch.equal(g_full[i], g_cut[i])
    x = {k: synth.to_f64(v) for k, v in t.items() if v is not None}
    ref = orc.attn_packed(None, x["k_clean"], x["v_clean"], x["q_noisy"], x["k_noisy"], x["v_noisy"], M,
                          do_noisy=x["do_noisy"], block_prefix=prefix)
    for i, n in ((1, "dk_clean"), (2, "dv_clean"), (3, "dq_noisy"), (4, "dk_noisy"), (5, "dv_noisy")):
        assert pu.rel_l2(synth.to_f64(g_full[i]), ref[n]) <= pu.TOL_GRAD, n


def test_packed_form_with_head_dimension_64_on_the_tensor_core_kernels():
    rng = np.random.default_rng(3)
    t = _draw(31, 1, 512, 256, 256, 4, 2, 64)
    _run_and_check(t, 32, binding.IMPL_TCGEN05, prefix=sorted(int(v) for v in rng.integers(0, 513, size=8)), pos0=128)
    _run_and_check(t, 32, binding.IMPL_TCGEN05, prefix=sorted(int(v) for v in rng.integers(0, 513, size=8)), pos0=128,
                   single_pass=True)
