"""GPU-vs-oracle parity, whole tensors, at sizes the full oracle finishes in seconds: several
tiles and ragged tails, the block-size extremes, both mask modes, GQA, K/V shards + merge."""
import numpy as np
import pytest
import torch

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import Workload, WORKLOADS

import parity_util as pu

pytestmark = pytest.mark.gpu

IMPLS = [binding.IMPL_PORTABLE, binding.IMPL_AUTO]

SMALL = [
    WORKLOADS["tiny"],
    Workload("d128_3tiles", 2, 4, 2, 128, 384, 32),
    Workload("ragged_tail", 1, 2, 1, 64, 200, 8),
    Workload("m1", 1, 2, 2, 64, 96, 1),
    Workload("m_eq_L", 1, 2, 1, 128, 128, 128),
    Workload("m256", 1, 4, 1, 128, 512, 256),
    Workload("m48_odd", 1, 2, 2, 128, 336, 48),
    Workload("gqa8", 1, 8, 1, 128, 256, 64, rope_theta=5e5),
    Workload("m128", 1, 2, 1, 128, 640, 128),
    Workload("m16_d128", 1, 2, 2, 128, 512, 16),
]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_forward_backward_match_oracle(w, impl):
    pu.check_full(w, impl)


WINDOWED = [
    Workload("w1", 1, 2, 1, 128, 256, 32, window=1),
    Workload("w7_m1", 1, 2, 2, 64, 160, 1, window=7),
    Workload("w_lt_block", 1, 2, 1, 128, 512, 64, window=40),
    Workload("w100_ragged", 1, 4, 2, 128, 456, 8, window=100),
    Workload("w128", 1, 2, 1, 128, 640, 32, window=128),
    Workload("w129", 1, 2, 1, 128, 640, 32, window=129),
    Workload("w300_m128", 2, 4, 2, 128, 768, 128, window=300),
    Workload("w_ge_L", 1, 2, 1, 64, 384, 16, window=1000),
]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("w", WINDOWED, ids=lambda w: w.name)
def test_sliding_window_matches_oracle(w, impl):
    """Sliding-window layers: clean keys limited to i - j < window, forward and backward."""
    pu.check_full(w, impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_sliding_window_mode_1_and_shards(impl):
    """The window composes with the whole-own-block clean mask and with a clean-key shard range."""
    pu.check_full(Workload("w_mode1", 1, 2, 1, 128, 384, 32, window=70), impl, mode=1)
    w = Workload("w_shard", 1, 2, 1, 128, 512, 32, window=150)
    inp = synth.make_inputs(w, "cpu", with_grad=False)
    g = pu.to_cuda(inp)
    x = pu.f64(inp)
    for a, b in [(0, 200), (200, 512), (300, 301)]:
        out = pu.gpu_fwd(g, w.block_size, kv_range=(a, b), include_noisy_diag=False, impl=impl, window=w.window)
        ref = orc.attn_forward(*[x[n] for n in pu.NAMES6], w.block_size, kv_begin=a, kv_end=b,
                               include_noisy_diag=False, window=w.window)
        for got, want in zip(out, ref):
            gotn = synth.to_f64(got)
            assert not np.isnan(gotn).any()
            assert (np.isneginf(gotn) == np.isneginf(want)).all()
            fin = np.isfinite(want)
            assert np.abs(gotn[fin] - want[fin]).max() <= pu.TOL_O


@pytest.mark.parametrize("impl", IMPLS)
def test_clean_mask_mode_1(impl):
    pu.check_full(Workload("mode1", 1, 2, 1, 128, 384, 32), impl, mode=1)
    pu.check_full(Workload("mode1_big_block", 1, 2, 1, 64, 512, 256), impl, mode=1)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("cuts", [[0, 128, 256, 384], [0, 40, 200, 384], [0, 0, 384]])
def test_shard_partials_and_merge(impl, cuts):
    """Clean-K/V shard partials plus the noisy-diagonal partial, merged on the GPU, equal the
    unsharded kernel and the oracle; each partial equals the oracle's partial."""
    w = Workload("shards", 2, 4, 2, 128, 384, 32)
    inp = synth.make_inputs(w, "cpu", with_grad=False)
    g = pu.to_cuda(inp)
    x = pu.f64(inp)
    M = w.block_size
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        out = pu.gpu_fwd(g, M, kv_range=(a, b), include_noisy_diag=False, impl=impl)
        ref = orc.attn_forward(*[x[n] for n in pu.NAMES6], M, kv_begin=a, kv_end=b, include_noisy_diag=False)
        for got, want in zip(out, ref):
            gotn = synth.to_f64(got)
            assert not np.isnan(gotn).any()
            assert (np.isneginf(gotn) == np.isneginf(want)).all()
            fin = np.isfinite(want)
            assert np.abs(gotn[fin] - want[fin]).max() <= pu.TOL_O if fin.any() else True
        parts.append(out)
    diag = binding.bdlm_attn_fwd(None, g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"], g["v_noisy"], M,
                                 kv_range=(0, 0), impl=impl)
    o_c, l_c = binding.bdlm_lse_merge([p[0] for p in parts], [p[1] for p in parts])
    o_n, l_n = binding.bdlm_lse_merge([p[2] for p in parts] + [diag[2]], [p[3] for p in parts] + [diag[3]])
    torch.cuda.synchronize()
    full_ref = orc.attn_forward(*[x[n] for n in pu.NAMES6], M)
    full_gpu = pu.gpu_fwd(g, M, impl=impl)
    for got, want, unsh, name in zip((o_c, l_c, o_n, l_n), full_ref, full_gpu, ["oc", "lc", "on", "ln"]):
        tol = pu.TOL_LSE if name[0] == "l" else pu.TOL_O
        assert np.abs(synth.to_f64(got) - want).max() <= tol, name
        assert np.abs(synth.to_f64(got) - synth.to_f64(unsh)).max() <= tol, name


def test_merge_kernel_matches_oracle_merge():
    """bdlm_lse_merge alone: bf16 and fp32 partials, empty (-inf) rows, all-empty rows."""
    rng = np.random.default_rng(5)
    B, L, H, d, n = 2, 300, 3, 64, 5
    for dtype in (torch.bfloat16, torch.float32):
        os_ = [torch.tensor(rng.normal(size=(B, L, H, d)), dtype=dtype) for _ in range(n)]
        ls = [torch.tensor(rng.normal(size=(B, H, L)) * 4, dtype=torch.float32) for _ in range(n)]
        ls[1][:, :, :50] = -float("inf")
        for l in ls:
            l[:, :, 100:110] = -float("inf")     # rows empty in every partial
        o, l = binding.bdlm_lse_merge([t.cuda() for t in os_], [t.cuda() for t in ls])
        torch.cuda.synchronize()
        ro, rl = orc.lse_merge([synth.to_f64(t) for t in os_], [synth.to_f64(t) for t in ls])
        got_l = synth.to_f64(l)
        assert (np.isneginf(got_l) == np.isneginf(rl)).all()
        fin = np.isfinite(rl)
        assert np.abs(got_l[fin] - rl[fin]).max() <= 1e-5
        assert np.abs(synth.to_f64(o) - ro).max() <= 2e-2   # bf16 output rounding of |O| up to ~4
        assert np.abs(synth.to_f64(o)[:, 100:110]).max() == 0


@pytest.mark.parametrize("impl", IMPLS)
def test_backward_is_bitwise_reproducible(impl):
    w = Workload("repro", 1, 4, 2, 128, 384, 32)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    out = pu.gpu_fwd(g, w.block_size, impl=impl)
    a = [t.clone() for t in pu.gpu_bwd(g, out, w.block_size, impl=impl)]
    b = pu.gpu_bwd(g, out, w.block_size, impl=impl)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_skipping_a_stream():
    w = Workload("skip", 1, 2, 1, 128, 256, 32)
    g = pu.to_cuda(synth.make_inputs(w, "cpu", with_grad=False))
    full = pu.gpu_fwd(g, w.block_size)
    only_n = binding.bdlm_attn_fwd(None, g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"], g["v_noisy"], w.block_size)
    only_c = binding.bdlm_attn_fwd(g["q_clean"], g["k_clean"], g["v_clean"], None, None, None, w.block_size)
    assert only_n[0] is None and torch.equal(only_n[2], full[2]) and torch.equal(only_n[3], full[3])
    assert only_c[2] is None and torch.equal(only_c[0], full[0]) and torch.equal(only_c[1], full[1])


@pytest.mark.parametrize("w", [Workload("sp_3tiles", 2, 4, 2, 128, 384, 32), Workload("sp_m256", 1, 4, 1, 128, 512, 256),
                               Workload("sp_m16", 1, 2, 2, 128, 512, 16),
                               Workload("sp_w200", 1, 2, 1, 128, 768, 32, window=200)], ids=lambda w: w.name)
def test_single_pass_backward_matches_oracle_and_two_pass(w):
    """The fused one-kernel backward (dQ through fp32 add-reductions): same tolerances against the oracle; dK
    and dV come from a fixed-order accumulation like those of the two-pass kernels."""
    inp = synth.make_inputs(w, "cpu")
    g = pu.to_cuda(inp)
    x = pu.f64(inp)
    M = w.block_size
    out = pu.gpu_fwd(g, M, window=w.window)
    two = [t.clone() for t in pu.gpu_bwd(g, out, M, window=w.window)]
    one = pu.gpu_bwd(g, out, M, single_pass=True, window=w.window)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    gref = orc.attn_backward(*[x[n] for n in pu.NAMES6], x["do_clean"], x["do_noisy"], M, window=w.window)
    for got, want in zip(one, gref):
        assert pu.rel_l2(synth.to_f64(got), want) <= pu.TOL_GRAD
    # dK, dV: the same products in fp32, summed over 64-row instead of 128-row query steps (a different but fixed
    # order): equal to the two-pass result up to the last bf16 bit of a few elements, and reproducible run to run
    for i in (1, 2, 4, 5):
        assert pu.rel_l2(synth.to_f64(one[i]), synth.to_f64(two[i])) <= 1e-3
    first = [t.clone() for t in one]
    again = pu.gpu_bwd(g, out, M, single_pass=True, window=w.window)
    torch.cuda.synchronize()
    for i in (1, 2, 4, 5):
        assert torch.equal(first[i], again[i])
    p = binding.make_params(w.batch, w.L, M, w.H, w.H_kv, w.d, bwd_single_pass=True)
    assert binding.bdlm_workspace_bytes(p, binding.BDLM_WS_BWD) >= 2 * w.batch * w.L * w.H * w.d * 4


@pytest.mark.parametrize("w,mode", [(Workload("mha_3tiles", 1, 2, 2, 128, 384, 32), 0),
                                    (Workload("g3_5tiles", 2, 3, 1, 128, 640, 64), 0),
                                    (Workload("mha_1tile", 1, 1, 1, 128, 128, 16), 1),
                                    (Workload("g1_window", 1, 2, 2, 128, 768, 32, window=200), 0),
                                    (Workload("g3_m256", 1, 3, 1, 128, 512, 256), 1)], ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_odd_group_sizes(w, mode):
    """An odd number of query heads per KV head (MHA included): the forward pairs two consecutive query tiles of
    one head per CTA -- odd tile counts leave the last pair half empty -- and the backward kernels walk G heads."""
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode)
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode, single_pass=True)


def test_trailing_padding_leaves_real_rows_unchanged():
    """A length that is no multiple of 128 takes the mma.sync kernels; padded with trailing rows (dO = 0 there) to
    a multiple of 128 it takes the tensor-core kernels, and nothing changes for the real rows: later positions are
    invisible to every earlier row of either stream."""
    w = Workload("ragged", 1, 4, 2, 128, 160, 32)
    inp = synth.make_inputs(w, "cpu")
    x = pu.f64(inp)
    M, L, Lp = w.block_size, w.L, 256
    pad = {}
    gen = torch.Generator().manual_seed(7)
    for n, t in inp.items():
        extra = torch.randn((t.shape[0], Lp - L) + tuple(t.shape[2:]), generator=gen).to(t.dtype)
        if n.startswith("do_"):
            extra.zero_()
        pad[n] = torch.cat([t, extra], dim=1).contiguous()
    g = pu.to_cuda(pad)
    out = pu.gpu_fwd(g, M, impl=binding.IMPL_TCGEN05)
    ref = orc.attn_forward(*[x[n] for n in pu.NAMES6], M)
    for got, want, tol, is_lse in ((out[0], ref[0], pu.TOL_O, False), (out[1], ref[1], pu.TOL_LSE, True),
                                   (out[2], ref[2], pu.TOL_O, False), (out[3], ref[3], pu.TOL_LSE, True)):
        gotn = synth.to_f64(got)
        gotn = gotn[:, :, :L] if is_lse else gotn[:, :L]
        assert np.abs(gotn - want).max() <= tol
    gref = orc.attn_backward(*[x[n] for n in pu.NAMES6], x["do_clean"], x["do_noisy"], M)
    for sp in (False, True):
        grads = pu.gpu_bwd(g, out, M, impl=binding.IMPL_TCGEN05, single_pass=sp)
        torch.cuda.synchronize()
        assert binding.bdlm_get_device_status() == 0
        for got, want in zip(grads, gref):
            assert pu.rel_l2(synth.to_f64(got)[:, :L], want) <= pu.TOL_GRAD


@pytest.mark.parametrize("impl", IMPLS)
def test_large_logits(impl):
    """Scores with a standard deviation of about 10 nats (q and k six times larger than in the workloads):
    sharply peaked rows, row maxima that keep growing along the keys -- the running-maximum bookkeeping of
    the forward (rescale only after a growth of 2^8) and the exp(S - LSE) recomputation of the backward."""
    w = Workload("peaked", 1, 4, 2, 128, 640, 32)
    inp = synth.make_inputs(w, "cpu")
    for n in ("q_clean", "k_clean", "q_noisy", "k_noisy"):
        inp[n] = (inp[n].float() * 6.0).to(torch.bfloat16)
    # make the clean keys' scores drift upwards along the sequence for some rows: every later tile raises the maximum
    ramp = torch.linspace(0.0, 3.0, w.L).view(1, w.L, 1, 1)
    inp["k_clean"] = (inp["k_clean"].float() + ramp * inp["q_clean"].float().mean(dim=(1, 2), keepdim=True).sign()).to(torch.bfloat16)
    pu.check_full(w, impl, inp=inp)


def test_default_backward_takes_the_fused_kernel_when_the_workspace_has_room():
    """bdlm_params zeroed (BDLM_BWD_AUTO): with the workspace bdlm_workspace_bytes recommends the fused kernel runs
    (dK, dV bitwise those of the forced fused call), with only the D rows' worth of workspace the two-pass kernels
    run (every gradient bitwise that of the forced two-pass call); a forced fused call refuses the small workspace."""
    w = Workload("auto_bwd", 1, 4, 2, 128, 512, 32)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    M = w.block_size
    out = pu.gpu_fwd(g, M)
    mk = lambda sp: binding.make_params(w.batch, w.L, M, w.H, w.H_kv, w.d, bwd_single_pass=sp)
    big = binding.bdlm_workspace_bytes(mk(None), binding.BDLM_WS_BWD)
    small = binding.bdlm_workspace_bytes(mk(False), binding.BDLM_WS_BWD)
    assert big == binding.bdlm_workspace_bytes(mk(True), binding.BDLM_WS_BWD)
    assert big >= small + 2 * w.batch * w.L * w.H * 128 * 4 and small >= 2 * w.batch * w.H * w.L * 4
    ws_big = torch.empty(big, dtype=torch.uint8, device="cuda")
    ws_small = torch.empty(small, dtype=torch.uint8, device="cuda")
    fused = [t.clone() for t in pu.gpu_bwd(g, out, M, single_pass=True, workspace=ws_big)]
    two = [t.clone() for t in pu.gpu_bwd(g, out, M, single_pass=False, workspace=ws_small)]
    auto_big = [t.clone() for t in pu.gpu_bwd(g, out, M, single_pass=None, workspace=ws_big)]
    auto_small = [t.clone() for t in pu.gpu_bwd(g, out, M, single_pass=None, workspace=ws_small)]
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    for a, b in zip(auto_small, two):
        assert torch.equal(a, b)
    for i in (1, 2, 4, 5):
        assert torch.equal(auto_big[i], fused[i])
    assert not all(torch.equal(two[i], fused[i]) for i in (1, 2, 4, 5))   # the two paths are told apart by their rounding
    for i in (0, 3):
        assert pu.rel_l2(synth.to_f64(auto_big[i]), synth.to_f64(two[i])) <= 1e-3
    with pytest.raises(binding.BdlmError) as e:
        pu.gpu_bwd(g, out, M, single_pass=True, workspace=ws_small)
    assert e.value.status == -3


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """The library's self-test kernel lets one bounded wait run out (a barrier nothing completes, a limit of about a
    millisecond of clock ticks): the device status reads BDLM_ERR_DEVICE_TIMEOUT exactly once, and the next
    forward on the same context is correct."""
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    binding.bdlm_selftest_wait_timeout(2_000_000)
    assert binding.bdlm_get_device_status() == -5
    assert binding.status_string(-5) == "BDLM_ERR_DEVICE_TIMEOUT"
    assert binding.bdlm_get_device_status() == 0
    with pytest.raises(binding.BdlmError):
        binding.bdlm_selftest_wait_timeout(0)
    pu.check_full(Workload("after_timeout", 1, 2, 1, 128, 256, 32), binding.IMPL_AUTO, check_bwd=False)


@pytest.mark.parametrize("w,mode", [(synth.WORKLOADS["tiny"], 0),                                  # the BASELINE tiny configuration: MHA, M = 16
                                    (Workload("d64_gqa", 2, 4, 2, 64, 384, 32), 0),
                                    (Workload("d64_g4_m256", 1, 4, 1, 64, 512, 256), 1),
                                    (Workload("d64_g3_window", 1, 3, 1, 64, 640, 64, window=200), 0)],
                         ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_head_dimension_64_on_the_tensor_core_kernels(w, mode):
    """d = 64 on the tcgen05 kernels (one 64-column panel per operand tile, four k-slices over the head dimension):
    forward, two-pass backward and fused backward, forced with impl = 2 so that a fallback would show as an error."""
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode)
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode, single_pass=True)
    # the portable kernels on the same inputs stay available as the cross-check
    pu.check_full(w, binding.IMPL_PORTABLE, mode=mode)


def test_head_dimension_64_default_dispatch_is_the_tensor_core_path():
    """impl = 0 takes the tensor-core kernels for d = 64 (bitwise the impl = 2 results), and the packed form does too."""
    w = Workload("d64_auto", 1, 4, 2, 64, 256, 16)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    M = w.block_size
    a = pu.gpu_fwd(g, M)
    b = pu.gpu_fwd(g, M, impl=binding.IMPL_TCGEN05)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    ga = pu.gpu_bwd(g, a, M)
    gb = pu.gpu_bwd(g, a, M, impl=binding.IMPL_TCGEN05)
    torch.cuda.synchronize()
    for x, y in zip(ga, gb):
        assert torch.equal(x, y)
    assert binding.bdlm_get_device_status() == 0


@pytest.mark.parametrize("w,mode", [(Workload("ragged_tail_tc", 1, 2, 1, 64, 200, 8), 0),          # one full tile + 72 rows
                                    (Workload("ragged_short_tc", 1, 4, 2, 128, 40, 8), 0),         # less than one tile
                                    (Workload("ragged_w100_tc", 1, 4, 2, 128, 456, 8, window=100), 0),
                                    (Workload("ragged_odd_tc", 2, 3, 1, 128, 322, 7), 1),          # rows not 16-byte aligned in LSE / D
                                    (Workload("ragged_m1_tc", 1, 2, 2, 64, 130, 1), 0),
                                    (Workload("ragged_bigblock_tc", 1, 4, 1, 128, 600, 300), 1)],
                         ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_lengths_that_are_no_multiple_of_the_tile_on_the_tensor_core_kernels(w, mode):
    """TMA zero-fills the part of a tile past the end of a tensor; keys past the end are never visible, rows past the
    end are neither read from LSE / D nor written.  Forced with impl = 2: forward, two-pass and fused backward."""
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode)
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode, single_pass=True)


def test_ragged_outputs_do_not_touch_memory_past_the_tensors():
    """Outputs and gradients sit inside larger buffers filled with a sentinel: nothing past the last real row moves."""
    w = Workload("ragged_guard", 1, 4, 2, 128, 200, 8)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    M, L = w.block_size, w.L
    pad = 64

    def guarded(like, lse=False):
        shape = (like.shape[0], like.shape[1], L + pad) if lse else (like.shape[0] * (L + pad),) + tuple(like.shape[2:])
        return torch.full(shape, 7.0, dtype=like.dtype, device="cuda")

    bufs_o = [guarded(g["q_clean"]), torch.full((w.batch * w.H * L + pad,), 7.0, device="cuda"),
              guarded(g["q_noisy"]), torch.full((w.batch * w.H * L + pad,), 7.0, device="cuda")]
    out = (bufs_o[0][:L].view(1, L, w.H, w.d), bufs_o[1][:w.H * L].view(1, w.H, L),
           bufs_o[2][:L].view(1, L, w.H, w.d), bufs_o[3][:w.H * L].view(1, w.H, L))
    binding.bdlm_attn_fwd(*[g[n] for n in pu.NAMES6], M, out=out, impl=binding.IMPL_TCGEN05)
    gb = [guarded(g[n]) for n in pu.NAMES6]
    grads = tuple(b[:L].view(1, L, g[n].shape[2], w.d) for b, n in zip(gb, pu.NAMES6))
    for sp in (False, True):
        binding.bdlm_attn_bwd(*[g[n] for n in pu.NAMES6], out[0], out[1], out[2], out[3], g["do_clean"], g["do_noisy"], M,
                              out=grads, impl=binding.IMPL_TCGEN05, single_pass=sp)
        torch.cuda.synchronize()
        assert binding.bdlm_get_device_status() == 0
        for b in (bufs_o[0], bufs_o[2]) + tuple(gb):
            assert float((b[L:].float() - 7.0).abs().max()) == 0.0
        for b in (bufs_o[1], bufs_o[3]):
            assert float((b[w.H * L:] - 7.0).abs().max()) == 0.0
        assert torch.isfinite(grads[0].float()).all()


def test_many_heads_take_the_row_wise_d_preprocess():
    """With several hundred heads the tile of the D preprocess (32 rows x all heads) no longer fits shared memory and the
    warp-per-row form runs instead; both forms feed the same backward."""
    w = Workload("many_heads", 1, 384, 96, 64, 128, 16)
    pu.check_full(w, binding.IMPL_AUTO)
