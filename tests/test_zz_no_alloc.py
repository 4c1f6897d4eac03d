"""The allocation-free backward entry point (bdlm_attn_bwd_static_scratch), for callers that are
not allowed to allocate device memory -- e.g. a plug-in inside a framework whose pool owns the
whole GPU, or a latency-critical loop that cannot take an allocator's device-wide sync.

It must give the regular backward's results, twice in a row (the built-in scratch array keeps
the previous call's contents), and must refuse sizes beyond its fixed limit.  This file is
collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import ctypes

import pytest
import torch

from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import Workload

import parity_util as pu

pytestmark = pytest.mark.gpu


def _max_abs_diff(a, b):
    return float((a.float() - b.float()).abs().max())


@pytest.mark.parametrize("w", [Workload("na_d128", 2, 4, 2, 128, 384, 32), Workload("na_d64", 1, 2, 2, 64, 256, 16)],
                         ids=lambda w: w.name)
def test_static_scratch_backward_matches_regular_backward_twice(w):
    M = w.block_size
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    fwd = pu.gpu_fwd(g, M)
    ref = [t.clone() for t in pu.gpu_bwd(g, fwd, M)]
    torch.cuda.synchronize()
    out = tuple(torch.empty_like(t) for t in ref)            # caller-owned outputs: the call allocates nothing
    g2 = dict(g)
    g2["do_clean"] = (g["do_clean"].float() * -2.0).to(torch.bfloat16)
    g2["do_noisy"] = (g["do_noisy"].float() * 0.5).to(torch.bfloat16)
    def two_calls(books):
        for call in range(2):
            if call == 1:
                # second call with a different upstream gradient first, so stale scratch would show
                binding.bdlm_attn_bwd_static_scratch(*[g2[n] for n in pu.NAMES6], fwd[0], fwd[1], fwd[2], fwd[3],
                                                     g2["do_clean"], g2["do_noisy"], M, out=out)
            for t in out:
                t.fill_(float("nan"))
            binding.bdlm_attn_bwd_static_scratch(*[g[n] for n in pu.NAMES6], fwd[0], fwd[1], fwd[2], fwd[3],
                                                 g["do_clean"], g["do_noisy"], M, out=out)
            torch.cuda.synchronize()
            if books is not None:
                assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == books[:2]
                assert torch.cuda.mem_get_info()[0] == books[2]
            assert binding.bdlm_get_device_status() == 0
            for got, want in zip(out, ref):
                assert torch.isfinite(got.float()).all()
                # same kernels, same fixed summation order: equal within the gradient tolerance (in fact bitwise)
                assert pu.rel_l2(synth.to_f64(got), synth.to_f64(want)) <= pu.TOL_GRAD
                assert _max_abs_diff(got, want) == 0.0

    # A first pass does everything once: the library looks up its scratch array's address on this device, and the
    # driver loads the code of every kernel used below (the library's and those of the test's own torch calls), which
    # takes device memory the first time.  Then the books are opened: in the second pass neither torch's allocator
    # nor the driver may hand out a byte at the points where the entry point has just run.
    two_calls(None)
    torch.cuda.synchronize()
    two_calls((torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]))


def test_static_scratch_rejects_sizes_beyond_its_limit():
    # batch*H*L just above the limit: refused before any pointer is touched or anything is launched
    rows = binding.STATIC_SCRATCH_ROWS
    p = binding.make_params(1, rows // 32 + 128, 128, 32, 8, 128)
    assert p.batch * p.H * p.L > rows
    fake = ctypes.c_void_p(0x1000)
    rc = binding.lib().bdlm_attn_bwd_static_scratch(ctypes.byref(p), *([fake] * 18), None)
    assert rc == -6
    assert binding.status_string(rc) == "BDLM_ERR_STATIC_SCRATCH_TOO_SMALL"
    # invalid parameters are still rejected as such
    bad = binding.make_params(1, 100, 16, 4, 2, 128)
    assert binding.lib().bdlm_attn_bwd_static_scratch(ctypes.byref(bad), *([fake] * 18), None) == -1


def test_static_scratch_always_runs_the_two_pass_kernels_and_reports_errors_like_the_regular_call():
    w = Workload("na_mode", 1, 4, 2, 128, 256, 32)
    M = w.block_size
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    fwd = pu.gpu_fwd(g, M)
    ref = [t.clone() for t in pu.gpu_bwd(g, fwd, M, single_pass=False)]
    out = tuple(torch.empty_like(t) for t in ref)
    args = [binding._ptr(g[n]) for n in pu.NAMES6] + [binding._ptr(t) for t in (fwd[0], fwd[2], fwd[1], fwd[3])] + \
           [binding._ptr(g["do_clean"]), binding._ptr(g["do_noisy"])] + [binding._ptr(t) for t in out]
    for sp in (None, True, False):     # the field is ignored: the fused kernel's accumulators do not fit a fixed array
        for t in out:
            t.zero_()
        p = binding.make_params(w.batch, w.L, M, w.H, w.H_kv, w.d, bwd_single_pass=sp)
        rc = binding.lib().bdlm_attn_bwd_static_scratch(ctypes.byref(p), *args, binding._stream())
        assert rc == 0
        torch.cuda.synchronize()
        for got, want in zip(out, ref):
            assert torch.equal(got, want)
    fake = ctypes.c_void_p(0x1000)
    d96 = binding.make_params(1, 256, 16, 4, 2, 96)
    assert binding.lib().bdlm_attn_bwd_static_scratch(ctypes.byref(d96), *([fake] * 18), None) == -2
    d96.bwd_single_pass = 1
    assert binding.lib().bdlm_attn_bwd_static_scratch(ctypes.byref(d96), *([fake] * 18), None) == -2
