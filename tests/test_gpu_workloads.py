"""Parity at the benchmark's full sizes: sampled query rows (256 per head and stream,
stratified over block, tile and shard boundaries) recomputed by the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import WORKLOADS

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["8k", "32k", "32k_m256", "32k_w1024"])
def test_sampled_rows_full_size(name):
    w = WORKLOADS[name]
    worst = pu.check_sampled(w, binding.IMPL_AUTO)
    print(name, worst)


@pytest.mark.parametrize("name", ["32k", "32k_w1024", "32k_m512", "32k_m1024"])
def test_sampled_rows_full_size_fused_backward(name):
    """The same check with the fused one-kernel backward, the configuration bench.py times."""
    w = WORKLOADS[name]
    worst = pu.check_sampled(w, binding.IMPL_AUTO, single_pass=True)
    print(name, "fused", worst)


def test_mha16k_sampled_rows():
    """One query head per KV head: the forward pairs consecutive query tiles of a head; both backward paths."""
    worst = pu.check_sampled(WORKLOADS["mha16k"], binding.IMPL_AUTO, single_pass=(False, True))
    print("mha16k", worst)


def test_dflash32k_sampled_rows_fused_backward():
    worst = pu.check_sampled_packed(WORKLOADS["dflash32k"], binding.IMPL_AUTO, single_pass=True)
    print("dflash32k fused", worst)


def test_dflash32k_sampled_rows():
    """DFlash2-shaped packed workload at the size bench.py runs it (2048 sampled blocks over 32K clean keys)."""
    worst = pu.check_sampled_packed(WORKLOADS["dflash32k"], binding.IMPL_AUTO)
    print("dflash32k", worst)


def test_csbp128k_shards_merge_and_oracle():
    """CSBP rank-local emulation: 8 contiguous clean-K/V shards, each partial computed on its
    own, merged with bdlm_lse_merge, compared with the unsharded kernel and the oracle."""
    w = WORKLOADS["csbp128k"]
    M = w.block_size
    g = synth.make_inputs(w, "cuda")
    step = w.L // w.kv_shards
    parts = [pu.gpu_fwd(g, M, kv_range=(s * step, (s + 1) * step), include_noisy_diag=False)
             for s in range(w.kv_shards)]
    diag = binding.bdlm_attn_fwd(None, g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"], g["v_noisy"], M,
                                 kv_range=(0, 0))
    o_c, l_c = binding.bdlm_lse_merge([p[0] for p in parts], [p[1] for p in parts])
    o_n, l_n = binding.bdlm_lse_merge([p[2] for p in parts] + [diag[2]], [p[3] for p in parts] + [diag[3]])
    del parts, diag
    full = pu.gpu_fwd(g, M)
    torch.cuda.synchronize()
    for got, ref, tol in ((o_c, full[0], pu.TOL_O), (l_c, full[1], pu.TOL_LSE), (o_n, full[2], pu.TOL_O), (l_n, full[3], pu.TOL_LSE)):
        assert float((got.float() - ref.float()).abs().max()) <= tol
    # the merged result feeds the oracle comparison and the (unsharded) backward
    # (both backward paths against one evaluation of the oracle: the fused one is what bench.py times at this size)
    pu.check_sampled(w, binding.IMPL_AUTO, g=g, fwd_out=(o_c, l_c, o_n, l_n), single_pass=(False, True))


def test_256k_sampled_rows():
    """Both backward paths (two-pass and fused) against one evaluation of the oracle's sampled rows."""
    w = WORKLOADS["256k"]
    worst = pu.check_sampled(w, binding.IMPL_AUTO, single_pass=(False, True))
    print("256k", worst)


def test_8k_sampled_rows_clean_mask_mode_1():
    """The other reading of "block-causal" (a clean query sees its whole own clean block) at a full-size workload,
    both backward paths."""
    worst = pu.check_sampled(WORKLOADS["8k"], binding.IMPL_AUTO, single_pass=(False, True), mode=1)
    print("8k mode 1", worst)
