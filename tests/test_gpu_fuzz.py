"""Seeded random configurations against the oracle: block sizes, lengths (tensor-core and ragged), head
groupings, mask mode, sliding window, packed blocks with random prefix tables, clean runs at random offsets,
clean-key shard ranges.  Each case is small enough for the full fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import Workload

import parity_util as pu
from test_gpu_packed import _draw, _run_and_check

pytestmark = pytest.mark.gpu


def _plain_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        d = int(rng.choice([64, 128, 128, 128]))
        M = int(rng.choice([1, 4, 8, 16, 32, 48, 64, 128, 256]))
        nblk = int(rng.integers(1, max(2, 640 // M) + 1))
        L = M * nblk
        if rng.random() < 0.6:                       # steer most cases onto the tensor-core path
            L = max(128, (L // 128) * 128)
            while L % M:
                L += 128
        Hkv = int(rng.choice([1, 2]))
        G = int(rng.choice([1, 2, 3, 4]))
        window = int(rng.choice([0, 0, 0, 1, 17, 128, 200]))
        mode = int(rng.choice([0, 0, 1]))
        cases.append((Workload(f"fuzz{i}", int(rng.choice([1, 2])), Hkv * G, Hkv, d, L, M, window=window, seed=100 + i), mode))
    return cases


@pytest.mark.parametrize("case", _plain_cases(24, 2024), ids=lambda c: f"{c[0].name}-L{c[0].L}-M{c[0].block_size}-H{c[0].H}/{c[0].H_kv}-d{c[0].d}-w{c[0].window}-m{c[1]}")
def test_random_plain_configurations(case):
    w, mode = case
    pu.check_full(w, binding.IMPL_AUTO, mode=mode)


@pytest.mark.parametrize("case", _plain_cases(24, 2024),
                         ids=lambda c: f"{c[0].name}-L{c[0].L}-M{c[0].block_size}-H{c[0].H}/{c[0].H_kv}-d{c[0].d}-w{c[0].window}-m{c[1]}")
def test_random_plain_configurations_fused_backward(case):
    """Every case again through the fused one-kernel backward, forced onto the tensor-core kernels (head dimension 64
    and lengths that are no multiple of the 128-row tile included)."""
    w, mode = case
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode, single_pass=True)


@pytest.mark.parametrize("case", _plain_cases(24, 2024),
                         ids=lambda c: f"{c[0].name}-L{c[0].L}-M{c[0].block_size}-H{c[0].H}/{c[0].H_kv}-d{c[0].d}-w{c[0].window}-m{c[1]}")
def test_random_plain_configurations_portable_kernels(case):
    """The mma.sync kernels stay the explicit cross-check (impl = 1) now that the default never reaches them."""
    w, mode = case
    pu.check_full(w, binding.IMPL_PORTABLE, mode=mode)


def _larger_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        L = 128 * int(rng.integers(5, 15))
        M = int(rng.choice([m for m in (8, 16, 24, 32, 48, 64, 96, 128, 192, 256, 384) if L % m == 0]))
        Hkv, G = int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 3, 4, 5]))
        cases.append((Workload(f"big{i}", int(rng.choice([1, 2])), Hkv * G, Hkv, 128, L, M,
                               window=int(rng.choice([0, 0, 0, 130, 700])), seed=300 + i), int(rng.choice([0, 0, 1]))))
    return cases


@pytest.mark.parametrize("case", _larger_cases(6, 5), ids=lambda c: f"{c[0].name}-L{c[0].L}-M{c[0].block_size}-H{c[0].H}/{c[0].H_kv}-w{c[0].window}-m{c[1]}")
def test_random_larger_configurations(case):
    """Five to fourteen tiles per stream, group sizes 1 to 5, through the tensor-core kernels and both backward paths."""
    w, mode = case
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode)
    pu.check_full(w, binding.IMPL_TCGEN05, mode=mode, single_pass=True, check_bwd=True)


def _packed_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        M = int(rng.choice([8, 16, 32, 64, 128]))
        Lk = int(rng.choice([128, 256, 384, 512, 203, 330]))
        nb = int(rng.integers(1, 7)) * max(1, 128 // M)
        Lq = int(rng.choice([0, 128, 256, 37])) if Lk >= 256 else 0
        if Lq and Lk % 128:
            Lq = 37
        window = int(rng.choice([0, 0, 50, 160]))
        if window:
            step = rng.integers(M, M + 40, size=nb)
            prefix = np.minimum(np.cumsum(step) - step[0], Lk).tolist()
            prefix = [p for p in prefix]
            for j in range(1, nb):                  # keep the blocks apart after clipping at Lk
                if prefix[j] - prefix[j - 1] < M:
                    window = 0
        if not window:
            prefix = sorted(int(v) for v in rng.integers(0, Lk + 1, size=nb))
        pos0 = int(rng.integers(0, Lk - Lq + 1)) if Lq else 0
        d = 128 if (Lk % 128 == 0 and Lq % 128 == 0 and (nb * M) % 128 == 0 and rng.random() < 0.8) else int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2]))
        G = int(rng.choice([1, 2, 4]))
        cases.append(dict(seed=500 + i, Lk=Lk, Lq=Lq, Ln=nb * M, H=Hkv * G, Hkv=Hkv, d=d, M=M, prefix=prefix, pos0=pos0,
                          window=window, mode=int(rng.choice([0, 0, 1]))))
    return cases


@pytest.mark.parametrize("c", _packed_cases(16, 77), ids=lambda c: f"s{c['seed']}-Lk{c['Lk']}-Lq{c['Lq']}-Ln{c['Ln']}-M{c['M']}-d{c['d']}-w{c['window']}")
def test_random_packed_configurations(c):
    t = _draw(c["seed"], 1, c["Lk"], c["Lq"], c["Ln"], c["H"], c["Hkv"], c["d"])
    _run_and_check(t, c["M"], binding.IMPL_AUTO, prefix=c["prefix"], pos0=c["pos0"], window=c["window"], mode=c["mode"])
    if c["d"] == 128 and c["Lk"] % 128 == 0 and c["Lq"] % 128 == 0 and c["Ln"] % 128 == 0:   # tensor-core shaped: also the fused backward
        _run_and_check(t, c["M"], binding.IMPL_AUTO, prefix=c["prefix"], pos0=c["pos0"], window=c["window"], mode=c["mode"],
                       single_pass=True)


@pytest.mark.parametrize("seed", range(6))
def test_random_shard_ranges_merge_to_the_full_result(seed):
    """Random cuts of the clean keys into shards: each shard's partial plus the noisy-diagonal partial, merged,
    equals the oracle's unsharded forward."""
    rng = np.random.default_rng(900 + seed)
    M = int(rng.choice([16, 32, 64]))
    L = 128 * int(rng.integers(2, 6))
    w = Workload(f"shardfuzz{seed}", 1, 4, 2, 128, L, M, seed=seed)
    inp = synth.make_inputs(w, "cpu", with_grad=False)
    g, x = pu.to_cuda(inp), pu.f64(inp)
    cuts = sorted(set([0, L] + [int(v) for v in rng.integers(0, L + 1, size=int(rng.integers(1, 5)))]))
    parts = [pu.gpu_fwd(g, M, kv_range=(a, b), include_noisy_diag=False) for a, b in zip(cuts[:-1], cuts[1:])]
    diag = binding.bdlm_attn_fwd(None, g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"], g["v_noisy"], M, kv_range=(0, 0))
    o_c, l_c = binding.bdlm_lse_merge([p[0] for p in parts], [p[1] for p in parts])
    o_n, l_n = binding.bdlm_lse_merge([p[2] for p in parts] + [diag[2]], [p[3] for p in parts] + [diag[3]])
    torch.cuda.synchronize()
    ref = orc.attn_forward(*[x[n] for n in pu.NAMES6], M)
    for got, want, tol in ((o_c, ref[0], pu.TOL_O), (l_c, ref[1], pu.TOL_LSE), (o_n, ref[2], pu.TOL_O), (l_n, ref[3], pu.TOL_LSE)):
        assert np.abs(synth.to_f64(got) - want).max() <= tol
