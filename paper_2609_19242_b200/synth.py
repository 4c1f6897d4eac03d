"""Seeded synthetic inputs for the BDLM attention layer.

This module only makes inputs and picks sample rows; it holds none of the attention
arithmetic, so both the CUDA path's callers and the CPU oracle's tests may use it.

The paper's throughput runs use sequences that all have exactly the stated context length
(section 5.1) and give no head counts or activation statistics; the workloads below use
Llama-3-8B-like head shapes with q/k/v ~ 0.5 * N(0,1) rounded to bf16 and upstream
gradients dO ~ N(0,1) rounded to bf16.  They stand in for the paper's long-context
workloads.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    H: int
    H_kv: int
    d: int
    L: int            # clean length; the noisy stream has the same length
    block_size: int
    rope_theta: float = 0.0   # > 0: rotate q and k before rounding to bf16
    kv_shards: int = 1        # > 1: forward is also run as that many clean-K/V shard partials
    seed: int = 0
    window: int = 0           # > 0: sliding-window layer, clean key j visible only if i - j < window
    n_blocks: int = 0         # > 0: DFlash2-style packed form -- no clean queries, n_blocks sampled blocks whose
                              # anchors (clean-prefix lengths) are drawn uniformly from [0, L] and sorted

    @property
    def packed(self):
        return self.n_blocks > 0

    def anchors(self):
        """Sorted anchor positions of the sampled blocks (packed workloads), int64 numpy."""
        rng = np.random.default_rng(self.seed + 7919)
        return np.sort(rng.integers(0, self.L + 1, size=self.n_blocks)).astype(np.int64)

    def pairs_per_head(self):
        """Unmasked (query, key) pairs per (batch, query head): clean L(L+1)/2 and noisy
        L(L+M)/2 (appendix B, Eq. aligned-rank-work with P = 1); with a sliding window the
        clean keys of row i are cut to the last `window` positions up to i."""
        L, M, W = self.L, self.block_size, self.window
        if self.packed:
            return 0, int((M * (M + self.anchors())).sum())
        if W <= 0:
            return L * (L + 1) // 2, L * (L + M) // 2
        i = np.arange(L, dtype=np.int64)
        clean = np.minimum(i + 1, W).sum()
        noisy = (M + np.maximum(0, (i // M) * M - np.maximum(0, i - W + 1))).sum()
        return int(clean), int(noisy)

    def flops(self):
        """(forward, backward) FLOPs over unmasked pairs only: 4d and 10d per pair."""
        c, n = self.pairs_per_head()
        pairs = (c + n) * self.batch * self.H
        return 4 * self.d * pairs, 10 * self.d * pairs


WORKLOADS = {
    "tiny": Workload("tiny", 1, 2, 2, 64, 256, 16),
    "8k": Workload("8k", 2, 16, 4, 128, 8192, 32),
    "32k": Workload("32k", 1, 32, 8, 128, 32768, 64, rope_theta=5e5),
    "csbp128k": Workload("csbp128k", 1, 32, 8, 128, 131072, 32, kv_shards=8),
    "256k": Workload("256k", 1, 32, 8, 128, 262144, 16),
    # paper-shaped block size (appendix J uses 128..1024, default 256); not a BASELINE config
    "32k_m256": Workload("32k_m256", 1, 32, 8, 128, 32768, 256, rope_theta=5e5),
    "32k_m512": Workload("32k_m512", 1, 32, 8, 128, 32768, 512, rope_theta=5e5),
    "32k_m1024": Workload("32k_m1024", 1, 32, 8, 128, 32768, 1024, rope_theta=5e5),
    # sliding-window layer of a hybrid model (appendix K: 1,024-token windows); not a BASELINE config
    "32k_w1024": Workload("32k_w1024", 1, 32, 8, 128, 32768, 64, rope_theta=5e5, window=1024),
    # DFlash2-shaped drafter layer (appendix E): 32K target-feature keys, 2048 sampled blocks of 16 tokens
    "dflash32k": Workload("dflash32k", 1, 32, 8, 128, 32768, 16, n_blocks=2048),
    # multi-head attention without KV sharing (one query head per KV head); not a BASELINE config
    "mha16k": Workload("mha16k", 1, 8, 8, 128, 16384, 32),
}


def small(w: Workload, **kw) -> Workload:
    return replace(w, **kw)


def _rope(x: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding in fp32, half-split pairing (x_k, x_{k+d/2}); token i of either
    stream uses position i.  x is [batch, L, heads, d]."""
    _, L, _, d = x.shape
    half = d // 2
    inv = theta ** (-torch.arange(half, device=x.device, dtype=torch.float32) / half)
    ang = torch.arange(L, device=x.device, dtype=torch.float32)[:, None] * inv[None, :]
    cos = ang.cos()[None, :, None, :]
    sin = ang.sin()[None, :, None, :]
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * cos - b * sin, a * sin + b * cos], dim=-1)


def make_inputs(w: Workload, device="cpu", with_grad=True):
    """Dict of bf16 tensors: q_clean,k_clean,v_clean,q_noisy,k_noisy,v_noisy and (optionally)
    do_clean, do_noisy.  The same seed on the same device type gives the same bits; callers
    that compare two implementations hand both the SAME tensors.  A packed (DFlash2-style)
    workload has no clean queries (q_clean, do_clean are None), noisy tensors of
    n_blocks*block_size rows and an int32 `block_prefix` tensor with the sorted anchors."""
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    out = {}

    def draw(rows, heads, sigma):
        return torch.randn(w.batch, rows, heads, w.d, generator=g, device=device,
                           dtype=torch.float32) * sigma

    for stream in ("clean", "noisy"):
        rows = w.n_blocks * w.block_size if (w.packed and stream == "noisy") else w.L
        q, k, v = draw(rows, w.H, 0.5), draw(rows, w.H_kv, 0.5), draw(rows, w.H_kv, 0.5)
        if w.rope_theta > 0:
            q, k = _rope(q, w.rope_theta), _rope(k, w.rope_theta)
        out[f"q_{stream}"] = q.to(torch.bfloat16)
        out[f"k_{stream}"] = k.to(torch.bfloat16)
        out[f"v_{stream}"] = v.to(torch.bfloat16)
        del q, k, v
    if with_grad:
        for stream in ("clean", "noisy"):
            rows = w.n_blocks * w.block_size if (w.packed and stream == "noisy") else w.L
            out[f"do_{stream}"] = draw(rows, w.H, 1.0).to(torch.bfloat16)
    if w.packed:
        out["q_clean"] = None
        if with_grad:
            out["do_clean"] = None
        out["block_prefix"] = torch.from_numpy(w.anchors()).to(torch.int32).to(device)
    return out


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a (bf16/fp32) tensor to a float64 numpy array on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def sample_rows(w: Workload, n: int, seed: int, extra=()):
    """Stratified query rows for the sampled-row checks: the rows where masks change
    (sequence ends, block and 128-tile boundaries, K/V-shard boundaries) plus a uniform
    random remainder.  Returns a sorted int64 array of n distinct rows in [0, L)."""
    L, M = w.L, w.block_size
    rng = np.random.default_rng(seed)
    fixed = [0, 1, M - 1, M, 127, 128, L - M - 1, L - M, L - 1, L // 2 - 1, L // 2]
    for blk in rng.integers(0, L // M, size=4):
        fixed += [int(blk) * M, int(blk) * M + M - 1]
    if w.kv_shards > 1:
        step = L // w.kv_shards
        for s in range(1, w.kv_shards):
            fixed += [s * step - 1, s * step, s * step + M]
    if w.window > 0:
        fixed += [w.window - 2, w.window - 1, w.window, w.window + M]
    fixed += list(extra)
    rows = sorted({r for r in fixed if 0 <= r < L})
    rows = rows[:n]
    if len(rows) < min(n, L):
        pool = np.setdiff1d(np.arange(L), np.asarray(rows, dtype=np.int64))
        more = rng.choice(pool, size=min(n, L) - len(rows), replace=False)
        rows = sorted(set(rows) | set(int(x) for x in more))
    return np.asarray(rows, dtype=np.int64)



# ------------------------------------------------------------------------------------------
# linear cross-entropy head (the step after the last layer)
# ------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class LceWorkload:
    """Hidden states h ~ N(0,1), output embedding W ~ N(0,1) * logit_std / sqrt(D) (logits with a standard deviation
    of `logit_std`), targets uniform over the vocabulary with a fraction `ignored` of positions set to -100 (clean
    positions and unmasked tokens carry no loss), per-token weights uniform in [0.5, 2] (the w(t_b) of Eq.
    bdlm-training-objective differ from block to block).  The paper gives neither the vocabulary nor the hidden size;
    the named workload uses Llama-3-8B's (D = 4096, V = 128256)."""
    name: str
    T: int
    D: int
    V: int
    logit_std: float = 2.0
    ignored: float = 0.25
    seed: int = 0

    def flops(self):
        """(forward, backward) FLOPs: the projection 2 T D V; backward = the dH and dW products, 4 T D V (the
        recomputation of the logits is executed but not counted)."""
        f = 2 * self.T * self.D * self.V
        return f, 2 * f


LCE_WORKLOADS = {
    "lce_tiny": LceWorkload("lce_tiny", 200, 64, 1000),
    "lce_8k": LceWorkload("lce_8k", 8192, 4096, 128256),
    # small enough for a full profiler capture, operands still larger than L2
    "lce_small": LceWorkload("lce_small", 4096, 2048, 32768),
}


def make_lce_inputs(w: LceWorkload, device="cpu"):
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    h = torch.randn(w.T, w.D, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    W = (torch.randn(w.V, w.D, generator=g, device=device, dtype=torch.float32) * (w.logit_std / w.D ** 0.5)).to(torch.bfloat16)
    labels = torch.randint(0, w.V, (w.T,), generator=g, device=device, dtype=torch.int32)
    drop = torch.rand(w.T, generator=g, device=device) < w.ignored
    labels = torch.where(drop, torch.full_like(labels, -100), labels)
    weight = 0.5 + 1.5 * torch.rand(w.T, generator=g, device=device, dtype=torch.float32)
    return {"h": h, "w": W, "labels": labels, "weight": weight}
