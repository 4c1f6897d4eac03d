#!/usr/bin/env python
"""Benchmark of the BDLM attention layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 32k] [--impl ours|reference]

A step is one forward plus one backward of the whole layer over one batch of seeded
synthetic inputs.  `value` counts FLOPs of unmasked (query, key) pairs only
(14 * d per pair: 4d forward, 10d backward).  Prints ONE JSON line on rank 0.

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its
own GPU: the layer as specified does not shard and has no collective, so the aggregate is
N replicas ("replicas only", weak scaling); ranks only meet at the timing barriers.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_19242_b200 import synth  # noqa: E402

METRIC = "BDLM attn fwd+bwd TFLOP/s (unmasked FLOPs)"
UNIT = "TFLOP/s"
NAMES6 = ["q_clean", "k_clean", "v_clean", "q_noisy", "k_noisy", "v_noisy"]

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of a kernel from a one-pass ncu capture of
# this command, keyed by (workload, kernel), each with the digest of the kernel sources it was captured on
# (kernel_source_digest): a figure is reported only for the build it belongs to.
_CAPTURED_ON = "4289fc252fec25f2"
NCU_TRAFFIC = {
    ("32k", "fwd"): {"bytes": 967480576 + 528095488, "kernel_source": _CAPTURED_ON},
    ("32k", "bwd_fused"): {"bytes": 5889652992 + 3375495168, "kernel_source": _CAPTURED_ON},
    ("32k", "bwd_dkdv"): {"bytes": 2371290368 + 249625600, "kernel_source": _CAPTURED_ON},
    ("32k", "bwd_dq"): {"bytes": 1543090432 + 519066880, "kernel_source": _CAPTURED_ON},
}
TRAFFIC_NOTE = ("dram__bytes_read.sum + dram__bytes_write.sum per launch from a one-pass ncu capture of this command on "
                "the 32k workload")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.index), "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            try:
                pw.append(float(r[2]))
            except ValueError:
                pass
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "power_w_max": max(pw) if pw else None}   # nvidia-smi averages power.draw over about a second: the maximum over the samples is the closest to the draw under load


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        parts = [p for p in vis.split(",") if p != ""]
        if local < len(parts) and parts[local].isdigit():
            return int(parts[local])
    return local


# ------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the fp64 oracle on a bounded sample of the workload
# ------------------------------------------------------------------------------------------
def oracle_sample(w, inp_cpu, rows_per_stream, seed):
    """Runs the oracle (forward + backward) for `rows_per_stream` sampled query rows of one
    (batch 0, head 0) per stream.  Returns (seconds, FLOPs of the visible pairs of those rows)."""
    from oracle import bdlm_oracle as orc
    M = w.block_size
    kv = {n: synth.to_f64(inp_cpu[n][0, :, 0]) for n in ("k_clean", "v_clean", "k_noisy", "v_noisy")}
    rng = np.random.default_rng(seed)
    flops = 0
    t0 = time.perf_counter()
    if w.packed:   # DFlash2-style blocks: noisy queries only, per-block prefix table
        anchors = w.anchors()
        Ln = w.n_blocks * M
        rows = np.sort(rng.choice(Ln, size=min(2 * rows_per_stream, Ln), replace=False))
        q_rows = synth.to_f64(inp_cpu["q_noisy"][0, rows, 0])
        do_rows = synth.to_f64(inp_cpu["do_noisy"][0, rows, 0])
        orc.attn_rows_packed(1, rows, q_rows, kv["k_clean"], kv["v_clean"], kv["k_noisy"], kv["v_noisy"], M,
                             do_rows=do_rows, block_prefix=anchors)
        flops = 14 * w.d * int((M + anchors[rows // M]).sum())
        return time.perf_counter() - t0, flops
    for s, (qn, dn) in enumerate((("q_clean", "do_clean"), ("q_noisy", "do_noisy"))):
        rows = np.sort(rng.choice(w.L, size=min(rows_per_stream, w.L), replace=False))
        q_rows = synth.to_f64(inp_cpu[qn][0, rows, 0])
        do_rows = synth.to_f64(inp_cpu[dn][0, rows, 0])
        orc.attn_rows(s, rows, q_rows, kv["k_clean"], kv["v_clean"], kv["k_noisy"], kv["v_noisy"], M, do_rows=do_rows,
                      window=w.window)
        if w.window > 0:
            lo = np.maximum(0, rows - w.window + 1)
            pairs = (rows + 1 - lo).sum() if s == 0 else (M + np.maximum(0, (rows // M) * M - lo)).sum()
        else:
            pairs = (rows + 1).sum() if s == 0 else ((rows // M + 1) * M).sum()
        flops += 14 * w.d * int(pairs)
    return time.perf_counter() - t0, flops


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return len(os.sched_getaffinity(0))


def cpu_inputs_for_oracle(w):
    """bf16 inputs of (batch 0, head 0 / KV head 0) only, on the host, same recipe as the GPU's."""
    small = synth.small(w, batch=1, H=1, H_kv=1)
    return synth.make_inputs(small, "cpu")


def timed_oracle_sample(w, inp, target_seconds, max_rows):
    """Calibrates on a small sample, then runs one sample sized for about `target_seconds` of CPU work."""
    oracle_sample(w, inp, 8, seed=99)                      # warm-up (BLAS threads, page faults)
    t_cal, _ = oracle_sample(w, inp, 64, seed=98)
    rows = int(min(max_rows, max(64, 64 * target_seconds / max(t_cal, 1e-3))))
    t, f = oracle_sample(w, inp, rows, seed=0)
    if t < 0.5 * target_seconds and rows < max_rows:   # the small calibration sample is dominated by fixed costs
        rows = int(min(max_rows, rows * target_seconds / max(t, 1e-3)))
        t, f = oracle_sample(w, inp, rows, seed=0)
    return rows, t, f


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = cpu_inputs_for_oracle(w)
    # each step is a bounded sample; the whole run is sized to end within a few minutes
    oracle_sample(w, inp, 8, seed=99)
    t_cal, _ = oracle_sample(w, inp, 64, seed=98)
    per_step_s = min(20.0, 120.0 / max(1, args.steps + args.warmup))
    rows = args.oracle_rows if args.oracle_rows > 0 else int(min(w.L, max(64, 64 * per_step_s / max(t_cal, 1e-3))))
    for i in range(args.warmup):
        oracle_sample(w, inp, rows, seed=100 + i)
    t_tot, f_tot = 0.0, 0
    for i in range(args.steps):
        t, f = oracle_sample(w, inp, rows, seed=i)
        t_tot += t
        f_tot += f
    val = f_tot / t_tot / 1e12
    cores = blas_threads()
    sample = f"{rows} sampled query rows per stream of (batch 0, head 0) per step, fwd+bwd, fp64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "batch": w.batch, "H": w.H, "H_kv": w.H_kv,
                                            "d": w.d, "L": w.L, "block_size": w.block_size, "window": w.window, "n_blocks": w.n_blocks},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(value_ms, device, world):
    """Slowest rank's time (every multi-GPU number is the max over ranks)."""
    if world <= 1:
        return float(value_ms)
    import torch.distributed as dist
    t = torch.tensor([float(value_ms)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flops_per_replica, ms_per_step, world):
    """Whole-job throughput of `world` independent replicas that each do `flops_per_replica` per step."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def kernel_source_digest():
    """sha256 over the tensor-core kernel sources: an ncu traffic figure belongs to the build it was captured on."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2609_19242_b200", "csrc")
    for f in ("bdlm_common.cuh", "tc_common.cuh", "tc_kernels.cu", "tc_bwd_kernels.cu"):
        with open(os.path.join(csrc, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


class LayerRun:
    """Inputs, outputs and workspace of one workload on the current device, and the calls of one step."""

    def __init__(self, w, binding, seed_offset, impl, fused):
        self.w, self.binding, self.impl, self.fused = w, binding, impl, fused
        self.M = w.block_size
        self.g = synth.make_inputs(synth.small(w, seed=w.seed + seed_offset), "cuda")
        self.fwd_out, self.grads, self.ws = self.make_buffers(self.g)

    def like(self, t):
        return None if t is None else torch.empty_like(t)

    def lse_like(self, q):
        w = self.w
        return None if q is None else torch.empty(w.batch, w.H, q.shape[1], dtype=torch.float32, device="cuda")

    def make_buffers(self, gg):
        """Outputs, gradients and workspace of one step for the inputs `gg`."""
        w, binding = self.w, self.binding
        fo = (self.like(gg["q_clean"]), self.lse_like(gg["q_clean"]), self.like(gg["q_noisy"]), self.lse_like(gg["q_noisy"]))
        gr = tuple(self.like(gg[n]) for n in NAMES6)
        rows = max(t.shape[1] for t in (gg["q_clean"], gg["q_noisy"]) if t is not None)
        wsz = 2 * (w.batch * w.H * rows * 4 + 256)
        if self.fused:   # fp32 dQ accumulators of the fused backward, one per query stream
            wsz += sum(t.shape[1] for t in (gg["q_clean"], gg["q_noisy"]) if t is not None) * w.batch * w.H * w.d * 4
        if not w.packed:
            wsz = max(wsz, binding.bdlm_workspace_bytes(
                binding.make_params(w.batch, w.L, self.M, w.H, w.H_kv, w.d, bwd_single_pass=self.fused), binding.BDLM_WS_BWD))
        return fo, gr, torch.empty(wsz, dtype=torch.uint8, device="cuda")

    def run_fwd(self, gg=None, fo=None, **kw):
        w, binding = self.w, self.binding
        gg = self.g if gg is None else gg
        fo = self.fwd_out if fo is None else fo
        if w.packed:
            binding.bdlm_attn_fwd_packed(*[gg[n] for n in NAMES6], self.M, block_prefix=gg["block_prefix"], out=fo,
                                         impl=self.impl, window=w.window, **kw)
        else:
            binding.bdlm_attn_fwd(*[gg[n] for n in NAMES6], self.M, out=fo, impl=self.impl, window=w.window, **kw)

    def run_bwd(self, gg=None, fo=None, gr=None, wsb=None, passes=0):
        w, binding = self.w, self.binding
        gg = self.g if gg is None else gg
        fo = self.fwd_out if fo is None else fo
        gr = self.grads if gr is None else gr
        wsb = self.ws if wsb is None else wsb
        if w.packed:
            binding.bdlm_attn_bwd_packed(*[gg[n] for n in NAMES6], fo[0], fo[1], fo[2], fo[3], gg["do_clean"],
                                         gg["do_noisy"], self.M, block_prefix=gg["block_prefix"], out=gr, workspace=wsb,
                                         impl=self.impl, passes=passes, window=w.window, single_pass=self.fused)
        else:
            binding.bdlm_attn_bwd(*[gg[n] for n in NAMES6], fo[0], fo[1], fo[2], fo[3], gg["do_clean"],
                                  gg["do_noisy"], self.M, out=gr, workspace=wsb, impl=self.impl, passes=passes,
                                  window=w.window, single_pass=self.fused)

    def kernel_names(self):
        # two-pass backward: dK/dV pass, then dQ pass; fused backward: one kernel for both (launched by the DKDV
        # pass bit together with the zero-fill of the fp32 dQ accumulators and their conversion; the DQ bit is a no-op)
        return ["fwd", "bwd_dsum", "bwd_fused" if self.fused else "bwd_dkdv", "bwd_dq"]

    def timed_steps(self, K, warmup, barrier, sampler=None):
        """W warm-up steps, then K timed steps with events between the kernels of a step.  Returns the total time of
        the K steps (ms, device clock), the per-step times and the mean time per kernel."""
        binding = self.binding
        for _ in range(warmup):
            self.run_fwd()
            self.run_bwd()
        torch.cuda.synchronize()
        if binding.bdlm_get_device_status() != 0:
            raise RuntimeError("device-side wait timed out during warm-up")
        names = self.kernel_names()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(K)]
        if sampler is not None:
            sampler.start()
            time.sleep(0.25)
        barrier()
        e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_start.record()
        for i in range(K):
            ev[i][0].record()
            self.run_fwd()
            ev[i][1].record()
            self.run_bwd(passes=binding.PASS_DSUM)
            ev[i][2].record()
            self.run_bwd(passes=binding.PASS_DKDV)
            ev[i][3].record()
            self.run_bwd(passes=binding.PASS_DQ)
            ev[i][4].record()
        e_stop.record()
        barrier()
        ms_total = e_start.elapsed_time(e_stop)
        clocks = sampler.stop() if sampler is not None else None
        if binding.bdlm_get_device_status() != 0:
            raise RuntimeError("device-side wait timed out during the timed region")
        per_step = [ev[i][0].elapsed_time(ev[i][len(names)]) for i in range(K)]
        per_kernel = {n: float(np.mean([ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(K)])) for j, n in enumerate(names)}
        return ms_total, per_step, per_kernel, clocks


def clock_normalised(ms, clocks):
    """ms x median SM MHz = clock cycles per step in units of 10^9: runs on power-capped boxes whose clocks settle at
    different frequencies are compared on this figure."""
    if not clocks or not clocks.get("sm_mhz"):
        return None
    return ms * clocks["sm_mhz"] * 1e-6


def fractions(tflops, peaks):
    return {"frac_burst": tflops / peaks["bf16_tflops"], "frac_sustained": tflops / peaks["bf16_tflops_sustained"],
            "frac_nominal_2250": tflops / 2250.0}


def sharded_forward_leg(run, peaks, steps, warmup):
    """The CSBP rank-local emulation as its configuration states it: the forward as one partial per contiguous
    clean-K/V shard (include_noisy_diag = 0) plus the noisy-diagonal partial (empty clean range), combined by
    bdlm_lse_merge (Eq. csbp-lse-merge) -- one merge call per query stream.  Timed with events: the partial
    launches, the two merges, and the whole."""
    w, binding = run.w, run.binding
    g, M, S = run.g, run.M, w.kv_shards
    step = w.L // S
    part_out = [(run.like(g["q_clean"]), run.lse_like(g["q_clean"]), run.like(g["q_noisy"]), run.lse_like(g["q_noisy"]))
                for _ in range(S)]
    diag_out = (None, None, run.like(g["q_noisy"]), run.lse_like(g["q_noisy"]))
    merged = (run.like(g["q_clean"]), run.lse_like(g["q_clean"]), run.like(g["q_noisy"]), run.lse_like(g["q_noisy"]))

    def partials():
        for s in range(S):
            run.run_fwd(fo=part_out[s], kv_range=(s * step, (s + 1) * step), include_noisy_diag=False)
        binding.bdlm_attn_fwd(None, g["k_clean"], g["v_clean"], g["q_noisy"], g["k_noisy"], g["v_noisy"], M,
                              out=diag_out, kv_range=(0, 0), impl=run.impl)

    def merges():
        binding.bdlm_lse_merge([p[0] for p in part_out], [p[1] for p in part_out], out=(merged[0], merged[1]))
        binding.bdlm_lse_merge([p[2] for p in part_out] + [diag_out[2]], [p[3] for p in part_out] + [diag_out[3]],
                               out=(merged[2], merged[3]))

    for _ in range(warmup):
        partials()
        merges()
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for i in range(steps):
        ev[i][0].record()
        partials()
        ev[i][1].record()
        merges()
        ev[i][2].record()
    torch.cuda.synchronize()
    if binding.bdlm_get_device_status() != 0:
        raise RuntimeError("device-side wait timed out in the sharded forward")
    ms_part = [ev[i][0].elapsed_time(ev[i][1]) for i in range(steps)]
    ms_merge = [ev[i][1].elapsed_time(ev[i][2]) for i in range(steps)]
    # bytes the two merges must move: every partial's O (bf16) and LSE (fp32) in, the merged O and LSE out
    o_bytes = w.batch * w.L * w.H * w.d * 2
    l_bytes = w.batch * w.H * w.L * 4
    merge_bytes = (S + 1) * (o_bytes + l_bytes) + (S + 2) * (o_bytes + l_bytes)
    f_fwd, _ = w.flops()
    ms_m = float(np.mean(ms_merge))
    ms_all = float(np.mean(ms_part)) + ms_m
    # agreement with the unsharded forward of the same inputs (already in run.fwd_out from the timed steps)
    diff = {"o_clean": float((merged[0].float() - run.fwd_out[0].float()).abs().max()),
            "lse_clean": float((merged[1] - run.fwd_out[1]).abs().max()),
            "o_noisy": float((merged[2].float() - run.fwd_out[2].float()).abs().max()),
            "lse_noisy": float((merged[3] - run.fwd_out[3]).abs().max())}
    return {"shards": S, "partials": f"{S} clean-K/V shard partials (both query streams) + 1 noisy-diagonal partial",
            "steps": steps, "ms_partials": float(np.mean(ms_part)), "ms_merge": ms_m, "ms_total": ms_all,
            "ms_total_min": float(np.min(np.add(ms_part, ms_merge))), "ms_total_median": float(np.median(np.add(ms_part, ms_merge))),
            "fwd_tflops": f_fwd / (ms_all * 1e-3) / 1e12,
            "merge": {"calls": 2, "n_partials": [S, S + 1], "algorithmic_bytes": merge_bytes,
                      "achieved_gbs": merge_bytes / (ms_m * 1e-3) / 1e9, "peak_gbs": peaks["hbm_gbs"],
                      "frac": merge_bytes / (ms_m * 1e-3) / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"],
                      "ms_min": float(np.min(ms_merge)), "ms_median": float(np.median(ms_merge))},
            "max_abs_diff_vs_unsharded_forward": diff}


def linear_ce_leg(binding, peaks, steps, warmup, name="lce_8k"):
    """The loss head after the last layer (token-chunked linear cross-entropy) on the Llama-3-8B-shaped workload:
    forward (projection with the log-sum-exp in the GEMM's epilogue) and backward (logits again + dz, dH, dW), timed
    separately with events.  Counted FLOPs: 2 T D V forward, 4 T D V backward (the recomputed logits are not counted)."""
    w = synth.LCE_WORKLOADS[name]
    g = synth.make_lce_inputs(w, "cuda")
    pf = binding.make_lce_params(w.T, w.D, w.V)
    ws_f = torch.empty(binding.bdlm_linear_ce_workspace_bytes(pf, binding.LCE_WS_FWD), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(binding.bdlm_linear_ce_workspace_bytes(pf, binding.LCE_WS_BWD), dtype=torch.uint8, device="cuda")
    out_f = (torch.empty(1, dtype=torch.float32, device="cuda"), torch.empty(w.T, dtype=torch.float32, device="cuda"),
             torch.empty(w.T, dtype=torch.float32, device="cuda"))
    out_b = (torch.empty_like(g["h"]), torch.empty_like(g["w"]))

    def fwd():
        binding.bdlm_linear_ce_fwd(g["h"], g["w"], g["labels"], g["weight"], out=out_f, workspace=ws_f)

    def bwd():
        binding.bdlm_linear_ce_bwd(g["h"], g["w"], g["labels"], out_f[2], g["weight"], out=out_b, workspace=ws_b)

    for _ in range(warmup):
        fwd()
        bwd()
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for i in range(steps):
        ev[i][0].record()
        fwd()
        ev[i][1].record()
        bwd()
        ev[i][2].record()
    torch.cuda.synchronize()
    if binding.bdlm_get_device_status() != 0:
        raise RuntimeError("device-side wait timed out in the linear cross-entropy leg")
    ms_f = [ev[i][0].elapsed_time(ev[i][1]) for i in range(steps)]
    ms_b = [ev[i][1].elapsed_time(ev[i][2]) for i in range(steps)]
    f_fwd, f_bwd = w.flops()
    tf_f = f_fwd / (float(np.mean(ms_f)) * 1e-3) / 1e12
    tf_b = f_bwd / (float(np.mean(ms_b)) * 1e-3) / 1e12
    tf_b_exec = 1.5 * tf_b
    out = {"workload": w.name, "T": w.T, "D": w.D, "V": w.V, "steps": steps, "warmup": warmup, "dtype": "bf16",
           "loss": float(out_f[0]),
           "fwd": {"ms": float(np.mean(ms_f)), "ms_min": float(np.min(ms_f)), "ms_median": float(np.median(ms_f)),
                   "tflops": tf_f, "roofline": dict(bound="tensor", achieved=tf_f, unit=UNIT, **fractions(tf_f, peaks))},
           "bwd": {"ms": float(np.mean(ms_b)), "ms_min": float(np.min(ms_b)), "ms_median": float(np.median(ms_b)),
                   "tflops_counted": tf_b, "tflops_executed": tf_b_exec,
                   "roofline": dict(bound="tensor", achieved=tf_b_exec, unit=UNIT,
                                    note="executed FLOPs (three products of 2 T D V each per chunk)", **fractions(tf_b_exec, peaks))},
           "logits_bytes_never_written": w.T * w.V * 2}
    del g, ws_f, ws_b, out_f, out_b
    torch.cuda.empty_cache()
    return out


def other_config_line(name, binding, peaks, impl, fused, steps, warmup, local):
    """One more workload on the same GPU, timed like the headline: value, per-kernel times, clocks."""
    w = synth.WORKLOADS[name]
    run = LayerRun(w, binding, 0, impl, fused)
    sampler = ClockSampler(physical_gpu_index(local))
    ms_total, per_step, per_kernel, clocks = run.timed_steps(steps, warmup, torch.cuda.synchronize, sampler)
    f_fwd, f_bwd = w.flops()
    ms_step = ms_total / steps
    tf = (f_fwd + f_bwd) / (ms_step * 1e-3) / 1e12
    out = {"workload": name, "L": w.L, "block_size": w.block_size, "steps": steps, "warmup": warmup,
           "value": tf, "unit": UNIT, "ms_per_step": ms_step, "ms_per_step_min": float(np.min(per_step)),
           "ms_per_step_median": float(np.median(per_step)), "per_kernel_ms": per_kernel, "clocks": clocks}
    out.update(fractions(tf, peaks))
    out["gclk_per_step"] = clock_normalised(ms_step, clocks)
    if w.kv_shards > 1:
        out["sharded_fwd"] = sharded_forward_leg(run, peaks, steps, warmup)
    del run
    torch.cuda.empty_cache()
    return out


def run_ours(args, w):
    from paper_2609_19242_b200 import binding
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    impl = args.kernel_impl
    fused = args.bwd == "fused"
    run = LayerRun(w, binding, rank, impl, fused)
    g, fwd_out, grads, ws = run.g, run.fwd_out, run.grads, run.ws
    like = run.like

    # ---- timed region: K steps, device time, events between the kernels of a step -------------
    K = args.steps
    names = run.kernel_names()
    sampler = ClockSampler(physical_gpu_index(local)) if rank == 0 else None
    ms_total, per_step, per_kernel_ms, clocks = run.timed_steps(K, args.warmup, barrier, sampler)
    ms_total = max_over_ranks(ms_total, "cuda", world)

    f_fwd, f_bwd = w.flops()
    ms_step = ms_total / K
    value = aggregate_tflops(f_fwd + f_bwd, ms_step, world)

    # ---- end to end through the public call with HOST buffers (pinned), copies inside ---------
    e2e = None
    if rank == 0 or world > 1:
        host_in = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in g.items()
                   if v is not None}
        host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in fwd_out + grads if t is not None]
        h2d = sum(t.numel() * t.element_size() for t in host_in.values())
        d2h = sum(t.numel() * t.element_size() for t in host_out)

        # Three streams and two sets of device buffers: the copies of step k+1 (host to device) and of step
        # k-1 (device to host) run under the kernels of step k.  Every step still copies all of its inputs in
        # and all of its results out inside the timed region; pipeline fill and drain are part of it too.
        g2 = {k_: like(v) for k_, v in g.items()}
        fo2, gr2, ws2 = run.make_buffers(g2)
        sets = [{"g": g, "fwd": fwd_out, "grads": grads, "ws": ws}, {"g": g2, "fwd": fo2, "grads": gr2, "ws": ws2}]
        s_comp = torch.cuda.current_stream()
        s_h2d, s_d2h = torch.cuda.Stream(), torch.cuda.Stream()

        def e2e_run(n):
            comp_done, d2h_done = [], []
            for k in range(n):
                st = sets[k & 1]
                with torch.cuda.stream(s_h2d):
                    if k >= 2:
                        s_h2d.wait_event(comp_done[k - 2])      # the set's inputs were last read by step k-2
                    for k_, v in host_in.items():
                        st["g"][k_].copy_(v, non_blocking=True)
                    h2d_done = torch.cuda.Event()
                    h2d_done.record(s_h2d)
                s_comp.wait_event(h2d_done)
                if k >= 2:
                    s_comp.wait_event(d2h_done[k - 2])          # the set's outputs have been read out
                run.run_fwd(st["g"], st["fwd"])
                run.run_bwd(st["g"], st["fwd"], st["grads"], st["ws"])
                ev_c = torch.cuda.Event()
                ev_c.record(s_comp)
                comp_done.append(ev_c)
                with torch.cuda.stream(s_d2h):
                    s_d2h.wait_event(ev_c)
                    for dst, src in zip(host_out, [t for t in st["fwd"] + st["grads"] if t is not None]):
                        dst.copy_(src, non_blocking=True)
                    ev_d = torch.cuda.Event()
                    ev_d.record(s_d2h)
                d2h_done.append(ev_d)
            s_comp.wait_event(d2h_done[-1])

        e2e_run(2)
        barrier()
        n_e2e = max(1, min(K, 40))   # as many steps as the device-timed region (pipeline fill and drain are inside)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        e2e_run(n_e2e)
        b.record()
        barrier()
        ms_e2e = a.elapsed_time(b) / n_e2e
        ms_e2e = max_over_ranks(ms_e2e, "cuda", world)
        e2e = {"value": aggregate_tflops(f_fwd + f_bwd, ms_e2e, world), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
               "steps": n_e2e, "overlap": "copies of neighbouring steps run under the kernels (3 streams, 2 buffer sets)"}
        del host_in, host_out, sets, g2, fo2, gr2, ws2

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (tensor-bound: algorithmic FLOPs / device time) -------
    # The counted backward is 5 GEMMs per pair (S, dP, dV, dK, dQ = 10d FLOPs).  The dK/dV pass owns
    # four of them (8d); the dQ pass owns dQ (2d) -- its recomputation of S and dP is not counted.
    # The fused kernel owns all five.
    algo_flops = {"fwd": f_fwd, "bwd_dkdv": f_bwd * 0.8, "bwd_dq": 0.0 if fused else f_bwd * 0.2, "bwd_dsum": 0.0,
                  "bwd_fused": f_bwd}
    dom = max((n for n in names if n != "bwd_dsum"), key=lambda n: per_kernel_ms[n])
    peak = peaks["bf16_tflops_sustained"] if ms_step * K > 1000.0 else peaks["bf16_tflops"]
    achieved = algo_flops[dom] / (per_kernel_ms[dom] * 1e-3) / 1e12
    digest = kernel_source_digest()
    cap = NCU_TRAFFIC.get((w.name, dom))
    traffic = cap["bytes"] if cap is not None and cap["kernel_source"] == digest else None
    if cap is None:
        traffic_note = TRAFFIC_NOTE + "; this workload has no capture"
    elif traffic is None:
        traffic_note = TRAFFIC_NOTE + "; the capture on record predates the current kernel source, so none is reported"
    else:
        traffic_note = TRAFFIC_NOTE
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "peak_source": peaks["source"] +
                (" sustained (timed region longer than 1 s)" if peak == peaks["bf16_tflops_sustained"] else " burst"),
                "traffic": traffic, "traffic_note": traffic_note, "kernel_source": digest,
                "per_kernel_ms": per_kernel_ms,
                "per_kernel_tflops": {n: (algo_flops[n] / (per_kernel_ms[n] * 1e-3) / 1e12) for n in names}}
    roofline.update(fractions(achieved, peaks))

    # ---- the other single-GPU configurations the target is stated on, and the paper-range block sizes ------
    others = None
    if world == 1 and args.other_configs and w.name == "32k":
        del run, g, fwd_out, grads, ws
        torch.cuda.empty_cache()
        others = {}
        for name, st_, wu_ in (("csbp128k", 3, 3), ("256k", 3, 3), ("32k_m512", 5, 3), ("32k_m1024", 5, 3), ("8k", 10, 3)):
            others[name] = other_config_line(name, binding, peaks, impl, fused, st_, wu_, local)
        others["linear_ce"] = linear_ce_leg(binding, peaks, 5, 3)

    # ---- CPU baseline: the oracle on a bounded sample, on this machine's host cores ---------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        inp = cpu_inputs_for_oracle(w)
        if args.oracle_rows > 0:
            oracle_sample(w, inp, 8, seed=99)
            rows = args.oracle_rows
            t, f = oracle_sample(w, inp, rows, seed=0)
        else:
            rows, t, f = timed_oracle_sample(w, inp, 20.0, w.L)
        cpu = {"value": f / t / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{rows} sampled query rows per stream of (batch 0, head 0), fwd+bwd, fp64, {t:.1f} s"}

    pct = fractions(value / world, peaks)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_min": float(np.min(per_step)), "ms_per_step_median": float(np.median(per_step)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "H": w.H, "H_kv": w.H_kv, "d": w.d, "L": w.L,
                       "block_size": w.block_size, "window": w.window, "n_blocks": w.n_blocks, "rope_theta": w.rope_theta, "parallelism": "replicas only",
                       "l2": "inputs larger than L2 (q/k/v/dO of one step exceed 126 MB)",
                       "kernel_impl": {0: "auto", 1: "portable", 2: "tcgen05"}[impl],
                       "backward": "fused (one kernel; dQ through fp32 add-reductions)" if fused else "two-pass (dK/dV, then dQ)"},
            "pct_of_bf16_peak": {"measured_burst": 100 * pct["frac_burst"], "measured_sustained": 100 * pct["frac_sustained"],
                                 "nominal_2250": 100 * pct["frac_nominal_2250"], "source": peaks["source"]},
            "clocks": clocks, "gclk_per_step": clock_normalised(ms_step, clocks), "e2e": e2e, "gpu_launches": (6 if fused else 5) * K, "roofline": roofline, "cpu_baseline": cpu,
            "other_configs": others}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="32k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--kernel-impl", type=int, default=0, help="0 auto, 1 portable mma.sync, 2 tcgen05")
    ap.add_argument("--oracle-rows", type=int, default=0, help="rows per stream in the oracle sample; 0 = size it for ~15 s")
    ap.add_argument("--bwd", default="fused", choices=["fused", "two_pass"],
                    help="backward: one fused kernel (dQ through fp32 add-reductions) or the bitwise reproducible two-pass path")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--linear-ce-only", action="store_true", help="run only the linear cross-entropy leg and print its JSON")
    ap.add_argument("--lce-workload", default="lce_8k", choices=sorted(synth.LCE_WORKLOADS))
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="skip the csbp128k / 256k / block-size legs that the default 32k run appends")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
        if args.linear_ce_only:
            from paper_2609_19242_b200 import binding
            torch.cuda.set_device(0)
            print(json.dumps({"linear_ce": linear_ce_leg(binding, load_peaks(), args.steps, args.warmup, args.lce_workload)}), flush=True)
            return
        run_ours(args, w)


if __name__ == "__main__":
    main()
