"""Helpers for the GPU-vs-oracle parity tests: run the CUDA path through the binding, run the
fp64 oracle on the same bf16 bits, compare within the stated tolerances."""
import numpy as np
import torch

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import binding, synth

# Tolerances of the parity bar (bf16 inputs, fp32 accumulation, bf16 P and dS operands).
TOL_O = 1e-2          # max |dO| elementwise on outputs
TOL_LSE = 1e-3        # max |dLSE|
TOL_GRAD = 2e-2       # relative L2 error of each of dQ, dK, dV per stream
TOL_DQ_ROW = 5e-2     # sampled-row checks: every single dQ row (Eq. correctness-query-gradient is per row, so one wrong
                      # row must not hide in the pooled figure above) must satisfy
                      #     |dQ_i - ref_i| <= TOL_DQ_ROW * |ref_i| + 2^-8 * scale * |dO_i| * |O_i| * max_j |k_j|.
                      # The second term is the error the kernels' arithmetic allows: they form dS = P * (dP - D) with
                      # D_i = dO_i . O_i taken from the bf16 output, so D carries up to 2^-9 |dO_i| |O_i| of rounding
                      # (twice that allowed here), which enters dQ_i as scale * dD_i * sum_j P_ij k_j.  Rows where dP - D
                      # cancels (row 1 with its two keys) lose several per cent that way; for a typical late row the term
                      # is a few per cent of |ref_i|, so a wrong row (error of the order of the row itself) still fails.


def dq_row_excess(got, ref, o_ref, do_rows, scale, k_max_norm):
    """Worst ratio of a dQ row's error to its allowance (see TOL_DQ_ROW); must be <= 1.  Rows are [n, d]."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    if ref.shape[0] == 0:
        return 0.0
    allow = TOL_DQ_ROW * np.linalg.norm(ref, axis=1) + \
        2.0 ** -8 * scale * np.linalg.norm(do_rows, axis=1) * np.linalg.norm(o_ref, axis=1) * k_max_norm
    return float((np.linalg.norm(got - ref, axis=1) / np.maximum(allow, 1e-300)).max())


NAMES6 = ["q_clean", "k_clean", "v_clean", "q_noisy", "k_noisy", "v_noisy"]


def rel_l2(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    if den == 0:
        return float(np.linalg.norm(got.ravel()))
    return float(np.linalg.norm((got - ref).ravel()) / den)


def to_cuda(inp):
    return {k: v.cuda().contiguous() for k, v in inp.items()}


def f64(inp):
    return {k: synth.to_f64(v) for k, v in inp.items()}


def gpu_fwd(g, M, **kw):
    return binding.bdlm_attn_fwd(*[g[n] for n in NAMES6], M, **kw)


def gpu_bwd(g, fwd_out, M, do_clean=None, do_noisy=None, **kw):
    """Backward through the binding.  Unless a test says otherwise this is the two-pass path (single_pass=False):
    the fused kernel and the library's automatic choice are asked for by name where they are under test."""
    kw.setdefault("single_pass", False)
    o_c, l_c, o_n, l_n = fwd_out
    return binding.bdlm_attn_bwd(*[g[n] for n in NAMES6], o_c, l_c, o_n, l_n,
                                 g["do_clean"] if do_clean is None else do_clean,
                                 g["do_noisy"] if do_noisy is None else do_noisy, M, **kw)


def check_full(w, impl, mode=0, check_bwd=True, inp=None, single_pass=False):
    """Whole-tensor parity against the full oracle (small shapes)."""
    inp = synth.make_inputs(w, "cpu") if inp is None else inp
    g = to_cuda(inp)
    x = f64(inp)
    M = w.block_size
    out = gpu_fwd(g, M, clean_mask_mode=mode, impl=impl, window=w.window)
    torch.cuda.synchronize()
    ref = orc.attn_forward(*[x[n] for n in NAMES6], M, clean_mask_mode=mode, window=w.window)
    for got, want, name in zip(out, ref, ["o_clean", "lse_clean", "o_noisy", "lse_noisy"]):
        gotn = synth.to_f64(got)
        assert np.isfinite(gotn).all(), name
        err = np.abs(gotn - want).max()
        assert err <= (TOL_LSE if "lse" in name else TOL_O), (name, err)
    if not check_bwd:
        return
    grads = gpu_bwd(g, out, M, clean_mask_mode=mode, impl=impl, window=w.window, single_pass=single_pass)
    torch.cuda.synchronize()
    gref = orc.attn_backward(*[x[n] for n in NAMES6], x["do_clean"], x["do_noisy"], M, clean_mask_mode=mode,
                             window=w.window)
    for got, want, name in zip(grads, gref, ["dq_clean", "dk_clean", "dv_clean", "dq_noisy", "dk_noisy", "dv_noisy"]):
        gotn = synth.to_f64(got)
        assert np.isfinite(gotn).all(), name
        err = rel_l2(gotn, want)
        assert err <= TOL_GRAD, (name, err)
    assert binding.bdlm_get_device_status() == 0


def check_sampled(w, impl, n_rows=256, g=None, fwd_out=None, check_bwd=True, report=None, single_pass=False, mode=0):
    """Sampled-row parity for sizes the full oracle cannot do: per (batch, head, stream)
    `n_rows` stratified query rows are recomputed by the oracle.  O and LSE come from the
    full forward.  dQ at the sampled rows comes from the full backward (a row's dQ depends on
    that row's dO only).  dK/dV are linear in dO, so a second backward with dO zeroed outside
    the sampled rows is compared, for every key, with the oracle's sum over those rows.
    `single_pass` selects the backward path; a tuple such as (False, True) checks several paths
    against one evaluation of the oracle (the worst figure over the paths is reported)."""
    M = w.block_size
    variants = tuple(single_pass) if isinstance(single_pass, (tuple, list)) else (single_pass,)
    if g is None:
        g = synth.make_inputs(w, "cuda")
    if fwd_out is None:
        fwd_out = gpu_fwd(g, M, impl=impl, window=w.window, clean_mask_mode=mode)
    torch.cuda.synchronize()
    G = w.H // w.H_kv
    rows_of = {}
    for b in range(w.batch):
        for h in range(w.H):
            for s in (0, 1):
                rows_of[(b, h, s)] = synth.sample_rows(w, n_rows, seed=1000 * b + 10 * h + s)
    grads, grads_sp = {}, {}
    if check_bwd:
        do_sp = [torch.zeros_like(g["do_clean"]), torch.zeros_like(g["do_noisy"])]
        for (b, h, s), rows in rows_of.items():
            r = torch.from_numpy(rows).cuda()
            src = g["do_clean"] if s == 0 else g["do_noisy"]
            do_sp[s][b, r, h] = src[b, r, h]
        for sp in variants:
            grads[sp] = [t.clone() for t in gpu_bwd(g, fwd_out, M, impl=impl, window=w.window, single_pass=sp,
                                                    clean_mask_mode=mode)]
            grads_sp[sp] = [t.clone() for t in gpu_bwd(g, fwd_out, M, do_clean=do_sp[0], do_noisy=do_sp[1], impl=impl,
                                                       window=w.window, single_pass=sp, clean_mask_mode=mode)]
        torch.cuda.synchronize()
        assert binding.bdlm_get_device_status() == 0
    worst = {"o": 0.0, "lse": 0.0, "dq": 0.0, "dq_row": 0.0, "dk": 0.0, "dv": 0.0}
    qn = ["q_clean", "q_noisy"]
    don = ["do_clean", "do_noisy"]
    for b in range(w.batch):
        for hk in range(w.H_kv):
            kv = {n: synth.to_f64(g[n][b, :, hk]) for n in ("k_clean", "v_clean", "k_noisy", "v_noisy")}
            acc = {n: np.zeros((w.L, w.d)) for n in ("dk_clean", "dv_clean", "dk_noisy", "dv_noisy")}
            k_max = float(max(np.linalg.norm(kv["k_clean"], axis=1).max(), np.linalg.norm(kv["k_noisy"], axis=1).max()))
            dq_num = {sp: [0.0, 0.0] for sp in variants}
            dq_den = [0.0, 0.0]
            for h in range(hk * G, (hk + 1) * G):
                for s in (0, 1):
                    rows = rows_of[(b, h, s)]
                    rt = torch.from_numpy(rows).cuda()
                    q_rows = synth.to_f64(g[qn[s]][b, rt, h])
                    do_rows = synth.to_f64(g[don[s]][b, rt, h]) if check_bwd else None
                    ref = orc.attn_rows(s, rows, q_rows, kv["k_clean"], kv["v_clean"], kv["k_noisy"],
                                        kv["v_noisy"], M, do_rows=do_rows, window=w.window, clean_mask_mode=mode)
                    o_got = synth.to_f64(fwd_out[2 * s][b, rt, h])
                    l_got = synth.to_f64(fwd_out[2 * s + 1][b, h, rt])
                    worst["o"] = max(worst["o"], float(np.abs(o_got - ref["o"]).max()))
                    worst["lse"] = max(worst["lse"], float(np.abs(l_got - ref["lse"]).max()))
                    if check_bwd:
                        for sp in variants:
                            dq_got = synth.to_f64(grads[sp][3 * s][b, rt, h])
                            dq_num[sp][s] += float(((dq_got - ref["dq"]) ** 2).sum())
                            worst["dq_row"] = max(worst["dq_row"], dq_row_excess(dq_got, ref["dq"], ref["o"], do_rows,
                                                                                 1.0 / np.sqrt(w.d), k_max))
                        dq_den[s] += float((ref["dq"] ** 2).sum())
                        for n in acc:
                            acc[n] += ref[n]
            if check_bwd:
                idx = {"dk_clean": 1, "dv_clean": 2, "dk_noisy": 4, "dv_noisy": 5}
                for sp in variants:
                    for s in (0, 1):
                        worst["dq"] = max(worst["dq"], (dq_num[sp][s] / max(dq_den[s], 1e-300)) ** 0.5)
                    for n, want in acc.items():
                        got = synth.to_f64(grads_sp[sp][idx[n]][b, :, hk])
                        assert np.isfinite(got).all(), n
                        worst[n[:2]] = max(worst[n[:2]], rel_l2(got, want))
    if report is not None:
        report.update(worst)
    assert worst["o"] <= TOL_O, worst
    assert worst["lse"] <= TOL_LSE, worst
    if check_bwd:
        assert worst["dq"] <= TOL_GRAD and worst["dk"] <= TOL_GRAD and worst["dv"] <= TOL_GRAD, worst
        assert worst["dq_row"] <= 1.0, worst
    return worst


def check_sampled_packed(w, impl, n_rows=256, single_pass=False):
    """Sampled-row parity of a packed (DFlash2-style) workload: O, LSE and dQ at sampled packed rows of
    every (batch, head); dK/dV of the clean and the packed noisy keys through a second backward whose dO is
    zero outside the sampled rows (dK/dV are linear in dO)."""
    M = w.block_size
    g = synth.make_inputs(w, "cuda")
    pfx = g["block_prefix"]
    anchors = w.anchors()
    args = [g[n] for n in NAMES6]
    out = binding.bdlm_attn_fwd_packed(*args, M, block_prefix=pfx, impl=impl)
    grads = binding.bdlm_attn_bwd_packed(*args, out[0], out[1], out[2], out[3], None, g["do_noisy"], M,
                                         block_prefix=pfx, impl=impl, single_pass=single_pass)
    Ln = w.n_blocks * M
    G = w.H // w.H_kv
    rng = np.random.default_rng(17)
    rows_of = {}
    do_sp = torch.zeros_like(g["do_noisy"])
    for b in range(w.batch):
        for h in range(w.H):
            fixed = [0, M - 1, M, Ln - M, Ln - 1, 127, 128]
            rest = rng.choice(Ln, size=n_rows, replace=False)
            rows = np.unique(np.concatenate([np.asarray(fixed), rest]))[:n_rows]
            rows_of[(b, h)] = rows
            r = torch.from_numpy(rows).cuda()
            do_sp[b, r, h] = g["do_noisy"][b, r, h]
    grads_sp = binding.bdlm_attn_bwd_packed(*args, out[0], out[1], out[2], out[3], None, do_sp, M,
                                            block_prefix=pfx, impl=impl, single_pass=single_pass)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    worst = {"o": 0.0, "lse": 0.0, "dq": 0.0, "dq_row": 0.0, "dk": 0.0, "dv": 0.0}
    for b in range(w.batch):
        for hk in range(w.H_kv):
            kv = {n: synth.to_f64(g[n][b, :, hk]) for n in ("k_clean", "v_clean", "k_noisy", "v_noisy")}
            acc = {"dk_clean": np.zeros((w.L, w.d)), "dv_clean": np.zeros((w.L, w.d)),
                   "dk_noisy": np.zeros((Ln, w.d)), "dv_noisy": np.zeros((Ln, w.d))}
            k_max = float(max(np.linalg.norm(kv["k_clean"], axis=1).max(), np.linalg.norm(kv["k_noisy"], axis=1).max()))
            num = den = 0.0
            for h in range(hk * G, (hk + 1) * G):
                rows = rows_of[(b, h)]
                rt = torch.from_numpy(rows).cuda()
                ref = orc.attn_rows_packed(1, rows, synth.to_f64(g["q_noisy"][b, rt, h]), kv["k_clean"], kv["v_clean"],
                                           kv["k_noisy"], kv["v_noisy"], M,
                                           do_rows=synth.to_f64(g["do_noisy"][b, rt, h]), block_prefix=anchors)
                worst["o"] = max(worst["o"], float(np.abs(synth.to_f64(out[2][b, rt, h]) - ref["o"]).max()))
                worst["lse"] = max(worst["lse"], float(np.abs(synth.to_f64(out[3][b, h, rt]) - ref["lse"]).max()))
                num += float(((synth.to_f64(grads[3][b, rt, h]) - ref["dq"]) ** 2).sum())
                worst["dq_row"] = max(worst["dq_row"], dq_row_excess(synth.to_f64(grads[3][b, rt, h]), ref["dq"], ref["o"],
                                                                     synth.to_f64(g["do_noisy"][b, rt, h]), 1.0 / np.sqrt(w.d), k_max))
                den += float((ref["dq"] ** 2).sum())
                for n in acc:
                    acc[n] += ref[n]
            worst["dq"] = max(worst["dq"], (num / max(den, 1e-300)) ** 0.5)
            idx = {"dk_clean": 1, "dv_clean": 2, "dk_noisy": 4, "dv_noisy": 5}
            for n, want in acc.items():
                got = synth.to_f64(grads_sp[idx[n]][b, :, hk])
                assert np.isfinite(got).all(), n
                worst[n[:2]] = max(worst[n[:2]], rel_l2(got, want))
    assert worst["o"] <= TOL_O and worst["lse"] <= TOL_LSE, worst
    assert worst["dq"] <= TOL_GRAD and worst["dk"] <= TOL_GRAD and worst["dv"] <= TOL_GRAD, worst
    assert worst["dq_row"] <= 1.0, worst
    return worst
