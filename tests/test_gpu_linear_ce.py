"""GPU-vs-oracle parity of the token-chunked linear cross-entropy, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import linear_ce_oracle as lce
from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import LceWorkload

pytestmark = pytest.mark.gpu

# bf16 inputs, fp32 accumulation and fp32 softmax statistics; dz rounded to bf16 before the gradient products
TOL_LSE = 1e-3        # max |lse - oracle|, as for the attention layer's LSE
TOL_NLL = 2e-3        # max |nll - oracle| (lse and the target logit each carry fp32 accumulation error)
TOL_LOSS_REL = 1e-4   # |loss - oracle| / |oracle|
TOL_GRAD = 2e-2       # relative L2 of dH and dW


def _rel(got, ref):
    return float(np.linalg.norm((got - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300))


def _check(w, token_chunk=0, weighted=True, grad_loss=1.0):
    inp = synth.make_lce_inputs(w, "cpu")
    g = {k: v.cuda() for k, v in inp.items()}
    tw = g["weight"] if weighted else None
    loss, nll, lse = binding.bdlm_linear_ce_fwd(g["h"], g["w"], g["labels"], tw)
    dh, dw = binding.bdlm_linear_ce_bwd(g["h"], g["w"], g["labels"], lse, tw, grad_loss=grad_loss, token_chunk=token_chunk)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    h64, w64 = synth.to_f64(inp["h"]), synth.to_f64(inp["w"])
    y = inp["labels"].numpy()
    wt = inp["weight"].double().numpy() if weighted else None
    ref_loss, ref_nll, ref_lse = lce.linear_ce_forward(h64, w64, y, wt, token_chunk=97)
    ref_dh, ref_dw = lce.linear_ce_backward(h64, w64, y, wt, grad_loss=grad_loss, token_chunk=97)
    assert np.abs(synth.to_f64(lse) - ref_lse).max() <= TOL_LSE
    assert np.abs(synth.to_f64(nll) - ref_nll).max() <= TOL_NLL
    assert abs(float(loss) - ref_loss) <= TOL_LOSS_REL * abs(ref_loss)
    got_dh, got_dw = synth.to_f64(dh), synth.to_f64(dw)
    assert np.isfinite(got_dh).all() and np.isfinite(got_dw).all()
    assert _rel(got_dh, ref_dh) <= TOL_GRAD, _rel(got_dh, ref_dh)
    assert _rel(got_dw, ref_dw) <= TOL_GRAD, _rel(got_dw, ref_dw)
    ign = y < 0
    if ign.any():
        assert np.abs(got_dh[ign]).max() == 0.0 and np.abs(synth.to_f64(nll)[ign]).max() == 0.0
    return loss, nll, lse, dh, dw


@pytest.mark.parametrize("w", [
    LceWorkload("one_tile", 128, 64, 256),
    LceWorkload("tiny", 200, 64, 1000),                       # ragged token tile and ragged vocabulary tile
    LceWorkload("several_tiles", 400, 192, 2568),             # several vocabulary runs (> 8 tiles of 256), K not a multiple of 64
    LceWorkload("wide", 300, 520, 776, logit_std=4.0),        # D beyond one 256-column N tile in the gradient products
    LceWorkload("one_token", 1, 64, 512),
], ids=lambda w: w.name)
def test_matches_oracle(w):
    _check(w)


def test_token_chunks_accumulate_dw_in_fp32_and_agree_with_one_chunk():
    w = LceWorkload("chunks", 600, 128, 1544)
    one = _check(w, token_chunk=0)
    three = _check(w, token_chunk=256, grad_loss=1.0)          # 256 + 256 + 88 tokens
    many = _check(w, token_chunk=128)                          # five chunks, the last one ragged
    assert torch.equal(one[3], three[3]) and torch.equal(one[3], many[3])   # dH rows do not depend on the chunking
    for other in (three, many):
        assert _rel(synth.to_f64(other[4]), synth.to_f64(one[4])) <= 4e-3   # dW: other fp32 summation order, one bf16 rounding


def test_unweighted_and_scaled_gradient():
    _check(LceWorkload("plain", 256, 64, 512), weighted=False, grad_loss=-0.37)


def test_results_are_bitwise_reproducible():
    w = LceWorkload("repro", 384, 128, 2048)
    inp = {k: v.cuda() for k, v in synth.make_lce_inputs(w, "cpu").items()}
    runs = []
    for _ in range(2):
        loss, nll, lse = binding.bdlm_linear_ce_fwd(inp["h"], inp["w"], inp["labels"], inp["weight"])
        dh, dw = binding.bdlm_linear_ce_bwd(inp["h"], inp["w"], inp["labels"], lse, inp["weight"], token_chunk=128)
        runs.append([t.clone() for t in (loss, nll, lse, dh, dw)])
    torch.cuda.synchronize()
    for a, b in zip(*runs):
        assert torch.equal(a, b)


def test_full_size_sampled_tokens():
    """The benchmark's size (8192 tokens, D = 4096, V = 128256): lse and nll of 64 sampled tokens against the oracle;
    dH rows of those tokens against the oracle (a token's dH depends on that token only); dW through linearity: a
    second backward whose weights are zero outside the sample is compared with the oracle's sum over the sample."""
    w = synth.LCE_WORKLOADS["lce_8k"]
    g = synth.make_lce_inputs(w, "cuda")
    loss, nll, lse = binding.bdlm_linear_ce_fwd(g["h"], g["w"], g["labels"], g["weight"])
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, 127, 128, 4095, 4096, w.T - 1], rng.choice(w.T, size=58, replace=False)]))
    rt = torch.from_numpy(rows).cuda()
    w_sp = torch.zeros_like(g["weight"])
    w_sp[rt] = g["weight"][rt]
    dh, _ = binding.bdlm_linear_ce_bwd(g["h"], g["w"], g["labels"], lse, g["weight"], token_chunk=2048)
    _, dw_sp = binding.bdlm_linear_ce_bwd(g["h"], g["w"], g["labels"], lse, w_sp, token_chunk=4096)
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    W64 = synth.to_f64(g["w"])
    h_rows = synth.to_f64(g["h"][rt])
    y_rows = g["labels"][rt].cpu().numpy()
    wt_rows = g["weight"][rt].double().cpu().numpy()
    ref_nll, ref_lse = lce.linear_ce_rows(h_rows, W64, y_rows)
    assert np.abs(synth.to_f64(lse[rt]) - ref_lse).max() <= TOL_LSE
    assert np.abs(synth.to_f64(nll[rt]) - ref_nll).max() <= TOL_NLL
    ref_dh, ref_dw = lce.linear_ce_backward(h_rows, W64, y_rows, wt_rows, token_chunk=16)
    assert _rel(synth.to_f64(dh[rt]), ref_dh) <= TOL_GRAD
    assert _rel(synth.to_f64(dw_sp), ref_dw) <= TOL_GRAD
    # the scalar loss against the per-token values the kernel itself wrote (the sum is the only new arithmetic here)
    want = float((g["weight"].double() * nll.double()).sum())
    assert abs(float(loss) - want) <= 1e-5 * abs(want)


def test_all_positions_ignored_gives_zero_loss_and_zero_gradients():
    w = LceWorkload("all_ignored", 130, 64, 520)
    inp = {k: v.cuda() for k, v in synth.make_lce_inputs(w, "cpu").items()}
    labels = torch.full_like(inp["labels"], -1)
    loss, nll, lse = binding.bdlm_linear_ce_fwd(inp["h"], inp["w"], labels, None)
    dh, dw = binding.bdlm_linear_ce_bwd(inp["h"], inp["w"], labels, lse, None)
    torch.cuda.synchronize()
    assert float(loss) == 0.0 and float(nll.abs().max()) == 0.0
    assert float(dh.float().abs().max()) == 0.0 and float(dw.float().abs().max()) == 0.0
    ref = lce.linear_ce_forward(synth.to_f64(inp["h"]), synth.to_f64(inp["w"]), labels.cpu().numpy())
    assert np.abs(synth.to_f64(lse) - ref[2]).max() <= TOL_LSE
