"""Pins for the linear cross-entropy oracle (oracle/linear_ce_oracle.py): library cross-entropy and autograd in
fp64, a pure-Python brute force, central differences, closed forms and token-chunk invariance."""
import math

import numpy as np
import pytest
import torch

from oracle import linear_ce_oracle as lce


def _case(seed, T=13, D=5, V=11, ignore=(2, 7), weighted=True):
    rng = np.random.default_rng(seed)
    h = rng.standard_normal((T, D))
    W = rng.standard_normal((V, D)) * 0.8
    y = rng.integers(0, V, size=T)
    for i in ignore:
        if i < T:
            y[i] = -100
    w = rng.uniform(0.2, 3.0, size=T) if weighted else None
    return h, W, y, w


@pytest.mark.parametrize("weighted", [False, True])
def test_matches_torch_cross_entropy_and_autograd(weighted):
    h, W, y, w = _case(1, weighted=weighted)
    ht = torch.tensor(h, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    per = torch.nn.functional.cross_entropy(ht @ Wt.T, torch.tensor(y), ignore_index=-100, reduction="none")
    wt = torch.ones(len(y), dtype=torch.float64) if w is None else torch.tensor(w)
    loss_t = (wt * per).sum()
    (0.7 * loss_t).backward()
    loss, nll, lse = lce.linear_ce_forward(h, W, y, w)
    assert abs(loss - float(loss_t.detach())) < 1e-11
    assert np.allclose(nll, per.detach().numpy(), atol=1e-12)
    assert np.allclose(lse, torch.logsumexp(ht @ Wt.T, dim=1).detach().numpy(), atol=1e-12)
    dH, dW = lce.linear_ce_backward(h, W, y, w, grad_loss=0.7)
    assert np.allclose(dH, ht.grad.numpy(), atol=1e-12)
    assert np.allclose(dW, Wt.grad.numpy(), atol=1e-12)


def test_matches_pure_python_brute_force():
    h, W, y, w = _case(2, T=6, D=3, V=4, ignore=(1,))
    T, D = h.shape
    V = W.shape[0]
    loss, nll, lse = lce.linear_ce_forward(h, W, y, w)
    dH, dW = lce.linear_ce_backward(h, W, y, w, grad_loss=1.5)
    tot = 0.0
    dH_b = [[0.0] * D for _ in range(T)]
    dW_b = [[0.0] * D for _ in range(V)]
    for t in range(T):
        z = [sum(h[t][k] * W[v][k] for k in range(D)) for v in range(V)]
        s = math.log(sum(math.exp(x) for x in z))
        assert abs(s - lse[t]) < 1e-12
        if y[t] < 0:
            assert nll[t] == 0.0
            continue
        assert abs((s - z[y[t]]) - nll[t]) < 1e-12
        tot += w[t] * (s - z[y[t]])
        for v in range(V):
            dz = 1.5 * w[t] * (math.exp(z[v] - s) - (1.0 if v == y[t] else 0.0))
            for k in range(D):
                dH_b[t][k] += dz * W[v][k]
                dW_b[v][k] += dz * h[t][k]
    assert abs(tot - loss) < 1e-12
    assert np.allclose(dH, np.array(dH_b), atol=1e-12) and np.allclose(dW, np.array(dW_b), atol=1e-12)


def test_gradients_match_central_differences():
    h, W, y, w = _case(3)
    dH, dW = lce.linear_ce_backward(h, W, y, w)
    rng = np.random.default_rng(0)
    eps = 1e-6
    for arr, grad in ((h, dH), (W, dW)):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=10, replace=False):
            old = flat[idx]
            flat[idx] = old + eps
            up = lce.linear_ce_forward(h, W, y, w)[0]
            flat[idx] = old - eps
            dn = lce.linear_ce_forward(h, W, y, w)[0]
            flat[idx] = old
            assert abs((up - dn) / (2 * eps) - grad.reshape(-1)[idx]) < 1e-6


def test_uniform_logits_closed_form():
    """W = 0: every logit is 0, lse = ln V, nll = ln V, dz = w (1/V - onehot): dH = 0 and dW_v = sum_t dz_tv h_t."""
    T, D, V = 9, 4, 7
    rng = np.random.default_rng(4)
    h = rng.standard_normal((T, D))
    y = rng.integers(0, V, size=T)
    w = rng.uniform(0.5, 2.0, size=T)
    loss, nll, lse = lce.linear_ce_forward(h, np.zeros((V, D)), y, w)
    assert np.allclose(lse, math.log(V)) and np.allclose(nll, math.log(V))
    assert abs(loss - w.sum() * math.log(V)) < 1e-12
    dH, dW = lce.linear_ce_backward(h, np.zeros((V, D)), y, w)
    assert np.abs(dH).max() == 0.0
    want = np.zeros((V, D))
    for t in range(T):
        for v in range(V):
            want[v] += w[t] * (1.0 / V - (1.0 if v == y[t] else 0.0)) * h[t]
    assert np.allclose(dW, want, atol=1e-13)
    # a dominant target logit: the loss of that token goes to 0 and so does its gradient
    Wbig = np.zeros((V, D))
    Wbig[3] = 50.0 * h[0] / (h[0] @ h[0])
    _, nll2, _ = lce.linear_ce_forward(h[:1], Wbig, np.array([3]))
    assert nll2[0] < 1e-15 * 1e6


@pytest.mark.parametrize("chunk", [1, 4, 5, 13, 100])
def test_token_chunk_count_does_not_change_the_result(chunk):
    h, W, y, w = _case(5)
    a = lce.linear_ce_forward(h, W, y, w)
    b = lce.linear_ce_forward(h, W, y, w, token_chunk=chunk)
    assert abs(a[0] - b[0]) < 1e-12 and np.allclose(a[1], b[1], atol=1e-14) and np.allclose(a[2], b[2], atol=1e-14)
    ga = lce.linear_ce_backward(h, W, y, w, grad_loss=-2.0)
    gb = lce.linear_ce_backward(h, W, y, w, grad_loss=-2.0, token_chunk=chunk)
    assert np.allclose(ga[0], gb[0], atol=1e-13) and np.allclose(ga[1], gb[1], atol=1e-13)


def test_ignored_and_zero_weight_positions_contribute_nothing():
    h, W, y, w = _case(6)
    w2 = w.copy()
    w2[4] = 0.0
    y3 = y.copy()
    y3[4] = -1
    a = lce.linear_ce_forward(h, W, y, w2)
    b = lce.linear_ce_forward(h, W, y3, w)
    assert abs(a[0] - b[0]) < 1e-13
    ga, gb = lce.linear_ce_backward(h, W, y, w2), lce.linear_ce_backward(h, W, y3, w)
    assert np.allclose(ga[0], gb[0], atol=1e-14) and np.allclose(ga[1], gb[1], atol=1e-14)
    assert np.abs(ga[0][4]).max() == 0.0 and np.abs(ga[0][2]).max() == 0.0   # row 2 is ignored in _case
    nll_r, lse_r = lce.linear_ce_rows(h[[0, 5]], W, y[[0, 5]])
    assert np.allclose(nll_r, a[1][[0, 5]], atol=1e-14) and np.allclose(lse_r, a[2][[0, 5]], atol=1e-14)
