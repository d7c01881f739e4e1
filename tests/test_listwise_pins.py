"""Pins of the listwise-loss oracle (oracle/listwise_oracle.py) against what the mathematics and a library fix: torch's
cross_entropy / kl_div, closed forms, invariances and finite differences."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import listwise_oracle as lw


def _scores(n, G, seed, scale=3.0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, G)) * scale, rng.standard_normal((n, G)) * scale


@pytest.mark.parametrize("n,G", [(1, 2), (7, 8), (64, 8), (5, 33)])
def test_contrastive_against_torch_cross_entropy(n, G):
    s, _ = _scores(n, G, 10 + n)
    loss, grad = lw.contrastive(s)
    ts = torch.tensor(s, dtype=torch.float64, requires_grad=True)
    ref = F.cross_entropy(ts, torch.zeros(n, dtype=torch.long))
    ref.backward()
    assert loss == pytest.approx(float(ref.detach()), rel=1e-12)
    assert np.allclose(grad, ts.grad.numpy(), rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("n,G,ts_,tt_", [(3, 8, 1.0, 1.0), (64, 8, 2.0, 0.5), (9, 17, 0.7, 3.0)])
def test_distill_against_torch_kl_div(n, G, ts_, tt_):
    s, t = _scores(n, G, 20 + n)
    loss, grad = lw.distill(s, t, ts_, tt_)
    x = torch.tensor(s, dtype=torch.float64, requires_grad=True)
    student = F.log_softmax(x / ts_, dim=-1)
    teacher = F.softmax(torch.tensor(t, dtype=torch.float64) / tt_, dim=-1)
    ref = F.kl_div(student, teacher, reduction="batchmean") * ts_ ** 2
    ref.backward()
    assert loss == pytest.approx(float(ref.detach()), rel=1e-12)
    assert np.allclose(grad, x.grad.numpy(), rtol=1e-11, atol=1e-15)


def test_closed_forms():
    n, G = 6, 8
    loss, grad = lw.contrastive(np.full((n, G), 2.5))
    assert loss == pytest.approx(np.log(G), rel=1e-14)
    expect = np.full((n, G), 1.0 / G / n)
    expect[:, 0] -= 1.0 / n
    assert np.allclose(grad, expect, rtol=1e-13)
    # a single passage per query: nothing to rank
    assert lw.contrastive(np.array([[3.0], [-1.0]]))[0] == pytest.approx(0.0, abs=1e-15)
    # student equal to the teacher at equal temperatures: zero divergence, zero gradient
    s, _ = _scores(n, G, 31)
    loss, grad = lw.distill(s, s + 4.0, 1.5, 1.5)  # a shift of the teacher's rows does not change its distribution
    assert loss == pytest.approx(0.0, abs=1e-14) and np.abs(grad).max() < 1e-15
    # two passages, teacher certain of the first, student indifferent: KL = log 2
    loss, _ = lw.distill(np.zeros((1, 2)), np.array([[800.0, -800.0]]), 1.0, 1.0)
    assert loss == pytest.approx(np.log(2.0), rel=1e-13)
    # no queries
    assert lw.contrastive(np.zeros((0, 8)))[0] == 0.0 and lw.distill(np.zeros((0, 8)), np.zeros((0, 8)), 1.0, 1.0)[0] == 0.0


def test_invariances():
    s, t = _scores(11, 8, 41)
    shift = np.random.default_rng(5).standard_normal((11, 1)) * 10
    for f in (lambda a: lw.contrastive(a), lambda a: lw.distill(a, t, 2.0, 1.0)):
        l0, g0 = f(s)
        l1, g1 = f(s + shift)
        assert l1 == pytest.approx(l0, rel=1e-12)
        assert np.allclose(g0, g1, rtol=1e-9, atol=1e-14)
        assert np.abs(g0.sum(axis=1)).max() < 1e-15  # a row's gradient sums to zero
        assert l0 >= 0.0
    # the divergence is not symmetric, so swapping the roles must change the value
    assert lw.distill(s, t, 1.0, 1.0)[0] != pytest.approx(lw.distill(t, s, 1.0, 1.0)[0], rel=1e-3)


def test_gradients_by_central_differences():
    s, t = _scores(4, 5, 51, scale=1.0)
    h = 1e-6
    for f in (lambda a: lw.contrastive(a), lambda a: lw.distill(a, t, 1.7, 0.6)):
        _, g = f(s)
        num = np.zeros_like(s)
        for i in range(s.shape[0]):
            for j in range(s.shape[1]):
                a, b = s.copy(), s.copy()
                a[i, j] += h
                b[i, j] -= h
                num[i, j] = (f(a)[0] - f(b)[0]) / (2 * h)
        assert np.allclose(g, num, rtol=1e-6, atol=1e-9)
