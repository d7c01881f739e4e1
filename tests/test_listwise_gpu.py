"""moe_listwise_loss on the GPU against the float64 oracle: loss and gradient for both kinds, odd group sizes, many rows,
no rows, and the argument checks."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import listwise_oracle as lw
from paper_2608_00916_b200 import binding

pytestmark = pytest.mark.gpu


EPS32 = 2.0 ** -23


def _tol(s, temp=1.0):
    """fp32 arithmetic on scores of magnitude S: s / temp - logsumexp carries an absolute rounding error of a few
    S eps, which is the relative error of every probability (each at most 1) and the absolute error of a row's loss."""
    return 8 * EPS32 * float(np.abs(s).max(initial=1.0)) / temp + 2e-6


def _draw(n, G, seed, scale):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n, G)) * scale).astype(np.float32), (rng.standard_normal((n, G)) * scale).astype(np.float32)


@pytest.mark.parametrize("n,G,scale", [(64, 8, 3.0), (1, 1, 1.0), (4097, 8, 10.0), (5, 33, 2.0), (3, 1000, 4.0), (40, 32, 30.0)])
def test_contrastive(n, G, scale):
    s, _ = _draw(n, G, 100 + n, scale)
    ref_loss, ref_grad = lw.contrastive(s)
    loss, grad = binding.listwise_loss(torch.from_numpy(s).cuda())
    assert float(loss.cpu()[0]) == pytest.approx(ref_loss, rel=2e-6, abs=_tol(s))
    assert np.abs(grad.cpu().numpy() - ref_grad).max() <= _tol(s) / n
    assert np.abs(grad.cpu().numpy().sum(axis=1)).max() <= G * _tol(s) / n


@pytest.mark.parametrize("n,G,ts,tt,scale", [(64, 8, 1.0, 1.0, 3.0), (64, 8, 2.0, 0.5, 3.0), (9, 17, 0.7, 3.0, 5.0),
                                              (2000, 8, 1.5, 1.5, 8.0), (2, 300, 1.0, 2.0, 2.0)])
def test_distill(n, G, ts, tt, scale):
    s, t = _draw(n, G, 200 + n, scale)
    ref_loss, ref_grad = lw.distill(s, t, ts, tt)
    loss, grad = binding.listwise_loss(torch.from_numpy(s).cuda(), torch.from_numpy(t).cuda(), ts, tt)
    tol = _tol(s, ts) + _tol(t, tt)
    assert float(loss.cpu()[0]) == pytest.approx(ref_loss, rel=2e-6, abs=tol * ts * ts)
    assert np.abs(grad.cpu().numpy() - ref_grad).max() <= tol * ts / n


def test_teacher_equal_to_student_and_certain_teacher():
    s, _ = _draw(16, 8, 7, 2.0)
    x = torch.from_numpy(s).cuda()
    loss, grad = binding.listwise_loss(x, (x + 4.0).contiguous(), 1.5, 1.5)
    assert abs(float(loss.cpu()[0])) <= 1e-5 and float(grad.abs().max().cpu()) <= 1e-6
    # a teacher that is certain of one passage has zero probabilities elsewhere: they contribute nothing, not NaN
    t = torch.full((4, 8), -1000.0, device="cuda")
    t[:, 3] = 1000.0
    loss, grad = binding.listwise_loss(torch.zeros(4, 8, device="cuda"), t, 1.0, 1.0)
    assert float(loss.cpu()[0]) == pytest.approx(np.log(8.0), rel=1e-5)
    assert torch.isfinite(grad).all()


def test_no_rows_repeatability_and_argument_checks():
    loss, grad = binding.listwise_loss(torch.empty(0, 8, device="cuda"))
    assert float(loss.cpu()[0]) == 0.0 and grad.numel() == 0
    s, t = _draw(777, 8, 9, 5.0)
    a = binding.listwise_loss(torch.from_numpy(s).cuda(), torch.from_numpy(t).cuda(), 2.0, 1.0)
    b = binding.listwise_loss(torch.from_numpy(s).cuda(), torch.from_numpy(t).cuda(), 2.0, 1.0)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    loss_only, none = binding.listwise_loss(torch.from_numpy(s).cuda(), want_grad=False)
    assert none is None and torch.isfinite(loss_only).all()
    lib = binding.load_library()
    x = torch.zeros(2, 8, device="cuda")
    out = torch.zeros(1, device="cuda")
    p = lambda v: C.c_void_p(v.data_ptr())
    bad = [(7, 2, 8, p(x), None, 1.0, 1.0, p(out)), (0, 2, 0, p(x), None, 1.0, 1.0, p(out)), (0, 2, 8, None, None, 1.0, 1.0, p(out)),
           (1, 2, 8, p(x), None, 1.0, 1.0, p(out)), (1, 2, 8, p(x), p(x), 0.0, 1.0, p(out)), (1, 2, 8, p(x), p(x), 1.0, -1.0, p(out)),
           (0, 2, 8, p(x), None, 1.0, 1.0, None), (0, -1, 8, p(x), None, 1.0, 1.0, p(out))]
    for kind, n, G, sc, te, ts, tt, lo in bad:
        assert lib.moe_listwise_loss(kind, n, G, sc, te, C.c_float(ts), C.c_float(tt), lo, None, None) == -1
