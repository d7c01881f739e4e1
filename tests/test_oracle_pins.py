"""Pins of the CPU oracle against facts that do not come from the oracle itself:
torch's own silu / matmul / softmax / autograd, closed forms, brute-force sorting, invariants and
central finite differences.  A dropped term, a wrong sign, a transposed operand or a wrong index in
oracle/moe_oracle.py fails at least one of these."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import moe_oracle as orc
from paper_2608_00916_b200 import synth


def _bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def _t64(bits):
    return torch.from_numpy(synth.bf16_bits_to_f64(bits))


def small_problem(T=12, d=10, E=6, k=3, f=7, seed=3, x_std=1.0, w_std=0.5, bias=True):
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=x_std, w_std=w_std, threads=1)
    if bias:
        rng = np.random.default_rng(seed)
        inp["b_r"] = (0.3 * rng.standard_normal(E)).astype(np.float32)
        # re-guard with the bias: regenerate until no violation (tiny sizes: brute force)
        for s in range(seed, seed + 50):
            cand = synth.make_inputs(shape, s, x_std=x_std, w_std=w_std, threads=1)
            l = synth._guard_logits(cand["x"], cand["W_r"], inp["b_r"])
            if not synth._gap_violations(l, k).any():
                cand["b_r"] = inp["b_r"]
                return cand
        raise RuntimeError("no guarded instance")
    return inp


def run_fw(inp, k, **kw):
    return orc.forward(inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"], k, b_r=inp["b_r"], **kw)


def run_bw(fw, inp, d_aux):
    return orc.backward(fw, inp["dy"], d_aux, inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"])


# ---------------------------------------------------------------------------------- forward pins
def test_single_expert_is_dense_swiglu_mlp():
    """E = 1, k = 1: gate is exactly 1 and y is a dense SwiGLU MLP (torch's silu and matmul)."""
    inp = small_problem(T=9, d=8, E=1, k=1, f=5, bias=False)
    fw = run_fw(inp, 1)
    x, Wg, Wu, Wd = _t64(inp["x"]), _t64(inp["W_gate"][0]), _t64(inp["W_up"][0]), _t64(inp["W_down"][0])
    ref = (F.silu(x @ Wg) * (x @ Wu)) @ Wd
    assert np.array_equal(fw["gates"], np.ones((9, 1)))
    assert np.array_equal(fw["idx"], np.zeros((9, 1), dtype=np.int32))
    np.testing.assert_allclose(fw["y"], ref.numpy(), rtol=1e-12, atol=1e-14)
    assert fw["aux"] == pytest.approx(1.0, abs=1e-12)


def test_identical_experts_equal_dense_mlp_for_any_routing():
    """All experts share one weight set: gates sum to 1, so y is the dense MLP and the summed expert
    weight gradients are the dense MLP's weight gradients (torch autograd)."""
    inp = small_problem(T=16, d=8, E=5, k=2, f=6, bias=True)
    for n in ("W_gate", "W_up", "W_down"):
        inp[n] = np.repeat(inp[n][:1], 5, axis=0)
    fw = run_fw(inp, 2)
    x = _t64(inp["x"]).requires_grad_(True)
    Wg, Wu, Wd = (_t64(inp[n][0]).requires_grad_(True) for n in ("W_gate", "W_up", "W_down"))
    y = (F.silu(x @ Wg) * (x @ Wu)) @ Wd
    np.testing.assert_allclose(fw["y"], y.detach().numpy(), rtol=1e-11, atol=1e-13)
    (y * _t64(inp["dy"])).sum().backward()
    bw = run_bw(fw, inp, 0.0)
    np.testing.assert_allclose(bw["dW_gate"].sum(0), Wg.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(bw["dW_up"].sum(0), Wu.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(bw["dW_down"].sum(0), Wd.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_k_equals_E_is_dense_mixture():
    """k = E: every expert is selected, gates are the full softmax, y = sum_e p_e FFN_e(x) by plain loops."""
    inp = small_problem(T=7, d=6, E=4, k=4, f=5, bias=True)
    fw = run_fw(inp, 4)
    x, Wr = _t64(inp["x"]), _t64(inp["W_r"])
    p = torch.softmax(x @ Wr + torch.from_numpy(inp["b_r"]).double(), dim=1)
    y = torch.zeros(7, 6, dtype=torch.float64)
    for t in range(7):
        for e in range(4):
            h = F.silu(x[t] @ _t64(inp["W_gate"][e])) * (x[t] @ _t64(inp["W_up"][e]))
            y[t] += p[t, e] * (h @ _t64(inp["W_down"][e]))
    np.testing.assert_allclose(fw["y"], y.numpy(), rtol=1e-11, atol=1e-13)
    # gates in pick order are the sorted probabilities
    np.testing.assert_allclose(fw["gates"], -np.sort(-p.numpy(), axis=1), rtol=1e-12)


def test_all_ties_closed_form():
    """W_r = 0: every logit ties, so idx = (0..k-1), gates = 1/k and aux = 1 exactly."""
    inp = small_problem(T=10, d=8, E=6, k=3, f=4, bias=False)
    inp["W_r"] = np.zeros_like(inp["W_r"])
    fw = run_fw(inp, 3)
    assert np.array_equal(fw["idx"], np.tile(np.arange(3, dtype=np.int32), (10, 1)))
    np.testing.assert_allclose(fw["gates"], 1.0 / 3.0, rtol=1e-15)
    assert fw["aux"] == pytest.approx(1.0, abs=1e-14)
    assert fw["counts"].tolist() == [10, 10, 10, 0, 0, 0]


def test_selection_against_brute_force_with_ties():
    """Hand-made logits with many equal values: selection equals sorting by (-logit, index)."""
    rng = np.random.default_rng(0)
    T, E, k = 40, 9, 4
    l = rng.integers(-2, 3, size=(T, E)).astype(np.float64)  # few distinct values -> many ties
    idx = orc.select_topk(l, k)
    for t in range(T):
        want = sorted(range(E), key=lambda e: (-l[t, e], e))[:k]
        assert idx[t].tolist() == want
    # the golden fixture spells one such case out by hand
    import json, os
    with open(os.path.join(os.path.dirname(__file__), "golden", "routing_ties.json")) as fh:
        gold = json.load(fh)
    got = orc.route_only(None, None, gold["k"], gold["E"], logits_in=np.array(gold["logits"]))
    assert got["idx"].tolist() == gold["idx"]
    assert got["counts"].tolist() == gold["counts"]
    assert got["perm"].tolist() == gold["perm"]
    np.testing.assert_allclose(got["gates"], np.array(gold["gates"]), rtol=1e-12)
    assert got["aux"] == pytest.approx(gold["aux"], rel=1e-12)


def test_softmax_topk_renorm_equals_softmax_over_selected():
    inp = small_problem(T=20, d=10, E=8, k=3, f=4)
    fw = run_fw(inp, 3)
    sel = np.take_along_axis(fw["logits"], fw["idx"].astype(np.int64), axis=1)
    want = torch.softmax(torch.from_numpy(sel), dim=1).numpy()
    np.testing.assert_allclose(fw["gates"], want, rtol=1e-12)
    np.testing.assert_allclose(fw["p"], torch.softmax(torch.from_numpy(fw["logits"]), dim=1).numpy(), rtol=1e-12)
    assert (fw["gates"] > 0).all()
    np.testing.assert_allclose(fw["gates"].sum(1), 1.0, rtol=1e-14)
    # pick order: descending logit
    assert (np.diff(sel, axis=1) < 0).all()


def test_routing_invariants_and_permutation_identity():
    inp = small_problem(T=33, d=10, E=7, k=3, f=4)
    fw = run_fw(inp, 3)
    T, k, E = 33, 3, 7
    assert fw["counts"].sum() == T * k
    for t in range(T):
        assert len(set(fw["idx"][t].tolist())) == k and fw["idx"][t].min() >= 0 and fw["idx"][t].max() < E
    perm, inv = fw["perm"], fw["inv"]
    assert sorted(perm.tolist()) == list(range(T * k))
    assert np.array_equal(inv[perm], np.arange(T * k))
    x = synth.bf16_bits_to_f64(inp["x"])
    np.testing.assert_array_equal(fw["xp"], x[perm // k])
    # unpermute(permute(x)) restores every (token, slot) copy
    np.testing.assert_array_equal(fw["xp"][inv].reshape(T, k, -1), np.repeat(x[:, None, :], k, axis=1))
    # rows of one expert: that expert, tokens strictly increasing
    for e in range(E):
        seg = perm[fw["offsets"][e]:fw["offsets"][e + 1]]
        assert (fw["idx"].reshape(-1)[seg] == e).all()
        assert (np.diff(seg // k) > 0).all()
    assert fw["offsets"][-1] == T * k and np.array_equal(np.diff(fw["offsets"]), fw["counts"])


def test_expert_relabelling_and_token_permutation():
    inp = small_problem(T=14, d=8, E=5, k=2, f=6)
    fw = run_fw(inp, 2)
    bw = run_bw(fw, inp, 0.2)
    rng = np.random.default_rng(5)
    pe = rng.permutation(5)
    inp2 = dict(inp)
    inp2["W_r"] = inp["W_r"][:, pe]
    inp2["b_r"] = inp["b_r"][pe]
    for n in ("W_gate", "W_up", "W_down"):
        inp2[n] = inp[n][pe]
    fw2 = run_fw(inp2, 2)
    bw2 = run_bw(fw2, inp2, 0.2)
    np.testing.assert_allclose(fw2["y"], fw["y"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(bw2["dx"], bw["dx"], rtol=1e-11, atol=1e-14)
    assert fw2["aux"] == pytest.approx(fw["aux"], rel=1e-13)
    np.testing.assert_allclose(bw2["dW_gate"], bw["dW_gate"][pe], rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(bw2["dW_r"], bw["dW_r"][:, pe], rtol=1e-11, atol=1e-14)
    pt = rng.permutation(14)
    inp3 = dict(inp)
    inp3["x"], inp3["dy"] = inp["x"][pt], inp["dy"][pt]
    fw3 = run_fw(inp3, 2)
    np.testing.assert_allclose(fw3["y"], fw["y"][pt], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(run_bw(fw3, inp3, 0.2)["dx"], bw["dx"][pt], rtol=1e-11, atol=1e-14)


def test_aux_normalisation():
    inp = small_problem(T=50, d=10, E=6, k=2, f=4)
    fw = run_fw(inp, 2)
    f_e = fw["counts"] / (50 * 2)
    P_e = fw["p"].mean(0)
    assert f_e.sum() == pytest.approx(1.0) and P_e.sum() == pytest.approx(1.0)
    assert fw["aux"] == pytest.approx(6 * float(np.dot(f_e, P_e)), rel=1e-13)


# ---------------------------------------------------------------------------------- backward pins
def torch_dense_mask_layer(inp, k, idx_fixed):
    """The layer written a different way: every expert runs on every token and a 0/1 mask keeps the
    selected ones; gates come from a masked softmax.  Gradients come from torch autograd."""
    x = _t64(inp["x"]).requires_grad_(True)
    Wr = _t64(inp["W_r"]).requires_grad_(True)
    b = torch.from_numpy(inp["b_r"]).double().requires_grad_(True)
    Wg = _t64(inp["W_gate"]).requires_grad_(True)
    Wu = _t64(inp["W_up"]).requires_grad_(True)
    Wd = _t64(inp["W_down"]).requires_grad_(True)
    T, E = x.shape[0], Wr.shape[1]
    l = x @ Wr + b
    mask = torch.zeros(T, E, dtype=torch.float64)
    mask.scatter_(1, torch.from_numpy(idx_fixed.astype(np.int64)), 1.0)
    p = torch.softmax(l, dim=1)
    gate = p * mask / (p * mask).sum(1, keepdim=True)  # [T,E], zero outside the selection
    H = F.silu(torch.einsum("td,edf->etf", x, Wg)) * torch.einsum("td,edf->etf", x, Wu)
    O = torch.einsum("etf,efd->etd", H, Wd)
    y = torch.einsum("te,etd->td", gate, O)
    counts = mask.sum(0)
    aux = E * ((counts / (T * k)) * p.mean(0)).sum()
    return y, aux, dict(x=x, W_r=Wr, b_r=b, W_gate=Wg, W_up=Wu, W_down=Wd)


@pytest.mark.parametrize("d_aux", [0.0, 0.37])
def test_backward_against_torch_autograd(d_aux):
    inp = small_problem(T=12, d=10, E=6, k=3, f=7)
    fw = run_fw(inp, 3)
    bw = run_bw(fw, inp, d_aux)
    y, aux, leaves = torch_dense_mask_layer(inp, 3, fw["idx"])
    np.testing.assert_allclose(fw["y"], y.detach().numpy(), rtol=1e-11, atol=1e-14)
    assert fw["aux"] == pytest.approx(float(aux.detach()), rel=1e-12)
    ((y * _t64(inp["dy"])).sum() + d_aux * aux).backward()
    for name, key in (("x", "dx"), ("W_r", "dW_r"), ("b_r", "db_r"), ("W_gate", "dW_gate"), ("W_up", "dW_up"),
                      ("W_down", "dW_down")):
        want = leaves[name].grad.numpy()
        np.testing.assert_allclose(bw[key], want, rtol=1e-9, atol=1e-12 * max(1.0, np.abs(want).max()), err_msg=key)


def test_backward_finite_differences():
    """Central differences in float64 on the loss <y,dy> + d_aux*aux with routing frozen by the gap guard."""
    inp = small_problem(T=6, d=8, E=4, k=2, f=6)
    d_aux, h = 0.37, 1e-6
    k = 2

    def to64(i):
        return {n: synth.bf16_bits_to_f64(i[n]) for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}

    v = to64(inp)
    b = inp["b_r"].astype(np.float64)

    def loss(vv, bb):
        # float64 evaluation of the definition through the oracle's own step functions on widened inputs
        l = orc.router_logits(vv["x"], vv["W_r"], bb)
        p = orc.softmax_rows(l)
        idx = orc.select_topk(l, k)
        assert np.array_equal(idx, fw["idx"]), "perturbation changed the routing"
        g = orc.gates_from(p, idx)
        y = np.zeros_like(vv["x"])
        for t in range(vv["x"].shape[0]):
            for j in range(k):
                e = idx[t, j]
                _, _, _, o = orc.expert_ffn(vv["x"][t:t + 1], vv["W_gate"][e], vv["W_up"][e], vv["W_down"][e])
                y[t] += g[t, j] * o[0]
        counts = np.bincount(idx.ravel(), minlength=l.shape[1])
        return float((y * vv["dy"]).sum()) + d_aux * orc.aux_loss(p, counts, k)

    fw = run_fw(inp, k)
    bw = run_bw(fw, inp, d_aux)
    assert loss(v, b) == pytest.approx(orc.loss_value(fw, inp["dy"], d_aux), rel=1e-12)
    rng = np.random.default_rng(11)
    for name, key in (("x", "dx"), ("W_r", "dW_r"), ("W_gate", "dW_gate"), ("W_up", "dW_up"), ("W_down", "dW_down")):
        flat_n = v[name].size
        for pos in rng.choice(flat_n, size=min(25, flat_n), replace=False):
            vp = {n: a.copy() for n, a in v.items()}
            vm = {n: a.copy() for n, a in v.items()}
            vp[name].reshape(-1)[pos] += h
            vm[name].reshape(-1)[pos] -= h
            num = (loss(vp, b) - loss(vm, b)) / (2 * h)
            ana = bw[key].reshape(-1)[pos]
            assert num == pytest.approx(ana, rel=2e-5, abs=2e-8), (name, pos)
    for e in range(4):
        bp, bm = b.copy(), b.copy()
        bp[e] += h
        bm[e] -= h
        assert (loss(v, bp) - loss(v, bm)) / (2 * h) == pytest.approx(bw["db_r"][e], rel=2e-5, abs=2e-8)


def test_backward_invariants():
    inp = small_problem(T=20, d=8, E=6, k=2, f=5)
    # make expert 4 unreachable: very negative bias
    inp["b_r"] = inp["b_r"].copy()
    inp["b_r"][4] = -50.0
    fw = run_fw(inp, 2)
    assert fw["counts"][4] == 0
    bw = run_bw(fw, inp, 0.25)
    np.testing.assert_allclose(bw["dl"].sum(1), 0.0, atol=1e-14)  # softmax shift invariance
    assert not bw["dW_gate"][4].any() and not bw["dW_up"][4].any() and not bw["dW_down"][4].any()
    bw0 = run_bw(fw, inp, 0.0)
    mask = np.zeros_like(bw0["dl"], dtype=bool)
    np.put_along_axis(mask, fw["idx"].astype(np.int64), True, axis=1)
    assert not bw0["dl"][~mask].any()


def test_sampled_helpers_agree_with_full_pass():
    inp = small_problem(T=18, d=8, E=5, k=2, f=6)
    fw = run_fw(inp, 2)
    bw = run_bw(fw, inp, 0.1)
    rt = orc.route_only(inp["x"], inp["W_r"], 2, 5, b_r=inp["b_r"])
    assert np.array_equal(rt["idx"], fw["idx"]) and np.array_equal(rt["perm"], fw["perm"])
    for t in (0, 7, 17):
        np.testing.assert_allclose(orc.token_rows(t, rt, inp["x"], inp["W_gate"], inp["W_up"], inp["W_down"]),
                                   fw["y"][t], rtol=1e-12, atol=1e-15)
    for t in (0, 7, 17):
        dx_t, dl_t = orc.token_backward(t, rt, inp["dy"], 0.1, inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"],
                                        inp["W_down"])
        np.testing.assert_allclose(dx_t, bw["dx"][t], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(dl_t, bw["dl"][t], rtol=1e-10, atol=1e-14)
    for e in range(5):
        a, b_, c = orc.expert_grads(e, rt, inp["dy"], inp["x"], inp["W_gate"], inp["W_up"], inp["W_down"])
        np.testing.assert_allclose(a, bw["dW_gate"][e], rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(b_, bw["dW_up"][e], rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(c, bw["dW_down"][e], rtol=1e-11, atol=1e-14)


def test_fp32_mode_close_to_fp64():
    inp = synth.make_config("tiny")
    k = 2
    f64 = run_fw(inp, k)
    f32 = run_fw(inp, k, dtype=np.float32)
    assert np.array_equal(f64["idx"], f32["idx"]) and np.array_equal(f64["perm"], f32["perm"])
    rel = np.linalg.norm(f32["y"] - f64["y"]) / np.linalg.norm(f64["y"])
    assert rel < 1e-5


# ---------------------------------------------------------------------------------- expert LoRA pins
def _lora_problem():
    inp = small_problem(T=10, d=8, E=4, k=2, f=6)
    lo = synth.make_lora(synth.MoEShape(10, 8, 4, 2, 6), 9, rank=3, std=0.4, threads=1)
    return inp, lo, 0.7


def _lora_run(inp, lo, s, k=2):
    args = (inp["W_gate"], inp["W_up"], inp["W_down"], lo["A1"], lo["B1_gate"], lo["B1_up"], lo["A2"], lo["B2"], s)
    fw = orc.lora_forward(inp["x"], inp["W_r"], *args, k, b_r=inp["b_r"])
    bw = orc.lora_backward(fw, inp["dy"], 0.2, inp["x"], inp["W_r"], *args)
    return fw, bw


def test_lora_with_zero_adapters_is_the_base_layer():
    inp, lo, s = _lora_problem()
    lo0 = dict(lo)
    lo0["B1_gate"], lo0["B1_up"], lo0["B2"] = (np.zeros_like(lo[n]) for n in ("B1_gate", "B1_up", "B2"))
    fw, bw = _lora_run(inp, lo0, s)
    base = run_fw(inp, 2)
    np.testing.assert_array_equal(fw["y"], base["y"])
    np.testing.assert_array_equal(bw["dx"], run_bw(base, inp, 0.2)["dx"])
    assert not bw["dA1"].any() and not bw["dA2"].any()  # dA = s dW B^T vanishes with B = 0


def test_lora_gradients_against_torch_autograd():
    """The adapted layer written with torch ops on the adapter parameters themselves (low-rank path computed as
    (x A) B, never forming W + s A B) and differentiated by autograd."""
    inp, lo, s = _lora_problem()
    fw, bw = _lora_run(inp, lo, s)
    k = 2
    x = _t64(inp["x"]).requires_grad_(True)
    Wr = _t64(inp["W_r"]); b = torch.from_numpy(inp["b_r"]).double()
    Wg, Wu, Wd = _t64(inp["W_gate"]), _t64(inp["W_up"]), _t64(inp["W_down"])
    P = {n: _t64(lo[n]).requires_grad_(True) for n in ("A1", "B1_gate", "B1_up", "A2", "B2")}
    T, E = x.shape[0], Wr.shape[1]
    l = x @ Wr + b
    mask = torch.zeros(T, E, dtype=torch.float64)
    mask.scatter_(1, torch.from_numpy(fw["idx"].astype(np.int64)), 1.0)
    p = torch.softmax(l, dim=1)
    gate = p * mask / (p * mask).sum(1, keepdim=True)
    y = torch.zeros_like(x)
    for e in range(E):
        u = x @ P["A1"][e]
        hg = x @ Wg[e] + s * (u @ P["B1_gate"][e])
        hu = x @ Wu[e] + s * (u @ P["B1_up"][e])
        a = F.silu(hg) * hu
        o = a @ Wd[e] + s * ((a @ P["A2"][e]) @ P["B2"][e])
        y = y + gate[:, e:e + 1] * o
    np.testing.assert_allclose(fw["y"], y.detach().numpy(), rtol=1e-10, atol=1e-13)
    aux = E * ((mask.sum(0) / (T * k)) * p.mean(0)).sum()
    ((y * _t64(inp["dy"])).sum() + 0.2 * aux).backward()
    np.testing.assert_allclose(bw["dx"], x.grad.numpy(), rtol=1e-9, atol=1e-12)
    for n, key in (("A1", "dA1"), ("B1_gate", "dB1_gate"), ("B1_up", "dB1_up"), ("A2", "dA2"), ("B2", "dB2")):
        want = P[n].grad.numpy()
        np.testing.assert_allclose(bw[key], want, rtol=1e-9, atol=1e-12 * max(1.0, np.abs(want).max()), err_msg=key)
