"""Parity of the CUDA layer (called through the C ABI) with the CPU oracle on the same seeded inputs.

Bars: routing indices, per-expert counts and the permutation are bit-exact; gates |d| <= 1e-5; logits
|d| <= 1e-5 max|l|; aux relative <= 1e-4; relative Frobenius error <= 1e-2 for y and every gradient (bf16
storage of the intermediates puts the expected error near 3e-3); weight-gradient slabs of experts that received
tokens <= 2e-2 each, and exactly zero for experts without tokens."""
import numpy as np
import pytest
import torch

from paper_2608_00916_b200 import synth
from gpu_util import ROW_TOL, Run, from_dev_bf16, oracle_run, rel_fro, rows_max_err
from paper_2608_00916_b200.binding import MoELayer, kernel_launches as binding_launches
from oracle import moe_oracle as orc

pytestmark = pytest.mark.gpu
TOL = 1e-2


def check_routing(fw, ofw):
    assert np.array_equal(fw["idx"].cpu().numpy(), ofw["idx"])
    assert np.array_equal(fw["counts"].cpu().numpy(), ofw["counts"])
    assert np.array_equal(fw["perm"].cpu().numpy(), ofw["perm"])
    assert np.abs(fw["gates"].cpu().numpy() - ofw["gates"]).max() <= 1e-5
    lg = fw["logits"].cpu().numpy()
    assert np.abs(lg - ofw["logits"]).max() <= 1e-5 * max(1.0, np.abs(ofw["logits"]).max())
    assert float(fw["aux"].cpu()[0]) == pytest.approx(ofw["aux"], rel=1e-4)


def check_all(r: Run, ofw, obw, d_aux, stages=True):
    fw = r.forward()
    check_routing(fw, ofw)
    d, f, k, E = r.d, r.f, r.k, r.E
    # the library folds the gate of a routed row into its saved activation: act and o are stored gate-scaled
    g_row = ofw["gates"].reshape(-1)[ofw["perm"]][:, None]
    if stages:
        for nm, w in (("xp", d), ("hg", f), ("hu", f), ("act", f), ("o", d)):
            got, pad = r.rows(nm, w)
            ref = ofw[nm] * g_row if nm in ("act", "o") else ofw[nm]
            assert rel_fro(got, ref) <= (0.0 if nm == "xp" else TOL), nm
            assert rows_max_err(got, ref) <= ROW_TOL, nm
            assert not pad.any(), f"pad rows of {nm} are not zero"
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL
    assert rows_max_err(from_dev_bf16(fw["y"]), ofw["y"]) <= ROW_TOL  # no single token row is wrong
    bw = r.backward(d_aux)
    if stages:
        assert rel_fro(r.layer.buffer("dg", torch.float32).cpu().numpy().reshape(-1, k), obw["dg"]) <= TOL
        # in backward the o buffer holds the gathered dy rows (d_o without its gate)
        dy_rows = synth.bf16_bits_to_f64(r.inp["dy"])[ofw["perm"] // k]
        for nm, w, ref in (("o", d, dy_rows), ("dhg", f, obw["dhg"]), ("dhu", f, obw["dhu"]), ("dxp", d, obw["dxp"])):
            got, pad = r.rows(nm, w)
            assert rel_fro(got, ref) <= (0.0 if nm == "o" else TOL), nm
            assert rows_max_err(got, ref) <= ROW_TOL, nm
            assert not pad.any(), f"pad rows of {nm} (backward) are not zero"
        assert rel_fro(r.layer.buffer("dl", torch.float32).cpu().numpy().reshape(-1, E), obw["dl"]) <= TOL
    for nm in ("dx", "dW_gate", "dW_up", "dW_down"):
        assert rel_fro(from_dev_bf16(bw[nm]), obw[nm]) <= TOL, nm
        assert rows_max_err(from_dev_bf16(bw[nm]), obw[nm]) <= ROW_TOL, nm
    assert rel_fro(bw["dW_r"].cpu().numpy(), obw["dW_r"]) <= TOL
    assert rows_max_err(bw["dW_r"].cpu().numpy(), obw["dW_r"]) <= ROW_TOL
    # dW_r against the float64 host contraction of x with the ORACLE's dl (not with the library's own dl)
    ref_dwr = synth.bf16_bits_to_f64(r.inp["x"]).T @ obw["dl"]
    assert rel_fro(bw["dW_r"].cpu().numpy(), ref_dwr) <= TOL
    assert rel_fro(bw["db_r"].cpu().numpy(), obw["db_r"]) <= TOL
    # per-expert slabs
    for nm in ("dW_gate", "dW_up", "dW_down"):
        g = from_dev_bf16(bw[nm])
        for e in range(E):
            if ofw["counts"][e] == 0:
                assert not g[e].any(), (nm, e)
            else:
                assert rel_fro(g[e], obw[nm][e]) <= 2e-2, (nm, e)
    return fw, bw


def test_tiny_config_stage_by_stage():
    inp = synth.make_config("tiny")
    ofw, obw = oracle_run(inp, 2, inp["d_aux"])
    check_all(Run(inp, 2), ofw, obw, inp["d_aux"])


@pytest.mark.parametrize("T,d,E,k,f,seed", [
    (1, 64, 4, 2, 64, 11),        # a single token
    (7, 128, 8, 3, 192, 12),      # fewer tokens than experts*k: several empty experts
    (255, 256, 8, 2, 320, 13),    # one short of a token tile; f not a multiple of 128 or 256
    (1000, 512, 16, 4, 384, 14),  # several row tiles per expert, ragged tails
    (333, 192, 5, 5, 320, 15),    # k = E: every expert takes every token; d not a multiple of 128
    (300, 128, 1, 1, 256, 16),    # E = 1, k = 1: dense SwiGLU MLP
    (2049, 256, 32, 8, 128, 17),  # more than 8 token tiles, k = 8
    (520, 320, 256, 6, 64, 18),   # the largest expert count
    (200, 128, 64, 32, 128, 19),  # the largest top_k
])
def test_odd_shapes(T, d, E, k, f, seed):
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    ofw, obw = oracle_run(inp, k, 0.05)
    check_all(Run(inp, k), ofw, obw, 0.05)


@pytest.mark.parametrize("flag", [1, 2, 16, 16 | 8])
@pytest.mark.parametrize("T,d,E,k,f,seed", [(1000, 512, 16, 4, 384, 14), (333, 192, 5, 5, 320, 15), (2049, 256, 32, 8, 128, 17),
                                            (3000, 256, 8, 2, 256, 21)])
def test_forced_tile_shapes(T, d, E, k, f, seed, flag):
    """Forcing CTA pairs (cta_group::2, 256-row tiles; flag 1), one-CTA tiles (flag 2) or the mixed schedule (complete
    pairs of row blocks on CTA pairs, leftover blocks on one-CTA tiles; flag 16, also with the router's gradient chain
    kept on the caller's stream, flag 8) for every expert GEMM gives the same results as the default per-GEMM
    choice.  The last shape has experts with one, an even and an odd number of row blocks."""
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    ofw, obw = oracle_run(inp, k, 0.05)
    check_all(Run(inp, k, flags=flag), ofw, obw, 0.05)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        E = int(rng.choice([1, 2, 3, 8, 12, 16, 24, 40, 64, 96, 128, 200, 256]))
        k = int(rng.integers(1, min(E, 9) + 1))
        d = 64 * int(rng.integers(1, 9))
        f = 64 * int(rng.integers(1, 9))
        T = int(rng.choice([1, 2, 31, 33, 127, 129, 500, 1023, 1500, 2600]))
        out.append((T, d, E, k, f, 1000 + i))
    return out


@pytest.mark.parametrize("T,d,E,k,f,seed", _random_shapes(24, 2024))
def test_random_shapes(T, d, E, k, f, seed):
    """A seeded sweep over odd combinations of sizes (every width a multiple of 64, expert counts with and without
    the tensor-core router path, token counts around tile boundaries): full stage-by-stage parity each time."""
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    if seed % 3 == 0:
        inp["b_r"] = (0.2 * np.random.default_rng(seed).standard_normal(E)).astype(np.float32)
        l = synth._guard_logits(inp["x"], inp["W_r"], inp["b_r"])
        keep = ~synth._gap_violations(l, k)
        if not keep.any():
            pytest.skip("no guarded token in this draw")
        inp["x"], inp["dy"] = inp["x"][keep], inp["dy"][keep]
    ofw, obw = oracle_run(inp, k, 0.03)
    check_all(Run(inp, k, flags=(0, 1, 2, 16)[seed % 4]), ofw, obw, 0.03)


@pytest.mark.parametrize("T,d,E,k,f", [(1, 64, 8, 2, 64), (47, 128, 256, 3, 64), (300, 192, 24, 4, 320), (1029, 256, 16, 8, 128)])
def test_no_write_outside_the_declared_buffers(T, d, E, k, f):
    """Canaries: the bytes after the workspace, the alignment gaps between its internal buffers and the bytes after
    every caller output keep their fill pattern through a forward + backward."""
    import ctypes as C
    from paper_2608_00916_b200.binding import MoELayer, _ptr, _check
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, 77)
    dev = {n: torch.from_numpy(inp[n].view(np.int16)).cuda().view(torch.bfloat16)
           for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
    layer = MoELayer(d, E, f, k)
    need = layer.workspace_bytes(T)
    PAD = 4096
    ws = torch.full((need + PAD,), 0xA5, dtype=torch.uint8, device="cuda")
    names = ["counts", "offsets", "pad_offsets", "logits", "idx", "gates", "inv", "row_gate", "xp", "hg", "hu", "act", "o",
             "dhg", "dhu", "dxp", "dxr", "dg", "dl", "status", "timers"]
    spans = sorted(layer.find(T, n) for n in names)

    def guarded(shape_, dtype):
        n = int(np.prod(shape_)) if len(shape_) else 1
        buf = torch.full((n * torch.empty((), dtype=dtype).element_size() + 256,), 0x5A, dtype=torch.uint8, device="cuda")
        return buf, buf[: buf.numel() - 256].view(dtype).view(*shape_) if n else buf[:0].view(dtype).view(*shape_)

    outs = {n: guarded(shp, dt) for n, shp, dt in (
        ("y", (T, d), torch.bfloat16), ("idx", (T, k), torch.int32), ("gates", (T, k), torch.float32),
        ("counts", (E,), torch.int32), ("perm", (T * k,), torch.int32), ("aux", (1,), torch.float32),
        ("dx", (T, d), torch.bfloat16), ("dW_r", (d, E), torch.float32), ("db_r", (E,), torch.float32),
        ("dW_gate", (E, d, f), torch.bfloat16), ("dW_up", (E, d, f), torch.bfloat16), ("dW_down", (E, f, d), torch.bfloat16))}
    o = {n: v[1] for n, v in outs.items()}
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    lib = layer.lib
    _check(lib, lib.moe_forward(layer.h, T, _ptr(dev["x"]), _ptr(dev["W_r"]), None, None, _ptr(dev["W_gate"]),
                                _ptr(dev["W_up"]), _ptr(dev["W_down"]), _ptr(o["y"]), _ptr(o["idx"]), _ptr(o["gates"]),
                                _ptr(o["counts"]), _ptr(o["perm"]), _ptr(o["aux"]), None, _ptr(ws), need, st), "fwd")
    _check(lib, lib.moe_backward(layer.h, T, _ptr(dev["dy"]), C.c_float(0.01), _ptr(dev["x"]), _ptr(dev["W_r"]),
                                 _ptr(dev["W_gate"]), _ptr(dev["W_up"]), _ptr(dev["W_down"]), _ptr(o["dx"]), _ptr(o["dW_r"]),
                                 _ptr(o["db_r"]), _ptr(o["dW_gate"]), _ptr(o["dW_up"]), _ptr(o["dW_down"]), _ptr(ws), need,
                                 st), "bwd")
    torch.cuda.synchronize()
    assert bool((ws[need:] == 0xA5).all()), "wrote past the workspace"
    for (off, n), (noff, _) in zip(spans, spans[1:]):
        gap = ws[off + n: noff]
        # only gaps that are pure alignment padding (< 256 bytes) are guaranteed to be nobody's buffer
        if 0 < gap.numel() < 256:
            assert bool((gap == 0xA5).all()), f"wrote into the padding after offset {off}+{n}"
    for n, (buf, _) in outs.items():
        assert bool((buf[-256:] == 0x5A).all()), f"wrote past {n}"


def test_skewed_small_with_bias_and_empty_experts():
    shape = synth.MoEShape(2048, 256, 32, 4, 256)
    inp = synth.make_inputs(shape, 7, x_std=1.0, skew=True)
    ofw, obw = oracle_run(inp, 4, 0.1)
    assert (ofw["counts"] == 0).sum() >= 3
    check_all(Run(inp, 4), ofw, obw, 0.1)


def test_exact_ties_through_logits_in():
    """Routing from caller-supplied logits with many exact ties must match the oracle bit for bit."""
    shape = synth.MoEShape(512, 128, 16, 4, 128)
    inp = synth.make_inputs(shape, 21, guard=False)
    rng = np.random.default_rng(3)
    logits = rng.integers(-2, 3, size=(512, 16)).astype(np.float32)
    logits[:64] = 0.0  # all-ties rows: idx must be 0..k-1
    ofw, obw = oracle_run(inp, 4, 0.0, logits_in=logits)
    r = Run(inp, 4, logits_in=logits)
    fw = r.forward()
    check_routing(fw, ofw)
    assert np.array_equal(fw["idx"].cpu().numpy()[:64], np.tile(np.arange(4, dtype=np.int32), (64, 1)))
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL


def test_all_ties_closed_form_on_gpu():
    """W_r = 0: idx = (0..k-1) for every token, gates 1/k, aux = 1 exactly."""
    shape = synth.MoEShape(300, 128, 8, 3, 128)
    inp = synth.make_inputs(shape, 22, guard=False)
    inp["W_r"] = np.zeros_like(inp["W_r"])
    r = Run(inp, 3)
    fw = r.forward()
    assert np.array_equal(fw["idx"].cpu().numpy(), np.tile(np.arange(3, dtype=np.int32), (300, 1)))
    np.testing.assert_allclose(fw["gates"].cpu().numpy(), 1.0 / 3.0, rtol=1e-6)
    assert float(fw["aux"].cpu()[0]) == pytest.approx(1.0, rel=1e-6)
    assert fw["counts"].cpu().numpy().tolist() == [300, 300, 300, 0, 0, 0, 0, 0]


def test_zero_tokens():
    shape = synth.MoEShape(0, 128, 8, 2, 128)
    inp = synth.make_inputs(shape, 23, guard=False)
    r = Run(inp, 2)
    fw = r.forward()
    assert fw["counts"].cpu().numpy().sum() == 0 and fw["y"].shape[0] == 0
    bw = r.backward(0.0)
    for nm in ("dW_gate", "dW_up", "dW_down"):
        assert not bw[nm].float().cpu().numpy().any()
    assert not bw["dW_r"].cpu().numpy().any()


def test_repeated_calls_are_bitwise_reproducible():
    inp = synth.make_inputs(synth.MoEShape(700, 256, 16, 4, 256), 24)
    r = Run(inp, 4)
    a = r.forward()
    ga = r.backward(0.02)
    b = r.forward()
    gb = r.backward(0.02)
    for n in ("y", "idx", "gates", "perm", "aux"):
        assert torch.equal(a[n], b[n]), n
    for n in ("dx", "dW_r", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(ga[n], gb[n]), n


def test_one_context_across_changing_token_counts():
    """A training loop feeds a different number of tokens every step: the same context (its workspace grows to the
    largest) alternates between token counts, each step stage by stage against the oracle and bitwise equal to a fresh
    context's result - no table, tensor map or count of an earlier step leaks into the next."""
    d, E, k, f = 256, 16, 4, 192
    layer = MoELayer(d, E, f, k)
    weights = synth.make_inputs(synth.MoEShape(8, d, E, k, f), 41)
    for step, T in enumerate([900, 130, 1411, 1, 900]):
        tok = synth.make_tokens(synth.MoEShape(T, d, E, k, f), 500 + step, weights["W_r"], None)
        inp = dict(weights, x=tok["x"], dy=tok["dy"])
        ofw, obw = oracle_run(inp, k, 0.05)
        r = Run(inp, k)
        fresh_fw, fresh_bw = check_all(r, ofw, obw, 0.05)
        dev = r.dev
        fw = layer.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
        bw = layer.backward(dev["dy"], 0.05)
        layer.poll()
        for n in ("y", "idx", "gates", "perm", "aux", "counts"):
            assert torch.equal(fw[n], fresh_fw[n]), (T, n)
        for n in ("dx", "dW_r", "dW_gate", "dW_up", "dW_down"):
            assert torch.equal(bw[n], fresh_bw[n]), (T, n)


def test_two_contexts_on_two_streams():
    """One context per stream: two layers of different shapes enqueue their steps interleaved on two streams and give
    bitwise the results of running alone."""
    cases = [(synth.MoEShape(1200, 256, 16, 4, 256), 51), (synth.MoEShape(700, 384, 8, 2, 320), 52)]
    runs = [Run(synth.make_inputs(sh, seed), sh.k) for sh, seed in cases]
    alone = []
    for r in runs:
        fw = r.forward()
        bw = r.backward(0.03)
        alone.append(({n: fw[n].clone() for n in ("y", "idx", "gates", "aux")},
                      {n: bw[n].clone() for n in ("dx", "dW_r", "dW_gate", "dW_up", "dW_down")}))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [None, None]
    for rep in range(3):
        for i, r in enumerate(runs):
            with torch.cuda.stream(streams[i]):
                fw = r.forward()
                outs[i] = (fw, None)
        for i, r in enumerate(runs):
            with torch.cuda.stream(streams[i]):
                outs[i] = (outs[i][0], r.backward(0.03))
    torch.cuda.synchronize()
    for i, r in enumerate(runs):
        r.layer.poll()
        for n, v in alone[i][0].items():
            assert torch.equal(outs[i][0][n], v), (i, n)
        for n, v in alone[i][1].items():
            assert torch.equal(outs[i][1][n], v), (i, n)


def test_backward_refuses_a_workspace_filled_by_another_forward():
    """The tables in the workspace belong to the forward call that filled it: a backward call (straight through the C
    ABI) naming another token count, or following a forward-only pass, is refused before any launch (it would index out
    of range); the matching call still works afterwards."""
    import ctypes as C
    inp = synth.make_inputs(synth.MoEShape(600, 128, 8, 2, 128), 81)
    r = Run(inp, 2)
    r.forward()
    good = r.backward(0.0)
    layer, dev = r.layer, r.dev
    p = lambda t: C.c_void_p(t.data_ptr())
    out = {n: torch.empty_like(v) for n, v in good.items() if v is not None}
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def c_backward(T):
        return layer.lib.moe_backward(layer.h, T, p(dev["dy"]), C.c_float(0.0), p(dev["x"]), p(dev["W_r"]), p(dev["W_gate"]),
                                      p(dev["W_up"]), p(dev["W_down"]), p(out["dx"]), p(out["dW_r"]), None, p(out["dW_gate"]),
                                      p(out["dW_up"]), p(out["dW_down"]), p(layer.ws), layer.ws.numel(), stream)

    layer.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
    before = binding_launches()
    assert c_backward(300) == -1      # forward was for 600 tokens
    assert binding_launches() == before
    assert c_backward(600) == 0
    torch.cuda.synchronize()
    for n in ("dx", "dW_r", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(out[n], good[n]), n
    # a forward-only pass leaves no pre-activations: no backward on its workspace
    layer.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"], inference=True)
    assert c_backward(600) == -1
    layer.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
    out["dx"].zero_()
    assert c_backward(600) == 0
    torch.cuda.synchronize()
    layer.poll()
    assert torch.equal(out["dx"], good["dx"])


@pytest.mark.parametrize("T,d,E,k,f,seed", [(1000, 512, 16, 4, 384, 14), (777, 256, 64, 8, 192, 27)])
def test_forward_inference_entry(T, d, E, k, f, seed):
    """moe_forward_inference: same y and routing as the training forward, from a workspace of only the inference size
    (no pre-activation buffers), and no backward afterwards."""
    from paper_2608_00916_b200.binding import MoEError
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    ofw, _ = oracle_run(inp, k, 0.0)
    r = Run(inp, k)
    v = r.dev
    assert r.layer.inference_workspace_bytes(T) < r.layer.workspace_bytes(T)
    fw = r.layer.forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"], want_logits=True, inference=True)
    r.layer.poll()
    assert r.layer.ws.numel() == max(r.layer.inference_workspace_bytes(T), 256)  # the small workspace sufficed
    check_routing(fw, ofw)
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL
    with pytest.raises(MoEError):
        r.layer.backward(v["dy"], 0.0)
    train = Run(inp, k).forward()
    assert torch.equal(train["y"], fw["y"])  # bitwise the same outputs as the training forward


@pytest.mark.parametrize("flag", [0, 1, 2, 16])
def test_backward_accumulate_over_micro_batches(flag):
    """moe_backward_accumulate adds the weight gradients of successive micro-batches into fp32 buffers: after
    three micro-batches (one of them leaving experts empty) the buffers hold the sum of the oracle's gradients."""
    d, E, k, f = 256, 16, 4, 320
    base = synth.make_inputs(synth.MoEShape(400, d, E, k, f), 51)
    acc = {"dW_r": torch.zeros(d, E, device="cuda"), "db_r": torch.zeros(E, device="cuda"),
           "dW_gate": torch.zeros(E, d, f, device="cuda"), "dW_up": torch.zeros(E, d, f, device="cuda"),
           "dW_down": torch.zeros(E, f, d, device="cuda")}
    ref = {n: 0.0 for n in ("dW_r", "db_r", "dW_gate", "dW_up", "dW_down")}
    for i, T in enumerate((400, 37, 513)):
        mb = synth.make_inputs(synth.MoEShape(T, d, E, k, f), 60 + i)
        inp = dict(base)
        inp["x"], inp["dy"] = mb["x"], mb["dy"]
        # re-guard the router gaps for these tokens against the shared W_r
        l = synth._guard_logits(inp["x"], inp["W_r"], None)
        keep = ~synth._gap_violations(l, k)
        inp["x"], inp["dy"] = inp["x"][keep], inp["dy"][keep]
        ofw, obw = oracle_run(inp, k, 0.02)
        r = Run(inp, k, flags=flag)
        r.forward()
        dx = r.layer.backward_accumulate(r.dev["dy"], 0.02, acc)
        r.layer.poll()
        assert rel_fro(from_dev_bf16(dx), obw["dx"]) <= TOL
        for n in ref:
            ref[n] = ref[n] + obw[n]
    for n in ref:
        assert rel_fro(acc[n].cpu().numpy(), ref[n]) <= TOL, n
    # fp32 accumulation keeps more of the gradient than the bf16 outputs of moe_backward do
    assert rel_fro(acc["dW_down"].cpu().numpy(), ref["dW_down"]) <= 3e-3


def test_step_host_matches_the_device_path():
    """moe_step_host (host buffers in, host buffers out, copies overlapped with compute on the context's own streams)
    returns the same bits as forward + backward on device tensors; a second call with resident weights too."""
    shape = synth.MoEShape(900, 256, 16, 4, 192)
    inp = synth.make_inputs(shape, 88)
    r = Run(inp, 4)
    fw = r.forward()
    bw = r.backward(inp["d_aux"], want_db=False)
    T, d, E, f = shape.T, shape.d, shape.E, shape.f
    host = {n: torch.from_numpy(inp[n].view(np.int16)).pin_memory() for n in ("x", "dy", "W_r", "W_gate", "W_up", "W_down")}
    host.update(y=torch.zeros(T, d, dtype=torch.int16).pin_memory(), dx=torch.zeros(T, d, dtype=torch.int16).pin_memory(),
                aux=torch.zeros(1).pin_memory(), dW_r=torch.zeros(d, E).pin_memory(),
                dW_gate=torch.zeros(E, d, f, dtype=torch.int16).pin_memory(),
                dW_up=torch.zeros(E, d, f, dtype=torch.int16).pin_memory(),
                dW_down=torch.zeros(E, f, d, dtype=torch.int16).pin_memory())
    layer = r.layer
    dev_buf = torch.empty(layer.e2e_device_bytes(T), dtype=torch.uint8, device="cuda")
    for copy_weights in (True, False):
        for n in ("y", "dx"):
            host[n].zero_()
        layer.step_host(T, dev_buf, host, inp["d_aux"], copy_weights=copy_weights)
        assert torch.equal(host["y"], fw["y"].view(torch.int16).cpu())
        assert torch.equal(host["dx"], bw["dx"].view(torch.int16).cpu())
        assert float(host["aux"][0]) == float(fw["aux"].cpu()[0])
    assert torch.equal(host["dW_r"], bw["dW_r"].cpu())
    for n in ("dW_gate", "dW_up", "dW_down"):
        assert torch.equal(host[n], bw[n].view(torch.int16).cpu()), n
    # pipelined form: two slots in flight, six steps alternating between two different batches
    inp2 = synth.make_inputs(shape, 89)
    inp2["W_r"], inp2["W_gate"], inp2["W_up"], inp2["W_down"] = inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"]
    r2 = Run(inp2, 4)
    fw2 = r2.forward()
    bw2 = r2.backward(inp["d_aux"], want_db=False)
    slots = []
    for sl, src in ((0, inp), (1, inp2)):
        slots.append({"x": torch.from_numpy(src["x"].view(np.int16)).pin_memory(),
                      "dy": torch.from_numpy(src["dy"].view(np.int16)).pin_memory(),
                      "y": torch.zeros(T, d, dtype=torch.int16).pin_memory(),
                      "dx": torch.zeros(T, d, dtype=torch.int16).pin_memory(), "aux": torch.zeros(1).pin_memory()})
    want = [(fw, bw), (fw2, bw2)]
    layer.step_host_begin(0, T, dev_buf, slots[0], inp["d_aux"])
    for i in range(1, 6):
        layer.step_host_begin(i % 2, T, dev_buf, slots[i % 2], inp["d_aux"])
        prev = (i - 1) % 2
        layer.step_host_end(prev)
        assert torch.equal(slots[prev]["y"], want[prev][0]["y"].view(torch.int16).cpu()), i
        assert torch.equal(slots[prev]["dx"], want[prev][1]["dx"].view(torch.int16).cpu()), i
        slots[prev]["y"].zero_()
        slots[prev]["dx"].zero_()
    layer.step_host_end(1)
    assert torch.equal(slots[1]["dx"], bw2["dx"].view(torch.int16).cpu())
    layer.poll()


@pytest.mark.parametrize("T,d,E,k,f,rank,seed", [
    (600, 256, 8, 2, 256, 16, 71),    # the paper's rank
    (1000, 512, 16, 4, 384, 16, 72),  # ragged tails, f not a multiple of 256
    (333, 192, 5, 3, 320, 8, 73),     # smallest rank, SIMT router path, widths not multiples of 128
    (257, 128, 12, 12, 64, 64, 74),   # largest rank, k = E
    (50, 128, 32, 2, 128, 24, 75),    # most experts empty
])
def test_expert_lora_against_the_oracle(T, d, E, k, f, rank, seed):
    """Expert LoRA through moe_lora_forward / moe_lora_backward against the oracle's definition (the plain layer
    evaluated with W + s A B; adapter gradients by the chain rule from the effective-weight gradients)."""
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    lo = synth.make_lora(shape, seed, rank=rank, std=0.05)
    scale = 2.0
    wargs = (inp["W_gate"], inp["W_up"], inp["W_down"], lo["A1"], lo["B1_gate"], lo["B1_up"], lo["A2"], lo["B2"], scale)
    ofw = orc.lora_forward(inp["x"], inp["W_r"], *wargs, k)
    obw = orc.lora_backward(ofw, inp["dy"], 0.02, inp["x"], inp["W_r"], *wargs)
    # the adapters must matter in this test: the adapted output differs visibly from the base layer's
    base = orc.forward(inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"], k)
    assert rel_fro(base["y"], ofw["y"]) > 0.05
    from gpu_util import to_dev_bf16
    r = Run(inp, k)
    v = r.dev
    dlo = {n: to_dev_bf16(lo[n]) for n in ("A1", "B1_gate", "B1_up", "A2", "B2")}
    fw = r.layer.lora_forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"], dlo, scale)
    r.layer.poll()
    assert np.array_equal(fw["idx"].cpu().numpy(), ofw["idx"])
    assert np.array_equal(fw["counts"].cpu().numpy(), ofw["counts"])
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL
    bw = r.layer.lora_backward(v["dy"], 0.02)
    r.layer.poll()
    assert rel_fro(from_dev_bf16(bw["dx"]), obw["dx"]) <= TOL
    assert rel_fro(bw["dW_r"].cpu().numpy(), obw["dW_r"]) <= TOL
    for n in ("dA1", "dB1_gate", "dB1_up", "dA2", "dB2"):
        got = from_dev_bf16(bw[n])
        assert rel_fro(got, obw[n]) <= TOL, n
        for e in range(E):
            if ofw["counts"][e] == 0:
                assert not got[e].any(), (n, e)


def test_bounded_wait_reports_timeout_and_context_survives():
    """A device-side wait that can never complete gives up and the status word says so.  The word is sticky: a forward
    and a backward enqueued after the failure do not erase it, the poll that reports it acknowledges it, and the same
    context and workspace keep working afterwards (no fault, no hang: the wait is bounded by construction)."""
    from paper_2608_00916_b200.binding import MoEError
    inp = synth.make_inputs(synth.MoEShape(300, 128, 8, 2, 128), 25)
    ofw, obw = oracle_run(inp, 2, 0.0)
    r = Run(inp, 2)
    r.forward()  # allocates the workspace, status ok
    r.layer.selftest_timeout()
    v = r.dev
    r.layer.forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"])  # neither call may clear the word
    r.layer.backward(v["dy"], 0.0)
    with pytest.raises(MoEError, match="bounded device-side wait"):
        r.layer.poll()
    r.layer.poll()  # reported once; acknowledged
    fw = r.forward()
    check_routing(fw, ofw)
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL
    # a workspace the library has never seen (arbitrary bytes in its status block) starts clean
    r2 = Run(inp, 2)
    r2.layer._ensure_ws(300)
    r2.layer.ws.fill_(0x5A)
    r2.layer.poll()  # nothing ran on it yet: ok
    fw2 = r2.forward()
    check_routing(fw2, ofw)
    r2.layer.selftest_timeout()
    with pytest.raises(MoEError, match="bounded device-side wait"):
        r2.layer.poll()


def test_pipelined_host_steps_report_a_recorded_timeout():
    """moe_step_host_end reads the status word together with the slot's results: a failure recorded before (or during)
    the step comes back from end() once, and the following steps run clean."""
    from paper_2608_00916_b200.binding import MoEError
    shape = synth.MoEShape(256, 128, 8, 2, 128)
    inp = synth.make_inputs(shape, 27)
    layer = MoELayer(shape.d, shape.E, shape.f, shape.k)
    T = shape.T
    host = {n: torch.from_numpy(inp[n].view(np.int16)).pin_memory() for n in ("x", "dy", "W_r", "W_gate", "W_up", "W_down")}
    host["y"] = torch.empty(T, shape.d, dtype=torch.int16).pin_memory()
    host["dx"] = torch.empty(T, shape.d, dtype=torch.int16).pin_memory()
    host["aux"] = torch.empty(1, dtype=torch.float32).pin_memory()
    host["dW_r"] = torch.empty(shape.d, shape.E, dtype=torch.float32).pin_memory()
    for n in ("dW_gate", "dW_up", "dW_down"):
        host[n] = torch.empty(inp["W_gate"].size, dtype=torch.int16).pin_memory()
    dev_buf = torch.empty(layer.e2e_device_bytes(T), dtype=torch.uint8, device="cuda")
    layer.step_host(T, dev_buf, host, 0.01, copy_weights=True)
    y_ok = host["y"].clone()
    # the workspace of the host steps lives inside dev_buf: record a timeout in ITS status word
    ws_off = layer.e2e_workspace_offset(T)
    layer.ws, layer.T = dev_buf[ws_off:], T
    layer.selftest_timeout()
    layer.step_host_begin(0, T, dev_buf, host, 0.01)
    with pytest.raises(MoEError, match="bounded device-side wait"):
        layer.step_host_end(0)
    host["y"].zero_()
    layer.step_host_begin(1, T, dev_buf, host, 0.01)
    layer.step_host_end(1)  # clean again
    assert torch.equal(host["y"], y_ok)
    layer.poll()


def test_forward_backward_replay_from_a_cuda_graph():
    """Neither call synchronises, allocates or reads anything back, so a forward + backward pair can be captured
    into a CUDA graph (after one eager call has set the kernels' attributes) and replayed: same bits as eager."""
    inp = synth.make_inputs(synth.MoEShape(512, 256, 16, 4, 256), 26)
    r = Run(inp, 4)
    v = r.dev
    eager_fw = r.layer.forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"])
    eager_bw = r.layer.backward(v["dy"], 0.03)
    torch.cuda.synchronize()
    keep = {n: eager_fw[n].clone() for n in ("y", "idx", "gates", "aux")} | {n: eager_bw[n].clone() for n in ("dx", "dW_r", "dW_gate")}
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            gfw = r.layer.forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"])
            gbw = r.layer.backward(v["dy"], 0.03)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    r.layer.poll()
    for n in ("y", "idx", "gates", "aux"):
        assert torch.equal(gfw[n], keep[n]), n
    for n in ("dx", "dW_r", "dW_gate"):
        assert torch.equal(gbw[n], keep[n]), n


def test_midsize_qwen_shape_full_oracle():
    """The Qwen3-30B-A3B expert shape with fewer tokens, full oracle in float32 mode."""
    shape = synth.MoEShape(2048, 2048, 128, 8, 768)
    inp = synth.make_inputs(shape, 31, x_std=1.0)
    ofw, obw = oracle_run(inp, 8, 0.01, dtype=np.float32)
    check_all(Run(inp, 8), ofw, obw, 0.01, stages=False)


# ------------------------------------------------------------------------------------------ full-size configurations
def sampled_parity(name, n_tokens=48):
    """Full-size workloads in the launch configuration the benchmark times.  The oracle routes every token
    (cheap) and computes y rows for sampled tokens plus complete weight gradients of four experts (hottest,
    median, coldest non-empty, one empty if present); properties cover the rest."""
    shape, seed, x_std, skew = synth.CONFIGS[name]
    inp = synth.make_inputs(shape, seed, x_std=x_std, skew=skew)
    k, E, T = shape.k, shape.E, shape.T
    rt = orc.route_only(inp["x"], inp["W_r"], k, E, b_r=inp.get("b_r"))
    r = Run(inp, k)
    fw = r.forward()
    check_routing(fw, rt)
    perm = fw["perm"].cpu().numpy()
    assert np.array_equal(np.sort(perm), np.arange(T * k))
    inv = r.ints("inv")
    pad = r.ints("pad_offsets")
    assert (np.diff(pad) % 128 == 0).all() and np.array_equal(np.diff(pad) >= fw["counts"].cpu().numpy(), np.ones(E, bool))
    assert len(np.unique(inv)) == T * k
    rng = np.random.default_rng(seed)
    toks = rng.choice(T, size=n_tokens, replace=False)
    y = from_dev_bf16(fw["y"][torch.from_numpy(toks).cuda()])
    ref = np.stack([orc.token_rows(int(t), rt, inp["x"], inp["W_gate"], inp["W_up"], inp["W_down"]) for t in toks])
    assert rel_fro(y, ref) <= TOL
    bw = r.backward(inp["d_aux"])
    counts = rt["counts"]
    order = np.argsort(counts)
    nonempty = order[counts[order] > 0]
    picks = {int(nonempty[-1]), int(nonempty[len(nonempty) // 2]), int(nonempty[0])}
    if (counts == 0).any():
        picks.add(int(order[0]))
    for e in sorted(picks):
        gg, gu, gd = orc.expert_grads(e, rt, inp["dy"], inp["x"], inp["W_gate"], inp["W_up"], inp["W_down"],
                                      dtype=np.float32)
        for nm, ref_e in (("dW_gate", gg), ("dW_up", gu), ("dW_down", gd)):
            got = from_dev_bf16(bw[nm][e])
            if counts[e] == 0:
                assert not got.any()
            else:
                assert rel_fro(got, ref_e) <= 2e-2, (nm, e, int(counts[e]))
    # dW_r against x^T dl with the GPU's own dl (host fp64 contraction), dl rows of sampled tokens sum to zero
    dl = r.layer.buffer("dl", torch.float32).view(T, E).double().cpu().numpy()
    assert np.abs(dl.sum(1)).max() <= 1e-4 * max(1.0, np.abs(dl).max())
    ref_dwr = synth.bf16_bits_to_f64(inp["x"]).T @ dl
    assert rel_fro(bw["dW_r"].cpu().numpy(), ref_dwr) <= 1e-3
    assert torch.isfinite(bw["dx"].float()).all()
    # dx and dl rows of sampled tokens against the oracle's per-token backward
    btoks = toks[: max(4, n_tokens // 4)]
    ref_dx, ref_dl = zip(*(orc.token_backward(int(t), rt, inp["dy"], inp["d_aux"], inp["x"], inp["W_r"], inp["W_gate"],
                                              inp["W_up"], inp["W_down"]) for t in btoks))
    got_dx = from_dev_bf16(bw["dx"][torch.from_numpy(btoks).cuda()])
    assert rel_fro(got_dx, np.stack(ref_dx)) <= TOL
    assert rel_fro(dl[btoks], np.stack(ref_dl)) <= TOL


def test_full_qwen_config_sampled():
    sampled_parity("qwen")


def test_full_skewed_config_sampled():
    sampled_parity("skewed")


def test_full_coarse_config_sampled():
    sampled_parity("coarse", n_tokens=8)


@pytest.mark.parametrize("name", ["sweep_T1000", "sweep_T4096", "sweep_T8191", "sweep_T32768", "sweep_T65536"])
def test_sweep_sampled(name):
    sampled_parity(name, n_tokens=24)


def test_grouped_weight_gradients_signal_ranges_of_experts():
    """moe_backward_accumulate_grouped: the weight gradients run range by range of experts, an event fires after each
    range, and the buffers end up bitwise as moe_backward_accumulate leaves them.  The reducer's side-stream plumbing
    is watched on one GPU through an injected stand-in for the all-reduce (it doubles a slab once its event has fired):
    every range must have been final before it was touched."""
    from paper_2608_00916_b200 import dist as pdist
    d, E, k, f = 256, 24, 4, 192
    inp = synth.make_inputs(synth.MoEShape(1800, d, E, k, f), 71)
    r = Run(inp, k)
    r.forward()

    def zeros():
        return {"dW_r": torch.zeros(d, E, device="cuda"), "dW_gate": torch.zeros(E, d, f, device="cuda"),
                "dW_up": torch.zeros(E, d, f, device="cuda"), "dW_down": torch.zeros(E, f, d, device="cuda")}
    plain = zeros()
    dx0 = r.layer.backward_accumulate(r.dev["dy"], 0.02, plain)
    touched = []

    def fake_all_reduce(t):
        touched.append(tuple(t.shape))
        t.mul_(2.0)  # on the communication stream, after the range's event
        return None
    red = pdist.GradAllReducer(n_groups=5, reduce_fn=fake_all_reduce)  # 24 experts -> ranges of 5, 5, 5, 5, 4
    assert red.group_ranges(E) == [(0, 5), (5, 10), (10, 15), (15, 20), (20, 24)]
    grouped = zeros()
    r.forward()
    dx1 = r.layer.backward_accumulate(r.dev["dy"], 0.02, grouped, group_events=red.events())
    red.start_grouped(grouped)
    red.wait()
    torch.cuda.synchronize()
    r.layer.poll()
    assert all(ev.query() for ev in red.events())
    assert torch.equal(dx0, dx1)
    for n in plain:
        assert torch.equal(grouped[n], 2.0 * plain[n]), n  # doubled exactly once, after the final value was there
    assert touched == [(5, f, d)] * 4 + [(4, f, d)] + [(5, d, f)] * 8 + [(4, d, f)] * 2 + [(d, E)]


def test_grouped_reduction_through_nccl_on_a_one_rank_group():
    """The data-parallel gradient path with the real collective (NCCL all_reduce per range of experts on the reducer's
    stream, as the grouped backward signals the ranges) in a child process on a one-rank group, where summing over the
    ranks changes nothing: bitwise the plain accumulation window.  More ranks need more GPUs than a test run has."""
    import os
    import subprocess
    import sys
    from paper_2608_00916_b200.dist import free_port
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "tests", "dp_reduce_probe.py"), str(free_port())],
                         capture_output=True, text=True, timeout=600, cwd=root)
    if "GROUP_READY" not in out.stdout:
        pytest.skip("this box cannot host a NCCL group: " + out.stderr[-300:])
    assert out.returncode == 0, out.stderr[-2000:]
    assert "REDUCE_OK" in out.stdout, out.stdout[-500:] + out.stderr[-1500:]


def test_fp32_router_weight():
    """MOE_FLAG_ROUTER_FP32: W_r arrives as genuine fp32 values (not representable in bf16); the library splits it into
    three exact bf16 terms, so logits, routing and gradients follow the oracle evaluated with the fp32 weight."""
    from paper_2608_00916_b200.binding import FLAG_ROUTER_FP32
    shape = synth.MoEShape(900, 256, 32, 4, 128)
    inp = synth.make_inputs(shape, 81)
    rng = np.random.default_rng(81)
    W32 = (0.02 * rng.standard_normal((shape.d, shape.E))).astype(np.float32)
    assert np.any(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(W32)) != W32)  # needs more than bf16
    # keep the tokens whose top-k gaps are safe under THIS weight
    l = synth.bf16_bits_to_f64(inp["x"]) @ W32.astype(np.float64)
    keep = ~synth._gap_violations(l, shape.k)
    inp["x"], inp["dy"] = inp["x"][keep], inp["dy"][keep]
    T = int(keep.sum())
    ofw = orc.forward(inp["x"], W32, inp["W_gate"], inp["W_up"], inp["W_down"], shape.k)
    obw = orc.backward(ofw, inp["dy"], 0.02, inp["x"], W32, inp["W_gate"], inp["W_up"], inp["W_down"])
    layer = MoELayer(shape.d, shape.E, shape.f, shape.k, FLAG_ROUTER_FP32)
    dev = {n: torch.from_numpy(inp[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("x", "W_gate", "W_up", "W_down", "dy")}
    W_r = torch.from_numpy(W32).cuda()
    fw = layer.forward(dev["x"], W_r, dev["W_gate"], dev["W_up"], dev["W_down"], want_logits=True)
    bw = layer.backward(dev["dy"], 0.02, want_db=True)
    layer.poll()
    check_routing(fw, ofw)
    # the logits carry the low-order bits of the weight: a bf16-rounded weight would be off by ~1e-3 relative
    lg = fw["logits"].cpu().numpy()
    bf = synth.bf16_bits_to_f64(inp["x"]) @ synth.bf16_bits_to_f64(synth.f32_to_bf16_bits(W32))
    assert np.abs(lg - ofw["logits"]).max() < 0.05 * np.abs(bf - ofw["logits"]).max()
    assert rel_fro(from_dev_bf16(fw["y"]), ofw["y"]) <= TOL
    for n in ("dx", "dW_gate", "dW_up", "dW_down"):
        assert rel_fro(from_dev_bf16(bw[n]), obw[n]) <= TOL, n
    assert rel_fro(bw["dW_r"].cpu().numpy(), obw["dW_r"]) <= TOL
    assert rel_fro(bw["db_r"].cpu().numpy(), obw["db_r"]) <= TOL
    # the router term of dx, isolated: dx minus the oracle's expert part
    assert T > 800


def test_debug_checks_report_a_corrupted_routing_table_without_touching_memory_out_of_range():
    """MOE_FLAG_DEBUG_CHECKS: a row index of the routing tables is overwritten with a value far outside the row buffers
    between forward and backward.  The checked kernels record MOE_ERR_DEVICE_BOUNDS and skip / redirect the access (so
    nothing faults); with an intact table the same context computes the same bits as an unchecked one."""
    from paper_2608_00916_b200.binding import FLAG_DEBUG_CHECKS, MoEError
    inp = synth.make_inputs(synth.MoEShape(500, 128, 16, 4, 128), 91)
    plain = Run(inp, 4)
    pfw = plain.forward()
    pbw = plain.backward(0.01)
    r = Run(inp, 4, flags=FLAG_DEBUG_CHECKS)
    fw = r.forward()
    bw = r.backward(0.01)
    for n in ("y", "idx", "gates"):
        assert torch.equal(fw[n], pfw[n]), n
    for n in ("dx", "dW_r", "dW_gate", "dW_down"):
        assert torch.equal(bw[n], pbw[n]), n
    # corrupt one entry of inv (the padded row of pair (token 7, slot 1)) and run backward again
    r.forward()
    inv = r.layer.buffer("inv", torch.int32)
    inv[7 * 4 + 1] = 2 ** 30
    v = r.dev
    r.layer.backward(v["dy"], 0.01)
    with pytest.raises(MoEError, match="bounds check"):
        r.layer.poll()
    # acknowledged: the context and the workspace work again
    fw2 = r.forward()
    assert torch.equal(fw2["y"], pfw["y"])
