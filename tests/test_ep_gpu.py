"""Expert parallelism (EP > 1): the ranks of a group, run inside one process on one GPU (ep.LocalGroup: the same
kernels a multi-GPU group runs, phases enqueued rank after rank), must reproduce the oracle applied to the
concatenation of the ranks' token batches: routing bit-exact per rank, the owners' row buffers in the oracle's
expert-major order, y and dx per token, the owned experts' weight gradients, and the sum over ranks of dW_r."""
import numpy as np
import pytest
import torch

from paper_2608_00916_b200 import ep, synth
from gpu_util import from_dev_bf16, oracle_run, rel_fro, to_dev_bf16
from oracle import moe_oracle as orc

pytestmark = pytest.mark.gpu
TOL = 1e-2


@pytest.mark.parametrize("d,E,k,f,tokens,seed,flags", [
    (256, 16, 4, 256, [300, 517], 31, 0),            # two ranks, uneven batches
    (128, 32, 8, 128, [100, 0, 333, 64], 32, 0),     # four ranks, one of them without tokens
    (128, 8, 4, 192, [260, 130, 50, 90], 33, 2),     # fewer owned experts (2) than top_k (4); one-CTA tiles
    (192, 64, 6, 64, [1500, 1100], 34, 1),           # 32 owned experts each, CTA-pair tiles
])
def test_local_group_matches_the_oracle_on_the_concatenated_batch(d, E, k, f, tokens, seed, flags):
    world = len(tokens)
    T = sum(tokens)
    shape = synth.MoEShape(T, d, E, k, f)
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    ofw, obw = oracle_run(inp, k, 0.0)
    bounds = np.concatenate([[0], np.cumsum(tokens)])
    dev = {n: to_dev_bf16(inp[n]) for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
    xs = [dev["x"][bounds[r]:bounds[r + 1]].contiguous() for r in range(world)]
    dys = [dev["dy"][bounds[r]:bounds[r + 1]].contiguous() for r in range(world)]
    grp = ep.LocalGroup(d, E, f, k, world, ep.rows_cap_bound(tokens, k, E, world), flags)
    fw, all_counts = grp.forward(xs, dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
    grp.poll()
    e_loc = E // world
    ac = all_counts.cpu().numpy()
    assert np.array_equal(ac.sum(axis=0), ofw["counts"])
    for r in range(world):
        sl = slice(bounds[r], bounds[r + 1])
        # routing of the rank's tokens: bit-exact; its own counts; aux over its own tokens
        assert np.array_equal(fw[r]["idx"].cpu().numpy(), ofw["idx"][sl])
        if tokens[r] > 0:
            assert np.abs(fw[r]["gates"].cpu().numpy() - ofw["gates"][sl]).max() <= 1e-5
        assert np.array_equal(ac[r], np.bincount(ofw["idx"][sl].ravel(), minlength=E))
        if tokens[r] > 0:
            local = orc.route_only(inp["x"][sl], inp["W_r"], k, E)
            assert float(fw[r]["aux"].cpu()[0]) == pytest.approx(local["aux"], rel=1e-4)
            assert rel_fro(from_dev_bf16(fw[r]["y"]), ofw["y"][sl]) <= TOL
        # placement: the device tables equal the host restatement
        plan = ep.plan_host(ac, r, world)
        rk = grp.ranks[r]
        assert np.array_equal(rk.buffer("ep_dest", torch.int32, False).cpu().numpy(), plan["dest_base"])
        assert np.array_equal(rk.buffer("counts", torch.int32, True).cpu().numpy(), plan["own_counts"])
        assert np.array_equal(rk.buffer("pad_offsets", torch.int32, True).cpu().numpy(), plan["own_pad_offsets"])
        if tokens[r] > 0:
            inv = rk.buffer("inv", torch.int32, False).view(tokens[r], k).cpu().numpy()
            assert np.array_equal(inv, ep.rows_of_rank(ofw["idx"][sl], plan["dest_base"]))
        # the owner's xp rows: expert by expert the oracle's rows of the concatenated batch, in its order; pad rows zero
        xp = rk.buffer("xp", torch.bfloat16, True).view(-1, d)
        for el in range(e_loc):
            e = r * e_loc + el
            n = int(plan["own_counts"][el])
            p0, p1 = int(plan["own_pad_offsets"][el]), int(plan["own_pad_offsets"][el + 1])
            got = xp[p0:p1].float().cpu().numpy()
            ref = ofw["xp"][ofw["offsets"][e]:ofw["offsets"][e + 1]]
            assert np.array_equal(got[:n], ref), (r, e)
            assert not got[n:].any(), (r, e)
    sender, owner = grp.backward(dys, 0.0, want_db=True)
    grp.poll()
    dW_r = np.zeros((d, E))
    db_r = np.zeros(E)
    for r in range(world):
        sl = slice(bounds[r], bounds[r + 1])
        if tokens[r] > 0:
            assert rel_fro(from_dev_bf16(sender[r]["dx"]), obw["dx"][sl]) <= TOL
            dl = grp.ranks[r].buffer("dl", torch.float32, False).view(tokens[r], E).cpu().numpy()
            assert rel_fro(dl, obw["dl"][sl]) <= TOL
        dW_r += sender[r]["dW_r"].cpu().numpy().astype(np.float64)
        db_r += sender[r]["db_r"].cpu().numpy().astype(np.float64)
        own = slice(r * e_loc, (r + 1) * e_loc)
        for n in ("dW_gate", "dW_up", "dW_down"):
            got = from_dev_bf16(owner[r][n])
            assert rel_fro(got, obw[n][own]) <= TOL, (r, n)
            for el in range(e_loc):
                if ofw["counts"][r * e_loc + el] == 0:
                    assert not got[el].any()
                else:
                    assert rel_fro(got[el], obw[n][r * e_loc + el]) <= 2e-2, (r, n, el)
    assert rel_fro(dW_r, obw["dW_r"]) <= TOL
    assert rel_fro(db_r, obw["db_r"]) <= TOL


def test_ep_with_one_rank_equals_the_plain_layer():
    """world = 1 degenerates to the one-GPU layer: same routing, y and gradients as moe_forward / moe_backward."""
    from gpu_util import Run
    shape = synth.MoEShape(700, 256, 16, 4, 128)
    inp = synth.make_inputs(shape, 35)
    r = Run(inp, shape.k)
    fw = r.forward()
    bw = r.backward(0.03)
    grp = ep.LocalGroup(shape.d, shape.E, shape.f, shape.k, 1, shape.T * shape.k)
    v = r.dev
    efw, _ = grp.forward([v["x"]], v["W_r"], v["W_gate"], v["W_up"], v["W_down"])
    sender, owner = grp.backward([v["dy"]], 0.03)
    grp.poll()
    assert torch.equal(efw[0]["idx"], fw["idx"]) and torch.equal(efw[0]["gates"], fw["gates"])
    assert torch.equal(efw[0]["y"], fw["y"]) and torch.equal(efw[0]["aux"], fw["aux"])
    assert torch.equal(sender[0]["dx"], bw["dx"]) and torch.equal(sender[0]["dW_r"], bw["dW_r"])
    for n in ("dW_gate", "dW_up", "dW_down"):
        assert torch.equal(owner[0][n], bw[n]), n


def test_dist_group_with_one_rank():
    """ep.DistGroup - the multi-process form (NCCL all_gather of the counts, owner workspace in symmetric memory and
    mapped through its rendezvous, group barriers between phases) - on a one-rank group in a child process: bitwise the
    plain layer.  More ranks need more GPUs than a test run has."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    from paper_2608_00916_b200.dist import free_port
    out = subprocess.run([sys.executable, os.path.join(root, "tests", "ep_dist_probe.py"), str(free_port())],
                         capture_output=True, text=True, timeout=600, cwd=root)
    if "DIST_GROUP_READY" not in out.stdout:
        pytest.skip("this box cannot host a NCCL group with symmetric memory: " + out.stderr[-300:])
    assert out.returncode == 0, out.stderr[-2000:]
    assert "DIST_GROUP_OK" in out.stdout, out.stdout[-500:] + out.stderr[-1500:]


def test_ep_main_gradients_accumulate_over_micro_batches():
    """moe_ep_expert_backward_accumulate: over a window of three micro-batches (uneven batches on two ranks) every rank's
    fp32 main gradients of its own experts equal the oracle's gradients summed over the window; experts that saw no row
    in the whole window keep the value the buffers started with."""
    d, E, k, f, world = 128, 16, 2, 192, 2
    e_loc = E // world
    batches = [[90, 40], [10, 200], [128, 128]]
    weights = synth.make_inputs(synth.MoEShape(8, d, E, k, f), 61)
    # a bias that leaves the last two experts without tokens in every micro-batch
    b_r = np.zeros(E, dtype=np.float32)
    b_r[-2:] = -50.0
    wdev = {n: to_dev_bf16(weights[n]) for n in ("W_r", "W_gate", "W_up", "W_down")}
    b_dev = torch.from_numpy(b_r).cuda()
    cap = ep.rows_cap_bound([max(b[r] for b in batches) for r in range(world)], k, E, world)
    grp = ep.LocalGroup(d, E, f, k, world, cap)
    acc = [{n: torch.zeros((e_loc,) + tuple(wdev[w].shape[1:]), dtype=torch.float32, device="cuda")
            for n, w in (("dW_gate", "W_gate"), ("dW_up", "W_up"), ("dW_down", "W_down"))} for _ in range(world)]
    sentinel = 0.25  # a recognisable start value in the slabs of the two experts that never get a row
    for t in acc[world - 1].values():
        t[-2:] = sentinel
    ref = {n: np.zeros(weights[w].shape, dtype=np.float64) for n, w in (("dW_gate", "W_gate"), ("dW_up", "W_up"), ("dW_down", "W_down"))}
    for step, tokens in enumerate(batches):
        T = sum(tokens)
        tok = synth.make_tokens(synth.MoEShape(T, d, E, k, f), 700 + step, weights["W_r"], b_r)
        inp = dict(weights, x=tok["x"], dy=tok["dy"], b_r=b_r)
        ofw, obw = oracle_run(inp, k, 0.0)
        assert ofw["counts"][-2:].sum() == 0
        for n in ref:
            ref[n] += obw[n]
        x, dy = to_dev_bf16(tok["x"]), to_dev_bf16(tok["dy"])
        bounds = np.concatenate([[0], np.cumsum(tokens)])
        xs = [x[bounds[r]:bounds[r + 1]].contiguous() for r in range(world)]
        dys = [dy[bounds[r]:bounds[r + 1]].contiguous() for r in range(world)]
        grp.forward(xs, wdev["W_r"], wdev["W_gate"], wdev["W_up"], wdev["W_down"], b_r=b_dev)
        grp.backward(dys, 0.0, acc=acc)
        grp.poll()
    for r in range(world):
        own = slice(r * e_loc, (r + 1) * e_loc)
        for n in ref:
            got = acc[r][n].cpu().numpy().astype(np.float64)
            if r == world - 1:
                assert np.all(got[-2:] == sentinel), n  # untouched
                assert rel_fro(got[:-2], ref[n][own][:-2]) <= TOL, (r, n)
            else:
                assert rel_fro(got, ref[n][own]) <= TOL, (r, n)


def test_rows_beyond_the_owner_buffers_are_refused_not_written():
    """A rows_cap that the routing exceeds: the plan refuses the step on every rank (same counts everywhere), nothing is
    written outside or inside the owner buffers' rows (canaries behind every owner workspace stay intact), y and dx are
    zeros, the failure is reported once as MOE_ERR_DEVICE_BOUNDS, and the same contexts then run a step that fits."""
    from paper_2608_00916_b200.binding import MoEError
    from gpu_util import Run
    d, E, k, f, world = 128, 16, 4, 128, 2
    rows_cap = 1024
    probe = ep.EPRank(d, E, f, k, world, 0, rows_cap)
    own_bytes = probe.own_bytes
    del probe
    canary = 1 << 20
    bufs = [torch.full((own_bytes + canary,), 0xA5, dtype=torch.uint8, device="cuda") for _ in range(world)]
    ranks = [ep.EPRank(d, E, f, k, world, r, rows_cap, own_ws=bufs[r][:own_bytes]) for r in range(world)]
    for rk in ranks:
        rk.set_peers([b.data_ptr() for b in bufs])
    grp = ep.LocalGroup.__new__(ep.LocalGroup)
    grp.world, grp.ranks = world, ranks

    def run(tokens, seed):
        shape = synth.MoEShape(sum(tokens), d, E, k, f)
        inp = synth.make_inputs(shape, seed, x_std=1.0)
        dev = {n: to_dev_bf16(inp[n]) for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
        b = np.concatenate([[0], np.cumsum(tokens)])
        xs = [dev["x"][b[r]:b[r + 1]].contiguous() for r in range(world)]
        dys = [dev["dy"][b[r]:b[r + 1]].contiguous() for r in range(world)]
        fw, _ = grp.forward(xs, dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
        sender, owner = grp.backward(dys, 0.0)
        torch.cuda.synchronize()
        return inp, fw, sender, owner

    # 2 x 700 tokens x 4 slots = 5600 rows for 2 owners of 1024 rows each: does not fit
    _, fw, sender, owner = run([700, 700], 71)
    for r in range(world):
        with pytest.raises(MoEError, match="bounds"):
            ranks[r].poll()
        ranks[r].poll()  # reported once
        assert not fw[r]["y"].float().abs().sum().item() and not sender[r]["dx"].float().abs().sum().item()
        for n in ("dW_gate", "dW_up", "dW_down"):
            assert not owner[r][n].float().abs().sum().item()
        assert bool((bufs[r][own_bytes:] == 0xA5).all())
        assert bool((ranks[r].buffer("inv", torch.int32, False) == -1).all())
    # a step that fits, on the same contexts: the oracle's results
    tokens = [100, 60]
    inp, fw, sender, owner = run(tokens, 72)
    ofw, obw = oracle_run(inp, k, 0.0)
    b = np.concatenate([[0], np.cumsum(tokens)])
    for r in range(world):
        ranks[r].poll()
        assert np.array_equal(fw[r]["idx"].cpu().numpy(), ofw["idx"][b[r]:b[r + 1]])
        assert rel_fro(from_dev_bf16(fw[r]["y"]), ofw["y"][b[r]:b[r + 1]]) <= TOL
        assert rel_fro(from_dev_bf16(sender[r]["dx"]), obw["dx"][b[r]:b[r + 1]]) <= TOL
        assert bool((bufs[r][own_bytes:] == 0xA5).all())


def test_phases_must_name_the_routed_token_count():
    """The sender workspace holds the routing of moe_ep_route's T tokens: a later phase that names another T is refused
    on the host before any launch."""
    import ctypes as C
    d, E, k, f = 128, 8, 2, 128
    inp = synth.make_inputs(synth.MoEShape(200, d, E, k, f), 91)
    x, W_r = to_dev_bf16(inp["x"]), to_dev_bf16(inp["W_r"])
    rk = ep.EPRank(d, E, f, k, 1, 0, 200 * k)
    rk.set_peers([rk.own_ws.data_ptr()])
    out = rk.route(x, W_r)
    rk.plan(out["counts_local"].view(1, E).contiguous())
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    p = lambda t: C.c_void_p(t.data_ptr())
    assert rk.lib.moe_ep_dispatch(rk.h, 100, p(x), 0, rk.peers, p(rk.send_ws), rk.send_ws.numel(), stream) == -1
    y = torch.empty(200, d, dtype=torch.bfloat16, device="cuda")
    assert rk.lib.moe_ep_combine(rk.h, 199, rk.peers, p(rk.send_ws), rk.send_ws.numel(), p(y), stream) == -1
    assert rk.lib.moe_ep_dispatch(rk.h, 200, p(x), 0, rk.peers, p(rk.send_ws), rk.send_ws.numel(), stream) == 0
    torch.cuda.synchronize()
    rk.poll()
