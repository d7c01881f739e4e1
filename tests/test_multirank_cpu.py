"""The N > 1 path of the benchmark is data parallel over tokens with replicated experts and no data-path
collective; its host logic (rendezvous, per-rank token draws, barrier, max-over-ranks timing, whole-job
throughput) runs here as two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    from oracle import moe_oracle as orc
    from paper_2608_00916_b200 import dist as pdist
    from paper_2608_00916_b200 import synth
    pdist.init(world, rank, backend="gloo")
    shape = synth.MoEShape(64, 64, 8, 2, 64)
    base = synth.make_inputs(shape, 500, threads=1)          # weights: same seed on every rank
    # the rank's own tokens, guarded against the router weight all ranks share
    mine = base if rank == 0 else synth.make_tokens(shape, pdist.shard_seed(500, rank), base["W_r"], base["b_r"], threads=1)
    gaps = synth._gap_violations(synth._guard_logits(mine["x"], base["W_r"], base["b_r"]), shape.k)
    assert not gaps.any()
    fw = orc.forward(mine["x"], base["W_r"], base["W_gate"], base["W_up"], base["W_down"], 2)
    pdist.barrier()
    ms = 10.0 * (rank + 1)  # pretend rank r took 10 (r + 1) ms
    q.put((rank, pdist.max_over_ranks(ms), pdist.job_throughput(shape.T, ms), float(np.abs(fw["y"]).sum()),
           int(base["W_gate"].view(np.uint16).sum()), int(mine["x"].view(np.uint16).sum())))
    pdist.finish()


def test_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    from paper_2608_00916_b200.dist import free_port
    port = free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, max0, thr0, y0, w0, x0), (r1, max1, thr1, y1, w1, x1) = res
    assert max0 == max1 == 20.0                      # slowest rank decides
    assert thr0 == thr1 == (64 + 64) / 0.020          # tokens of all ranks over that time
    assert w0 == w1                                   # replicated weights
    assert x0 != x1 and y0 != y1                      # different token batches per rank


def _reduce_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch
    from oracle import moe_oracle as orc
    from paper_2608_00916_b200 import dist as pdist
    from paper_2608_00916_b200 import synth
    pdist.init(world, rank, backend="gloo")
    shape = synth.MoEShape(48, 64, 6, 2, 64)
    base = synth.make_inputs(shape, 700, threads=1)
    mine = base if rank == 0 else synth.make_tokens(shape, pdist.shard_seed(700, rank), base["W_r"], base["b_r"], threads=1)
    fw = orc.forward(mine["x"], base["W_r"], base["W_gate"], base["W_up"], base["W_down"], 2)
    bw = orc.backward(fw, mine["dy"], 0.0, mine["x"], base["W_r"], base["W_gate"], base["W_up"], base["W_down"])
    acc = [torch.from_numpy(bw[n].astype(np.float32)).clone() for n in ("dW_gate", "dW_up", "dW_down", "dW_r")]
    local = [a.clone() for a in acc]
    red = pdist.GradAllReducer(experts_per_bucket=4)
    assert [(e0, e1) for t, e0, e1 in red.buckets(acc) if t.dim() == 3][:2] == [(0, 4), (4, 6)]
    red.start(acc)
    red.wait()
    q.put((rank, [a.numpy() for a in acc], [a.numpy() for a in local]))
    pdist.finish()


def test_gradient_all_reduce_over_two_gloo_ranks():
    """Data-parallel ranks hold different token batches and replicated experts; after GradAllReducer every rank holds
    the sum of both ranks' weight gradients (bucketed along the expert axis, asynchronous)."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    from paper_2608_00916_b200.dist import free_port
    port = free_port()
    procs = [ctx.Process(target=_reduce_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, red0, loc0), (_, red1, loc1) = res
    for a0, a1, l0, l1 in zip(red0, red1, loc0, loc1):
        np.testing.assert_allclose(a0, l0 + l1, rtol=1e-6, atol=1e-7)
        np.testing.assert_array_equal(a0, a1)
        assert np.abs(l0 - l1).max() > 0


def test_rank_environment_of_the_launcher():
    """What `bench.py --gpus N` hands to each rank it starts: rank, local rank, world size, loopback rendezvous, and
    NCCL's communicator log line left on unless the caller chose otherwise.  No GPU is touched."""
    from paper_2608_00916_b200 import dist as pdist
    port = pdist.free_port()
    assert 1024 < port < 65536
    for world in (2, 8):
        envs = [pdist.rank_environment(r, world, port, base_env={"PATH": "/bin"}) for r in range(world)]
        assert [e["RANK"] for e in envs] == [str(r) for r in range(world)]
        assert [e["LOCAL_RANK"] for e in envs] == [str(r) for r in range(world)]
        assert all(e["WORLD_SIZE"] == str(world) and e["MASTER_ADDR"] == "127.0.0.1" and e["MASTER_PORT"] == str(port)
                   for e in envs)
        assert all(e["NCCL_DEBUG"] == "INFO" and e["PATH"] == "/bin" for e in envs)
    assert pdist.rank_environment(0, 2, port, base_env={"NCCL_DEBUG": "WARN"})["NCCL_DEBUG"] == "WARN"


def test_launcher_starts_gloo_ranks(tmp_path):
    """The launcher behind `bench.py --gpus N` starts N processes that find each other: here two CPU ranks that
    initialise gloo from the environment they were given and agree on the max-over-ranks time."""
    from paper_2608_00916_b200 import dist as pdist
    script = os.path.join(ROOT, "tests", "rank_probe.py")
    rc = pdist.launch_ranks(2, script, [str(tmp_path)], timeout=180)
    assert rc == 0
    got = sorted((tmp_path / f"rank{r}.txt").read_text() for r in range(2))
    assert got == ["0 2 0 20.0", "1 2 1 20.0"]
    # a rank that fails makes the launcher report it
    assert pdist.launch_ranks(2, script, [str(tmp_path), "fail-on-1"], timeout=180) != 0


# ------------------------------------------------------------------------------------------ expert parallelism
def _ep_worker(rank, world, port, q):
    """One CPU rank of an expert-parallel group.  The exchange logic under test is the host restatement of the
    placement (ep.plan_host / ep.rows_of_rank): counts all-gather, per-rank expert ownership, destination rows inside
    the owner's expert-major buffers, the inverse map used by the combine.  The per-expert arithmetic is the oracle's
    (test infrastructure); rows travel between the ranks through the gloo group."""
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch
    import torch.distributed as dist
    from oracle import moe_oracle as orc
    from paper_2608_00916_b200 import dist as pdist
    from paper_2608_00916_b200 import ep, synth
    pdist.init(world, rank, backend="gloo")
    d, E, k, f = 64, 8, 3, 64
    tokens = [37, 0, 52, 21][:world] if world == 4 else [45, 30]
    T = sum(tokens)
    inp = synth.make_inputs(synth.MoEShape(T, d, E, k, f), 900 + world, threads=1)  # the concatenated batch
    b = np.concatenate([[0], np.cumsum(tokens)])
    sl = slice(b[rank], b[rank + 1])
    e_loc = E // world
    x = orc.widen_bf16(inp["x"][sl])
    dy = orc.widen_bf16(inp["dy"][sl])
    Wg, Wu, Wd = (orc.widen_bf16(inp[n][rank * e_loc:(rank + 1) * e_loc]) for n in ("W_gate", "W_up", "W_down"))
    route = orc.route_only(inp["x"][sl], inp["W_r"], k, E) if tokens[rank] else {"idx": np.zeros((0, k), np.int64),
                                                                                    "gates": np.zeros((0, k))}
    idx, gates = route["idx"], route["gates"]
    # --- counts all-gather
    mine = torch.from_numpy(np.bincount(idx.ravel(), minlength=E).astype(np.int64))
    gathered = [torch.zeros(E, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, mine)
    all_counts = torch.stack(gathered).numpy()
    plan = ep.plan_host(all_counts, rank, world)
    inv = ep.rows_of_rank(idx, plan["dest_base"])

    def exchange(payload_of_pair):
        """Sends payload(t, j) of every pair to the owner of its expert, addressed by its destination row."""
        out = [[] for _ in range(world)]
        for t in range(idx.shape[0]):
            for j in range(k):
                out[int(idx[t, j]) // e_loc].append((int(inv[t, j]), payload_of_pair(t, j)))
        box = [None] * world
        dist.all_gather_object(box, out)
        return [item for src in range(world) for item in box[src][rank]]

    # --- dispatch x rows (with their gates) into the owner's padded expert-major buffer
    rows_pad = int(plan["own_pad_offsets"][-1])
    xp = np.zeros((rows_pad, d))
    filled = np.zeros(rows_pad, dtype=bool)
    for r, (row, g) in exchange(lambda t, j: (x[t], float(gates[t, j]))):
        assert not filled[r]
        xp[r], filled[r] = row, True
    # every real row of every owned segment was written exactly once, pad rows never
    for el in range(e_loc):
        p0 = int(plan["own_pad_offsets"][el])
        n = int(plan["own_counts"][el])
        assert filled[p0:p0 + n].all() and not filled[p0 + n:int(plan["own_pad_offsets"][el + 1])].any()
    # --- experts (oracle arithmetic), outputs pulled back by destination row
    o = np.zeros((rows_pad, d))
    hg, hu = np.zeros((rows_pad, f)), np.zeros((rows_pad, f))
    for el in range(e_loc):
        p0, n = int(plan["own_pad_offsets"][el]), int(plan["own_counts"][el])
        hg[p0:p0 + n], hu[p0:p0 + n], _, o[p0:p0 + n] = orc.expert_ffn(xp[p0:p0 + n], Wg[el], Wu[el], Wd[el])
    box = [None] * world
    dist.all_gather_object(box, o)
    y = np.zeros((idx.shape[0], d))
    for t in range(idx.shape[0]):
        for j in range(k):
            y[t] += gates[t, j] * box[int(idx[t, j]) // e_loc][int(inv[t, j])]
    # --- backward of the expert path: g dy rows to the owners, dxp rows back
    d_o = np.zeros((rows_pad, d))
    for r, row in exchange(lambda t, j: gates[t, j] * dy[t]):
        d_o[r] = row
    dxp = np.zeros((rows_pad, d))
    for el in range(e_loc):
        p0, n = int(plan["own_pad_offsets"][el]), int(plan["own_counts"][el])
        s_ = slice(p0, p0 + n)
        da = d_o[s_] @ Wd[el].T
        sg = 1.0 / (1.0 + np.exp(-hg[s_]))
        dhg = da * hu[s_] * sg * (1.0 + hg[s_] * (1.0 - sg))
        dhu = da * hg[s_] * sg
        dxp[s_] = dhg @ Wg[el].T + dhu @ Wu[el].T
    dist.all_gather_object(box, dxp)
    dx_experts = np.zeros((idx.shape[0], d))
    for t in range(idx.shape[0]):
        for j in range(k):
            dx_experts[t] += box[int(idx[t, j]) // e_loc][int(inv[t, j])]
    # --- reference: the oracle on the concatenated batch (every rank can afford it at this size)
    fw = orc.forward(inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"], k)
    bw = orc.backward(fw, inp["dy"], 0.0, inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"])
    dx_router = bw["dl"][sl] @ orc.widen_bf16(inp["W_r"]).T
    ok_rows = all(np.array_equal(xp[int(plan["own_pad_offsets"][el]):int(plan["own_pad_offsets"][el]) + int(plan["own_counts"][el])],
                                 fw["xp"][fw["offsets"][rank * e_loc + el]:fw["offsets"][rank * e_loc + el + 1]])
                  for el in range(e_loc))
    q.put((rank, bool(np.array_equal(idx, fw["idx"][sl])), ok_rows,
           float(np.abs(y - fw["y"][sl]).max()) if tokens[rank] else 0.0,
           float(np.abs(dx_experts + dx_router - bw["dx"][sl]).max()) if tokens[rank] else 0.0,
           float(np.abs(fw["y"]).max())))
    pdist.finish()


import pytest  # noqa: E402


@pytest.mark.parametrize("world", [2, 4])
def test_expert_parallel_exchange_over_gloo_ranks(world):
    """EP group on CPU ranks: after the counts all-gather every rank places its rows inside the owners' buffers; the
    owners' segments come out in the order of the concatenated batch, and y / dx of every rank's tokens equal the
    oracle's on the concatenated batch (routing bit-exact, values to rounding)."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    from paper_2608_00916_b200.dist import free_port
    port = free_port()
    procs = [ctx.Process(target=_ep_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, routing_same, rows_in_order, y_err, dx_err, scale in res:
        assert routing_same and rows_in_order, rank
        assert y_err <= 1e-9 * max(scale, 1.0) and dx_err <= 1e-9, (rank, y_err, dx_err)
