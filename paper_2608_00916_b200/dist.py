"""Multi-GPU plumbing for the benchmark: one process per GPU, data parallel over tokens.

The layer shards over tokens with the experts replicated (expert-parallel degree 1), so the data path needs
no collective; torch.distributed only provides the barrier around the timed region and the max-over-ranks
reduction of its duration.  Works with the gloo backend on CPU (tests) and nccl on GPUs."""
from __future__ import annotations

import os

_state = {"world": 1, "rank": 0, "backend": None}


def init(world: int, rank: int, backend: str = "nccl") -> None:
    _state.update(world=world, rank=rank, backend=backend)
    if world <= 1:
        return
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)


def shard_seed(seed: int, rank: int) -> int:
    """Seed of the token batch drawn by `rank`; rank 0 keeps the workload's own seed."""
    return seed + 7919 * rank


def rank_environment(rank: int, world: int, port: int, base_env=None) -> dict:
    """Environment of rank `rank` of a one-node job: what torch.distributed's env:// rendezvous and bench.py read."""
    env = dict(os.environ if base_env is None else base_env)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), LOCAL_WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    env.setdefault("NCCL_DEBUG", "INFO")  # leaves the communicator's transport line (NVLS or not) in the log
    return env


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n: int, script: str, argv, port: int | None = None, python: str | None = None, timeout=None) -> int:
    """Starts `n` copies of `python script argv...`, one per rank (rank r is meant for GPU r), waits for all of them
    and returns the first non-zero exit code (0 if none).  Rank 0 inherits stdout; the other ranks' stdout is dropped
    (they print nothing by contract), every rank keeps stderr."""
    import subprocess
    import sys
    port = free_port() if port is None else port
    procs = []
    for r in range(n):
        procs.append(subprocess.Popen([python or sys.executable, script, *argv], env=rank_environment(r, n, port),
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        try:
            code = p.wait(timeout=timeout)
        except subprocess.TimeoutExpired:
            p.kill()  # exactly the process started here
            code = 124
        rc = rc or code
    return rc


def barrier() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        if _state["backend"] == "nccl":
            import torch
            dist.barrier(device_ids=[torch.cuda.current_device()])  # the rank's own GPU, not a guess from the rank number
        else:
            dist.barrier()


def max_over_ranks(value: float) -> float:
    if _state["world"] <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if _state["backend"] == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if _state["world"] <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if _state["backend"] == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(tokens_this_rank: int, ms_this_rank: float) -> float:
    """Whole-job tokens/s: tokens of all ranks over the slowest rank's time."""
    total = sum_over_ranks(tokens_this_rank)
    ms = max_over_ranks(ms_this_rank)
    return total / (ms / 1e3)


class GradAllReducer:
    """Sums the weight-gradient buffers of the data-parallel ranks (the one exchange step of the sharded layer: tokens
    are split over the ranks, experts are replicated, so dW_gate / dW_up / dW_down / dW_r must be added up).

    Two ways to start the reduction of the fp32 buffers filled by MoELayer.backward_accumulate:

    * start_grouped(acc, events): for a backward pass that ran with `group_events=events` (see events()).  The library
      records an event as soon as a range of experts has its final dW_down (then dW_gate / dW_up); the communication
      stream waits for exactly that event and all-reduces the range's slab, so the reduction of the first ranges runs
      while the later weight-gradient launches, the dgrad GEMM between them and the router's chain are still
      computing.  dW_r, which is complete only at the end of the pass, goes last.
    * start(tensors): whole buffers, cut along the expert axis into buckets, after everything has been enqueued (the
      reduction then overlaps only what follows the backward pass).  Also the form for CPU tensors (gloo).

    wait() joins before the optimizer reads the buffers.  With one rank both are no-ops unless a `reduce_fn` is given
    (tests inject one to watch the stream plumbing on a single GPU)."""

    def __init__(self, experts_per_bucket: int = 16, n_groups: int = 4, reduce_fn=None):
        self.experts_per_bucket = max(1, int(experts_per_bucket))
        self.n_groups = max(1, int(n_groups))
        self.reduce_fn = reduce_fn
        self._work = []
        self._side = None
        self._done = None
        self._events = None

    def _active(self) -> bool:
        return _state["world"] > 1 or self.reduce_fn is not None

    def _reduce(self, t):
        if self.reduce_fn is not None:
            return self.reduce_fn(t)
        import torch.distributed as dist
        return dist.all_reduce(t, op=dist.ReduceOp.SUM, async_op=True)

    def buckets(self, tensors):
        """(tensor, first expert, last expert + 1) slices in launch order; tensors without an expert axis (dW_r) last."""
        out = []
        for t in tensors:
            if t.dim() == 3:
                for e0 in range(0, t.shape[0], self.experts_per_bucket):
                    out.append((t, e0, min(t.shape[0], e0 + self.experts_per_bucket)))
        for t in tensors:
            if t.dim() != 3:
                out.append((t, 0, t.shape[0]))
        return out

    def group_ranges(self, E: int):
        """Expert ranges of the grouped backward pass: n_groups ranges of ceil(E / n_groups) experts (the last may be
        shorter or empty), the split moe_backward_accumulate_grouped uses."""
        per = (E + self.n_groups - 1) // self.n_groups
        return [(min(E, g * per), min(E, (g + 1) * per)) for g in range(self.n_groups)]

    def events(self):
        """The 2 n_groups CUDA events to hand to MoELayer.backward_accumulate(..., group_events=...)."""
        import torch
        if self._events is None:
            self._events = [torch.cuda.Event() for _ in range(2 * self.n_groups)]
        return self._events

    def start_grouped(self, acc: dict) -> None:
        """acc: the dict given to backward_accumulate (dW_gate, dW_up, dW_down, dW_r)."""
        if not self._active():
            return
        import torch
        if self._side is None:
            self._side = torch.cuda.Stream()
        ev = self.events()
        n = self.n_groups
        ranges = self.group_ranges(acc["dW_down"].shape[0])
        tail = torch.cuda.Event()
        tail.record(torch.cuda.current_stream())  # everything of the pass, dW_r included, has been enqueued
        with torch.cuda.stream(self._side):
            for g, (e0, e1) in enumerate(ranges):
                self._side.wait_event(ev[g])
                if e1 > e0:
                    self._work.append(self._reduce(acc["dW_down"][e0:e1]))
            for g, (e0, e1) in enumerate(ranges):
                self._side.wait_event(ev[n + g])
                if e1 > e0:
                    self._work.append(self._reduce(acc["dW_gate"][e0:e1]))
                    self._work.append(self._reduce(acc["dW_up"][e0:e1]))
            self._side.wait_event(tail)
            self._work.append(self._reduce(acc["dW_r"]))
            self._done = torch.cuda.Event()
            self._done.record(self._side)

    def start(self, tensors) -> None:
        if not self._active():
            return
        import torch
        on_cuda = tensors[0].is_cuda
        if on_cuda:
            if self._side is None:
                self._side = torch.cuda.Stream()
            ev = torch.cuda.Event()
            ev.record(torch.cuda.current_stream())
            self._side.wait_event(ev)
        ctx = torch.cuda.stream(self._side) if on_cuda else _NullCtx()
        with ctx:
            for t, e0, e1 in self.buckets(tensors):
                self._work.append(self._reduce(t[e0:e1]))
            if on_cuda:
                self._done = torch.cuda.Event()
                self._done.record(self._side)

    def wait(self) -> None:
        import torch
        for w in self._work:
            if w is not None:
                w.wait()
        self._work = []
        if self._done is not None:
            torch.cuda.current_stream().wait_event(self._done)
            self._done = None


class _NullCtx:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def finish() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
