"""Expert parallelism (EP > 1) on top of the C ABI's moe_ep_* entry points: argument marshalling and the two group
operations the library leaves to its caller (the all-gather of the per-rank expert counts and the barrier between
phases).  Every step of the layer itself - routing, placement, the dispatch of token rows into the owning rank's
buffers, the expert GEMMs, the combine, the backward pass - runs in the CUDA library.

Rank r of `world` owns the experts [r E/world, (r+1) E/world) and keeps its own token batch (paper, Section
"Expert-Parallel MoE Training").  Three layers here:

* placement arithmetic on the host (`plan_host`, `rows_of_rank`): a restatement of what moe_ep_plan / moe_ep_dispatch
  compute on the device, used to check them and by the CPU-rank test of the exchange;
* `EPRank`: one rank's context, workspaces and phase calls;
* `LocalGroup`: all ranks of a group inside ONE process on ONE GPU, phases run rank after rank on one stream (the order
  of the launches is the barrier) - how the path is exercised where only one GPU is available; `DistGroup`: one rank
  per process / GPU with torch.distributed (NCCL all-gather of the counts, symmetric-memory mapping of the owner
  workspaces, a group barrier between phases).
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .binding import MoEConfig, _check, _ptr, load_library

ROW_PAD = 128


# --------------------------------------------------------------------------------------------- host arithmetic
def plan_host(all_counts: np.ndarray, rank: int, world: int) -> dict:
    """Placement of rank `rank`'s rows and the segment table of the experts it owns.

    all_counts[r, e] = rows rank r routes to expert e.  Expert e lives on rank e // (E / world); on its owner the
    segment of e starts at the sum of the 128-row-padded totals of that owner's experts before e, holds the rows of
    rank 0 first, then rank 1, ..., and the rows of one rank in token order.
    Returns dest_base [E] (first row of this rank's rows of expert e inside e's owner buffers), own_counts [E/world],
    own_offsets [E/world + 1] (unpadded) and own_pad_offsets [E/world + 1]."""
    all_counts = np.asarray(all_counts, dtype=np.int64)
    W, E = all_counts.shape
    assert W == world and E % world == 0
    e_loc = E // world
    tot = all_counts.sum(axis=0)
    before = all_counts[:rank].sum(axis=0)
    padded = (tot + ROW_PAD - 1) // ROW_PAD * ROW_PAD
    seg_start = np.zeros(E, dtype=np.int64)
    for o in range(world):
        sl = slice(o * e_loc, (o + 1) * e_loc)
        seg_start[sl] = np.concatenate([[0], np.cumsum(padded[sl])[:-1]])
    own = slice(rank * e_loc, (rank + 1) * e_loc)
    return {"dest_base": (seg_start + before).astype(np.int64), "own_counts": tot[own].copy(),
            "own_offsets": np.concatenate([[0], np.cumsum(tot[own])]),
            "own_pad_offsets": np.concatenate([[0], np.cumsum(padded[own])])}


def rows_of_rank(idx: np.ndarray, dest_base: np.ndarray) -> np.ndarray:
    """inv[t, j]: row, inside the owner's buffers, of the rank's pair (t, j): dest_base of its expert plus the number
    of earlier tokens of this rank that picked the same expert."""
    T, k = idx.shape
    inv = np.empty((T, k), dtype=np.int64)
    seen = np.zeros(dest_base.shape[0], dtype=np.int64)
    for t in range(T):
        for j in range(k):
            e = int(idx[t, j])
            inv[t, j] = dest_base[e] + seen[e]
        for j in range(k):
            seen[int(idx[t, j])] += 1
    return inv


def rows_cap_bound(tokens_per_rank, k: int, E: int, world: int) -> int:
    """Upper bound on the rows any one rank can receive: every token of every rank picks at most min(k, E/world) of
    its experts."""
    return int(sum(tokens_per_rank)) * min(k, E // world)


# --------------------------------------------------------------------------------------------- one rank
class EPRank:
    """Context, workspaces and phase calls of one rank.  Tensors are torch CUDA tensors (carriers of device pointers)."""

    def __init__(self, d: int, E: int, f: int, top_k: int, world: int, rank: int, rows_cap: int, flags: int = 0,
                 own_ws=None):
        import torch
        self.lib = load_library()
        self.d, self.E, self.f, self.k, self.world, self.rank = d, E, f, top_k, world, rank
        self.e_loc = E // world
        cfg = MoEConfig(d, E, f, top_k, flags)
        h = C.c_void_p()
        _check(self.lib, self.lib.moe_ep_create(C.byref(cfg), world, rank, rows_cap, C.byref(h)), "moe_ep_create")
        self.h = h
        self.own_bytes = int(self.lib.moe_ep_own_workspace_bytes(self.h))
        self.own_ws = own_ws if own_ws is not None else torch.empty(max(self.own_bytes, 256), dtype=torch.uint8, device="cuda")
        assert self.own_ws.numel() >= self.own_bytes
        self.send_ws = None
        self.T = None
        self.peers = None

    def __del__(self):
        try:
            if getattr(self, "h", None):
                self.lib.moe_destroy(self.h)
                self.h = None
        except Exception:
            pass

    def set_peers(self, pointers) -> None:
        """pointers[r]: address, in this process, of rank r's owner workspace."""
        assert len(pointers) == self.world
        self.peers = (C.c_void_p * self.world)(*[C.c_void_p(int(p)) for p in pointers])

    def _stream(self):
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def _ensure_send(self, T: int):
        import torch
        need = int(self.lib.moe_ep_send_workspace_bytes(self.h, T))
        if self.send_ws is None or self.send_ws.numel() < need:
            self.send_ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        self.T = T

    def buffer(self, name: str, dtype, own_side: bool):
        off, n = C.c_size_t(), C.c_size_t()
        _check(self.lib, self.lib.moe_ep_workspace_find(self.h, self.T, 1 if own_side else 0, name.encode(), C.byref(off),
                                                        C.byref(n)), f"moe_ep_workspace_find({name})")
        ws = self.own_ws if own_side else self.send_ws
        return ws[off.value:off.value + n.value].view(dtype)

    # ---- phases
    def route(self, x, W_r, b_r=None):
        import torch
        T = x.shape[0]
        self._ensure_send(T)
        out = {"idx": torch.empty(T, self.k, dtype=torch.int32, device=x.device),
               "gates": torch.empty(T, self.k, dtype=torch.float32, device=x.device),
               "counts_local": torch.empty(self.E, dtype=torch.int32, device=x.device),
               "aux": torch.empty(1, dtype=torch.float32, device=x.device)}
        _check(self.lib, self.lib.moe_ep_route(self.h, T, _ptr(x), _ptr(W_r), _ptr(b_r), _ptr(out["idx"]), _ptr(out["gates"]),
                                               _ptr(out["counts_local"]), _ptr(out["aux"]), _ptr(self.send_ws),
                                               self.send_ws.numel(), self._stream()), "moe_ep_route")
        self._x, self._W_r = x, W_r
        return out

    def plan(self, all_counts):
        assert all_counts.dtype.is_floating_point is False and tuple(all_counts.shape) == (self.world, self.E)
        _check(self.lib, self.lib.moe_ep_plan(self.h, self.T, _ptr(all_counts), _ptr(self.send_ws), self.send_ws.numel(),
                                              _ptr(self.own_ws), self.own_ws.numel(), self._stream()), "moe_ep_plan")

    def dispatch(self, src, backward: bool = False):
        _check(self.lib, self.lib.moe_ep_dispatch(self.h, self.T, _ptr(src), 1 if backward else 0, self.peers,
                                                  _ptr(self.send_ws), self.send_ws.numel(), self._stream()), "moe_ep_dispatch")

    def expert_forward(self, W_gate, W_up, W_down):
        for w, shp in ((W_gate, (self.e_loc, self.d, self.f)), (W_up, (self.e_loc, self.d, self.f)),
                       (W_down, (self.e_loc, self.f, self.d))):
            assert tuple(w.shape) == shp and w.is_contiguous()
        _check(self.lib, self.lib.moe_ep_expert_forward(self.h, _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(self.own_ws),
                                                        self.own_ws.numel(), self._stream()), "moe_ep_expert_forward")
        self._W = (W_gate, W_up, W_down)

    def combine(self):
        import torch
        y = torch.empty(self.T, self.d, dtype=torch.bfloat16, device="cuda")
        _check(self.lib, self.lib.moe_ep_combine(self.h, self.T, self.peers, _ptr(self.send_ws), self.send_ws.numel(),
                                                 _ptr(y), self._stream()), "moe_ep_combine")
        return y

    def expert_backward(self, acc=None):
        """acc: dict of fp32 dW_gate / dW_up / dW_down of the owned experts' shapes to ADD the gradients into (the
        main gradients of an accumulation window); None: new bf16 tensors, overwritten."""
        import torch
        W_gate, W_up, W_down = self._W
        if acc is not None:
            for n, w in (("dW_gate", W_gate), ("dW_up", W_up), ("dW_down", W_down)):
                assert acc[n].dtype == torch.float32 and tuple(acc[n].shape) == tuple(w.shape) and acc[n].is_contiguous()
            _check(self.lib, self.lib.moe_ep_expert_backward_accumulate(
                self.h, _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(acc["dW_gate"]), _ptr(acc["dW_up"]), _ptr(acc["dW_down"]),
                _ptr(self.own_ws), self.own_ws.numel(), self._stream()), "moe_ep_expert_backward_accumulate")
            return acc
        out = {"dW_gate": torch.empty_like(W_gate), "dW_up": torch.empty_like(W_up), "dW_down": torch.empty_like(W_down)}
        _check(self.lib, self.lib.moe_ep_expert_backward(self.h, _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(out["dW_gate"]),
                                                         _ptr(out["dW_up"]), _ptr(out["dW_down"]), _ptr(self.own_ws),
                                                         self.own_ws.numel(), self._stream()), "moe_ep_expert_backward")
        return out

    def router_backward(self, d_aux: float, want_db: bool = False):
        import torch
        out = {"dx": torch.empty(self.T, self.d, dtype=torch.bfloat16, device="cuda"),
               "dW_r": torch.empty(self.d, self.E, dtype=torch.float32, device="cuda"),
               "db_r": torch.empty(self.E, dtype=torch.float32, device="cuda") if want_db else None}
        _check(self.lib, self.lib.moe_ep_router_backward(self.h, self.T, C.c_float(d_aux), _ptr(self._x), _ptr(self._W_r),
                                                         self.peers, _ptr(self.send_ws), self.send_ws.numel(), _ptr(out["dx"]),
                                                         _ptr(out["dW_r"]), _ptr(out["db_r"]), self._stream()),
               "moe_ep_router_backward")
        return out

    def poll(self) -> None:
        for ws, what in ((self.send_ws, "sender"), (self.own_ws, "owner")):
            if ws is not None:
                _check(self.lib, self.lib.moe_poll_status(self.h, _ptr(ws), self._stream()), f"device status ({what} workspace)")


# --------------------------------------------------------------------------------------------- groups
class LocalGroup:
    """All ranks of an EP group in one process on one GPU.  Every phase is enqueued for rank 0, 1, ... in turn on the
    current stream, so a phase starts only after the previous phase has finished on every rank: the launch order plays
    the part of the group barrier, no kernel waits for another, and the "peer" pointers are ordinary device pointers.
    The kernels are the ones a multi-GPU group runs."""

    def __init__(self, d, E, f, top_k, world, rows_cap, flags: int = 0):
        self.world = world
        self.ranks = [EPRank(d, E, f, top_k, world, r, rows_cap, flags) for r in range(world)]
        ptrs = [rk.own_ws.data_ptr() for rk in self.ranks]
        for rk in self.ranks:
            rk.set_peers(ptrs)

    def forward(self, xs, W_r, W_gate, W_up, W_down, b_r=None):
        """xs[r]: tokens of rank r; W_gate / W_up / W_down: FULL [E, ...] tensors, sliced per owner here."""
        import torch
        R = self.ranks
        e_loc = R[0].e_loc
        routed = [rk.route(x, W_r, b_r) for rk, x in zip(R, xs)]
        all_counts = torch.stack([o["counts_local"] for o in routed]).contiguous()  # the all-gather of a real group
        for rk in R:
            rk.plan(all_counts)
        for rk, x in zip(R, xs):
            rk.dispatch(x)
        for r, rk in enumerate(R):
            sl = slice(r * e_loc, (r + 1) * e_loc)  # a slice along the leading axis is contiguous: a view, no copy
            rk.expert_forward(W_gate[sl], W_up[sl], W_down[sl])
        ys = [rk.combine() for rk in R]
        return [dict(o, y=y) for o, y in zip(routed, ys)], all_counts

    def backward(self, dys, d_aux: float, want_db: bool = False, acc=None):
        """acc: one dict of fp32 main gradients per rank (see EPRank.expert_backward), or None."""
        R = self.ranks
        for rk, dy in zip(R, dys):
            rk.dispatch(dy, backward=True)
        owner = [rk.expert_backward(None if acc is None else acc[r]) for r, rk in enumerate(R)]
        sender = [rk.router_backward(d_aux, want_db) for rk in R]
        return sender, owner

    def poll(self):
        for rk in self.ranks:
            rk.poll()


class DistGroup:
    """One rank per process and GPU (torch.distributed initialised with the NCCL backend).  The owner workspace lives in
    symmetric memory so that every rank can map its peers' copies; the per-rank expert counts travel by all_gather.
    The group barrier between phases is, by default, the symmetric-memory handle's device-side barrier (a small kernel
    on the current stream in which the ranks signal one another through their signal pads, release / acquire at system
    scope, with the library's own time-out): the stream never drains and the host never waits.  device_barrier=False
    falls back to a host barrier (stream synchronise + dist.barrier).  The tests run both on a one-rank group (they have
    one GPU; LocalGroup runs the same kernels for more ranks there)."""

    def __init__(self, d, E, f, top_k, rows_cap, flags: int = 0, group=None, device_barrier: bool = True):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        self.dist, self.group = dist, group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        probe = EPRank(d, E, f, top_k, self.world, self.rank, rows_cap, flags)
        buf = symm.empty(max(probe.own_bytes, 256), dtype=torch.uint8, device="cuda")
        hdl = symm.rendezvous(buf, group if group is not None else dist.group.WORLD)
        self.rk = EPRank(d, E, f, top_k, self.world, self.rank, rows_cap, flags, own_ws=buf)
        self.rk.set_peers(list(hdl.buffer_ptrs))
        self.hdl = hdl
        self.device_barrier = bool(device_barrier) and hasattr(hdl, "barrier")
        del probe

    def _barrier(self):
        import torch
        if self.device_barrier:
            self.hdl.barrier()  # enqueued on the current stream
            return
        torch.cuda.current_stream().synchronize()
        self.dist.barrier(self.group)

    def forward(self, x, W_r, W_gate_own, W_up_own, W_down_own, b_r=None):
        import torch
        rk = self.rk
        out = rk.route(x, W_r, b_r)
        all_counts = torch.empty(self.world, rk.E, dtype=torch.int32, device=x.device)
        self.dist.all_gather_into_tensor(all_counts, out["counts_local"], group=self.group)
        rk.plan(all_counts)
        self._barrier()
        rk.dispatch(x)
        self._barrier()
        rk.expert_forward(W_gate_own, W_up_own, W_down_own)
        self._barrier()
        out["y"] = rk.combine()
        return out

    def backward(self, dy, d_aux: float, want_db: bool = False, acc=None):
        rk = self.rk
        self._barrier()  # every rank has finished reading the forward outputs it combines
        rk.dispatch(dy, backward=True)
        self._barrier()
        owner = rk.expert_backward(acc)
        self._barrier()
        return rk.router_backward(d_aux, want_db), owner
