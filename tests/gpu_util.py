"""Helpers shared by the GPU parity tests: tensor transport and stage-by-stage comparison with the oracle."""
import numpy as np
import torch

from oracle import moe_oracle as orc
from paper_2608_00916_b200.binding import MoELayer


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def from_dev_bf16(t: torch.Tensor) -> np.ndarray:
    """bf16 CUDA tensor -> float64 numpy"""
    return t.float().cpu().numpy().astype(np.float64)


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref.astype(np.float64).ravel())
    num = np.linalg.norm(got.astype(np.float64).ravel() - ref.astype(np.float64).ravel())
    return float(num / den) if den > 0 else float(num)


def rows_max_err(got: np.ndarray, ref: np.ndarray) -> float:
    """Largest error of any single row: max_r |got_r - ref_r| / max(|ref_r|, rms_r' |ref_r'|) (2-norms over the last
    axis).  A whole-tensor norm hides a wrong row among thousands; this does not.  Each row is measured against its own
    size, except that rows much smaller than the typical row are measured against the typical row (their rounding
    errors are set by the operands, not by their own cancelled sum)."""
    got = got.astype(np.float64).reshape(-1, got.shape[-1])
    ref = ref.astype(np.float64).reshape(-1, ref.shape[-1])
    if ref.shape[0] == 0:
        return 0.0
    num = np.linalg.norm(got - ref, axis=1)
    own = np.linalg.norm(ref, axis=1)
    rms = np.sqrt(np.mean(own * own))
    den = np.maximum(own, rms)
    if rms == 0:
        return float(num.max())
    return float((num / den).max())


ROW_TOL = 3e-2  # bound on rows_max_err: about ten bf16 roundings' worth, far below the O(1) of a wrong row


class Run:
    """Runs the CUDA layer on an instance from synth.make_inputs and keeps the device tensors."""

    def __init__(self, inp: dict, k: int, logits_in=None, flags: int = 0):
        self.inp = inp
        T, d = inp["x"].shape
        E, _, f = inp["W_gate"].shape
        self.T, self.d, self.E, self.f, self.k = T, d, E, f, k
        self.layer = MoELayer(d, E, f, k, flags)
        self.dev = {n: to_dev_bf16(inp[n]) for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
        self.b_r = None if inp.get("b_r") is None else torch.from_numpy(inp["b_r"]).cuda()
        self.logits_in = None if logits_in is None else torch.from_numpy(np.ascontiguousarray(logits_in, np.float32)).cuda()
        self.fw = None
        self.bw = None

    def forward(self):
        v = self.dev
        self.fw = self.layer.forward(v["x"], v["W_r"], v["W_gate"], v["W_up"], v["W_down"], b_r=self.b_r,
                                     logits_in=self.logits_in, want_logits=True)
        self.layer.poll()
        return self.fw

    def backward(self, d_aux: float, want_db=True):
        self.bw = self.layer.backward(self.dev["dy"], d_aux, want_db=want_db)
        self.layer.poll()
        return self.bw

    # internal buffers -------------------------------------------------------------
    def ints(self, name):
        return self.layer.buffer(name, torch.int32).cpu().numpy()

    def rows(self, name, width):
        """Internal padded row buffer -> canonical (unpadded, expert-major) rows as float64, plus the pad rows."""
        buf = self.layer.buffer(name, torch.bfloat16).view(-1, width)
        off = self.ints("offsets").astype(np.int64)
        pad = self.ints("pad_offsets").astype(np.int64)
        R = int(off[-1])
        src = np.empty(R, dtype=np.int64)
        is_pad = np.ones(int(pad[-1]), dtype=bool)
        for e in range(self.E):
            n = int(off[e + 1] - off[e])
            src[off[e]:off[e + 1]] = pad[e] + np.arange(n)
            is_pad[pad[e]:pad[e] + n] = False
        full = buf[: int(pad[-1])].float().cpu().numpy().astype(np.float64)
        return full[src], full[is_pad]


def oracle_run(inp, k, d_aux, logits_in=None, dtype=np.float64):
    fw = orc.forward(inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"], k, b_r=inp.get("b_r"),
                     logits_in=logits_in, dtype=dtype)
    bw = orc.backward(fw, inp["dy"], d_aux, inp["x"], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"],
                      dtype=dtype)
    return fw, bw
