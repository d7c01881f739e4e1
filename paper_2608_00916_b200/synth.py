"""Seeded synthetic inputs for the MoE FFN layer (shared by the tests, the oracle side and the CUDA side).

This module holds no step of the layer itself.  It draws Gaussian tensors from counter-based
Philox streams keyed by (seed, tensor id, chunk), rounds them to bf16 (round-to-nearest-even),
and *conditions* the draw so that routing is well posed:

* gap guard: a token row of ``x`` is redrawn while two of its k+1 largest router logits
  (evaluated in float64 with a library matmul on the bf16-rounded values) are closer than
  ``1e-4``; the bound is the one the layer's acceptance rule states for bit-exact routing;
* skewed routing: an additive router bias shaped so that expert load follows a
  Zipf(s = 1.2) law, strengthened until several experts are empty and the hottest one holds
  more than ten times the mean load.

The token batches stand in for the hidden states of a reranker training step (8 queries x
8 passages x 256-token query+passage sequences = 16384 tokens, Section "Expert-Parallel MoE
Training" and the training-recipe appendix of the paper); no dataset item is used or needed,
because the layer only ever sees hidden-state shapes.

bf16 tensors are carried as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

GAP = 1e-4  # minimum distance between neighbouring logits among the k+1 largest of a token

# tensor ids of the Philox keys
_TID = {"x": 1, "W_r": 2, "W_gate": 3, "W_up": 4, "W_down": 5, "dy": 6, "x_redraw": 7, "pi": 8,
        "A1": 9, "B1_gate": 10, "B1_up": 11, "A2": 12, "B2": 13}


@dataclasses.dataclass(frozen=True)
class MoEShape:
    T: int  # tokens
    d: int  # model width
    E: int  # experts
    k: int  # experts per token (top_k)
    f: int  # expert width

    @property
    def R(self) -> int:  # routed rows
        return self.T * self.k


# name -> (shape, seed, x_std, skew).  The five benchmark configurations; "sweep_T*" are the
# token-count sweep at the Qwen3-30B-A3B expert shape.
CONFIGS = {
    "tiny": (MoEShape(256, 256, 8, 2, 512), 1000, 0.02, False),
    "qwen": (MoEShape(16384, 2048, 128, 8, 768), 1001, 1.0, False),
    "skewed": (MoEShape(16384, 2048, 128, 8, 768), 1002, 1.0, True),
    "coarse": (MoEShape(16384, 4096, 8, 2, 14336), 1003, 1.0, False),
    # the coarse configuration cut down (a quarter of the tokens and of the expert width, same d, E, k and the same
    # 1024 rows per expert per 4096 tokens) so that a profiler capture holds about 2 GB instead of 12 GB on the device
    "coarse_reduced": (MoEShape(4096, 4096, 8, 2, 3584), 1003, 1.0, False),
    "sweep_T1000": (MoEShape(1000, 2048, 128, 8, 768), 1004, 1.0, False),
    "sweep_T4096": (MoEShape(4096, 2048, 128, 8, 768), 1005, 1.0, False),
    "sweep_T8191": (MoEShape(8191, 2048, 128, 8, 768), 1006, 1.0, False),
    "sweep_T32768": (MoEShape(32768, 2048, 128, 8, 768), 1007, 1.0, False),
    "sweep_T65536": (MoEShape(65536, 2048, 128, 8, 768), 1008, 1.0, False),
}


# ----------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------- draws
def _stream(seed: int, tid: int, chunk: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64(tid) * np.uint64(1 << 32) + np.uint64(chunk)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def normal_bf16(seed: int, name: str, shape: tuple, std: float, threads: int = 8) -> np.ndarray:
    """N(0, std) tensor rounded to bf16.  The leading axis is cut into chunks, each with its own
    Philox key, so the value of a chunk does not depend on how many threads drew the others."""
    tid = _TID[name]
    lead = shape[0]
    rest = int(np.prod(shape[1:], dtype=np.int64)) if len(shape) > 1 else 1
    # chunk rows so that one chunk is about 4M elements
    rows_per_chunk = max(1, min(lead, (1 << 22) // max(rest, 1)))
    out = np.empty((lead, rest), dtype=np.uint16)
    starts = list(range(0, lead, rows_per_chunk))

    def work(ci: int) -> None:
        r0 = starts[ci]
        r1 = min(lead, r0 + rows_per_chunk)
        g = _stream(seed, tid, ci)
        v = g.standard_normal((r1 - r0, rest), dtype=np.float32)
        v *= np.float32(std)
        out[r0:r1] = f32_to_bf16_bits(v)

    if len(starts) > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(len(starts))))
    else:
        for ci in range(len(starts)):
            work(ci)
    return out.reshape(shape)


def _guard_logits(x_bits: np.ndarray, Wr_bits: np.ndarray, b_r) -> np.ndarray:
    """float64 logits used only to condition the draw (gap guard, bias calibration)."""
    l = bf16_bits_to_f64(x_bits) @ bf16_bits_to_f64(Wr_bits)
    if b_r is not None:
        l = l + b_r.astype(np.float64)[None, :]
    return l


def _gap_violations(l: np.ndarray, k: int) -> np.ndarray:
    """Tokens whose k+1 largest logits (k largest when k == E) contain two values closer than GAP."""
    E = l.shape[1]
    m = min(k + 1, E)
    top = -np.sort(-l, axis=1)[:, :m]
    if m < 2:
        return np.zeros(l.shape[0], dtype=bool)
    return (top[:, :-1] - top[:, 1:] < GAP).any(axis=1)


def _load_histogram(l: np.ndarray, k: int) -> np.ndarray:
    E = l.shape[1]
    sel = np.argpartition(-l, min(k, E) - 1, axis=1)[:, :k]
    return np.bincount(sel.ravel(), minlength=E)


def zipf_bias(seed: int, E: int, sigma_l: float, alpha: float, s: float = 1.2) -> np.ndarray:
    """b_e = alpha * sigma_l * ln(q_pi(e) / q_max) with q_r ~ r^-s and pi a seeded permutation."""
    q = np.arange(1, E + 1, dtype=np.float64) ** (-s)
    pi = _stream(seed, _TID["pi"], 0).permutation(E)
    b = alpha * sigma_l * np.log(q[pi] / q.max())
    return b.astype(np.float32)


def _guard_tokens(x: np.ndarray, W_r: np.ndarray, b_r, k: int, seed: int, x_std: float) -> int:
    """Redraws (in place) the token rows of x that violate the gap guard against router (W_r, b_r); returns how many
    rows were redrawn in total."""
    redrawn = 0
    d = x.shape[1]
    for attempt in range(64):
        l = _guard_logits(x, W_r, b_r)
        bad = np.nonzero(_gap_violations(l, k))[0]
        if bad.size == 0:
            return redrawn
        g = _stream(seed, _TID["x_redraw"], attempt)
        v = g.standard_normal((bad.size, d), dtype=np.float32) * np.float32(x_std)
        x[bad] = f32_to_bf16_bits(v)
        redrawn += int(bad.size)
    raise RuntimeError("gap guard did not converge")


def make_tokens(shape: MoEShape, seed: int, W_r: np.ndarray, b_r=None, x_std: float = 1.0, guard: bool = True,
                threads: int = 8) -> dict:
    """A token batch (x, dy) of its own seed for a router that is given: the batch of a data-parallel rank, whose
    tokens must keep the gap guard against the weights every rank shares."""
    x = normal_bf16(seed, "x", (shape.T, shape.d), x_std, threads)
    redrawn = _guard_tokens(x, W_r, b_r, shape.k, seed, x_std) if (guard and shape.T > 0) else 0
    return {"x": x, "dy": normal_bf16(seed, "dy", (shape.T, shape.d), 1.0, threads), "redrawn": redrawn}


def make_inputs(shape: MoEShape, seed: int, x_std: float = 1.0, skew: bool = False, w_std: float = 0.02,
                guard: bool = True, threads: int = 8) -> dict:
    """Draw one problem instance.

    Returns a dict with bf16 bit tensors ``x [T,d]``, ``W_r [d,E]``, ``W_gate [E,d,f]``, ``W_up [E,d,f]``,
    ``W_down [E,f,d]``, ``dy [T,d]``, the float32 router bias ``b_r [E]`` (or None), ``d_aux`` and ``meta``
    (redraw count, bias strength, realised expert-load histogram of the guard logits).
    """
    T, d, E, k, f = shape.T, shape.d, shape.E, shape.k, shape.f
    W_r = normal_bf16(seed, "W_r", (d, E), w_std, threads)
    x = normal_bf16(seed, "x", (T, d), x_std, threads)
    meta = {"shape": dataclasses.asdict(shape), "seed": seed, "x_std": x_std, "skew": skew, "redrawn": 0,
            "alpha": None, "stands_in_for": "reranker hidden states (8 queries x 8 passages x 256 tokens)"}
    b_r = None
    if skew:
        l0 = _guard_logits(x, W_r, None)
        sigma_l = float(l0.std())
        alpha = 1.1
        while True:
            b_r = zipf_bias(seed, E, sigma_l, alpha)
            h = _load_histogram(l0 + b_r.astype(np.float64)[None, :], k)
            if ((h == 0).sum() >= 3 and h.max() >= 10.0 * h.mean()) or alpha > 4.0:
                break
            alpha = round(alpha + 0.1, 10)
        meta["alpha"] = alpha
        meta["sigma_l"] = sigma_l
    if guard and T > 0:
        meta["redrawn"] = _guard_tokens(x, W_r, b_r, k, seed, x_std)
        meta["histogram"] = _load_histogram(_guard_logits(x, W_r, b_r), k).tolist() if E <= 256 else None
    out = {
        "x": x, "W_r": W_r, "b_r": b_r,
        "W_gate": normal_bf16(seed, "W_gate", (E, d, f), w_std, threads),
        "W_up": normal_bf16(seed, "W_up", (E, d, f), w_std, threads),
        "W_down": normal_bf16(seed, "W_down", (E, f, d), w_std, threads),
        "dy": normal_bf16(seed, "dy", (T, d), 1.0, threads),
        "d_aux": 0.01,
        "meta": meta,
    }
    return out


def make_config(name: str, **overrides) -> dict:
    shape, seed, x_std, skew = CONFIGS[name]
    return make_inputs(shape, seed, x_std=x_std, skew=skew, **overrides)


def make_lora(shape: MoEShape, seed: int, rank: int = 16, std: float = 0.05, threads: int = 8) -> dict:
    """Rank-`rank` adapters for the experts' fc1 (A1 [E,d,r], B1_gate / B1_up [E,r,f]) and fc2 (A2 [E,f,r],
    B2 [E,r,d]), all N(0, std) in bf16 (a trained state: in a fresh adapter the B matrices would be zero)."""
    E, d, f = shape.E, shape.d, shape.f
    return {"A1": normal_bf16(seed, "A1", (E, d, rank), std, threads),
            "B1_gate": normal_bf16(seed, "B1_gate", (E, rank, f), std, threads),
            "B1_up": normal_bf16(seed, "B1_up", (E, rank, f), std, threads),
            "A2": normal_bf16(seed, "A2", (E, f, rank), std, threads),
            "B2": normal_bf16(seed, "B2", (E, rank, d), std, threads), "rank": rank}
