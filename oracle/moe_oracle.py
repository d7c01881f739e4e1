"""CPU oracle of the MoE FFN layer, forward and backward.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this file; the product
(the CUDA library and its Python binding) never does, and this file imports nothing from the product.

What it computes.  The paper (Section "Expert-Parallel MoE Training") names the layer only: a
Qwen3-30B-A3B-style block with 128 experts and top-8 routing, made of a router weight and per-expert
fc1 / fc2 projections (the LoRA target-group listing).  The layer's result has a plain definition, so
the oracle is that definition written out, one function per step, in the order
router logits -> softmax -> top-k (lowest index wins ties) -> renormalised gates -> expert-major
token permutation -> per-expert SwiGLU FFN -> gate-weighted combine -> auxiliary load-balance loss,
and the backward pass is the chain rule through exactly those steps.  A library matmul (numpy ``@``)
serves as the contraction step; nothing is blocked, fused or reordered.

Precision.  All arithmetic runs in ``dtype`` (float64 by default; float32 is offered because the
acceptance rule describes an fp32 reference and full-size runs are faster with it).  Inputs are the
bf16-rounded tensors widened to ``dtype``; there is no intermediate bf16 rounding.  Routing decisions
are taken on the logits in ``dtype``.

Readings where the paper is silent (all taken from the benchmark spec of the layer):
softmax over all E logits, then top-k, then renormalisation of the k selected probabilities; the
comparison runs on logits; slots are stored in pick order (descending logit, ties ascending index);
an optional additive bias on the logits moves selection and gates alike; SwiGLU experts without
biases; dropless routing (every (token, slot) pair is computed); the gate multiplies at the combine;
the auxiliary loss is E * sum_e f_e * P_e with f_e = c_e / (T k) and P_e the mean full-softmax
probability of expert e, returned without coefficient, and its gradient flows through P_e only.

Pins (tests/test_oracle_pins.py): dense-MLP special cases checked against torch's own silu / matmul,
the all-ties closed form (idx = 0..k-1, gates 1/k, aux = 1), brute-force sorting with hand-made ties,
the permutation identities, expert relabelling, k = E dense mixture, central finite differences in
float64, and gradients from torch autograd through an independently structured dense-mask forward.
No function here is unpinned.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------------------------- inputs
def widen_bf16(bits: np.ndarray, dtype=np.float64) -> np.ndarray:
    """bf16 bit patterns (uint16) -> ``dtype`` (exact).  A floating-point array is taken as values, not bit patterns,
    and only converted to ``dtype`` (the router weight may be given in fp32)."""
    if np.issubdtype(np.asarray(bits).dtype, np.floating):
        return np.asarray(bits).astype(dtype)
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(dtype)


# --------------------------------------------------------------------------------------------- routing
def router_logits(x: np.ndarray, W_r: np.ndarray, b_r=None) -> np.ndarray:
    """l[t,e] = sum_c x[t,c] W_r[c,e] (+ b[e])."""
    l = x @ W_r
    if b_r is not None:
        l = l + b_r.astype(l.dtype)[None, :]
    return l


def softmax_rows(l: np.ndarray) -> np.ndarray:
    """p = softmax(l) over the expert axis, with the row maximum subtracted first."""
    z = np.exp(l - l.max(axis=1, keepdims=True))
    return z / z.sum(axis=1, keepdims=True)


def select_topk(l: np.ndarray, k: int) -> np.ndarray:
    """k rounds per token: take the largest logit not taken yet, the lowest index among equals.
    idx[t, j] is the expert taken in round j."""
    T, E = l.shape
    work = l.copy()
    idx = np.empty((T, k), dtype=np.int32)
    rows = np.arange(T)
    for j in range(k):
        a = np.argmax(work, axis=1)  # first occurrence of the maximum = lowest index
        idx[:, j] = a
        work[rows, a] = -np.inf
    return idx


def gates_from(p: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """g[t,j] = p[t, idx[t,j]] / sum_j' p[t, idx[t,j']]."""
    sel = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    return sel / sel.sum(axis=1, keepdims=True)


def permutation(idx: np.ndarray, E: int):
    """Expert-major order of the routed (token, slot) pairs.

    counts[e] = number of pairs routed to e; offsets = exclusive prefix sum (length E + 1);
    perm[r] = t*k + j of the pair in row r, rows sorted by (expert, token); inv is its inverse."""
    T, k = idx.shape
    flat = idx.reshape(-1).astype(np.int64)
    counts = np.bincount(flat, minlength=E).astype(np.int32)
    offsets = np.zeros(E + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(counts)
    # flat position is t*k + j, so a stable sort on the expert id alone orders by (expert, token, slot);
    # a token takes an expert at most once, hence this is the (expert, token) order.
    perm = np.argsort(flat, kind="stable").astype(np.int32)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.size, dtype=np.int32)
    return counts, offsets, perm, inv


def aux_loss(p: np.ndarray, counts: np.ndarray, k: int):
    """aux = E * sum_e (c_e / (T k)) * ((1/T) sum_t p[t,e])."""
    T, E = p.shape
    f_e = counts.astype(p.dtype) / (T * k)
    P_e = p.sum(axis=0) / T
    return E * float((f_e * P_e).sum())


# --------------------------------------------------------------------------------------------- experts
def silu(h: np.ndarray) -> np.ndarray:
    return h / (1.0 + np.exp(-h))


def expert_ffn(xr: np.ndarray, Wg: np.ndarray, Wu: np.ndarray, Wd: np.ndarray):
    """One expert on its rows: hg = x Wg, hu = x Wu, a = silu(hg) * hu, o = a Wd."""
    hg = xr @ Wg
    hu = xr @ Wu
    a = silu(hg) * hu
    o = a @ Wd
    return hg, hu, a, o


# --------------------------------------------------------------------------------------------- forward
def forward(x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits, k: int, b_r=None, logits_in=None,
            dtype=np.float64, keep: bool = True, expert_weights=None) -> dict:
    """Whole layer.  Arguments are bf16 bit tensors x[T,d], W_r[d,E], W_gate/W_up[E,d,f], W_down[E,f,d].

    ``logits_in`` (float array [T,E]) replaces the router contraction when given, so that ties can be
    constructed by hand.  With ``keep`` the per-row intermediates (in permuted row order) are returned
    for the backward pass and for stage-by-stage comparison.  ``expert_weights(e)`` may supply expert e's
    (W_gate, W_up, W_down) as float arrays instead of the bf16 tensors (used by the low-rank adapter variant)."""
    if expert_weights is None:
        def expert_weights(e):
            return widen_bf16(Wg_bits[e], dtype), widen_bf16(Wu_bits[e], dtype), widen_bf16(Wd_bits[e], dtype)
    x = widen_bf16(x_bits, dtype)
    T, d = x.shape
    E = Wg_bits.shape[0]
    f = Wg_bits.shape[2]
    if logits_in is not None:
        l = np.asarray(logits_in).astype(dtype)
    else:
        l = router_logits(x, widen_bf16(Wr_bits, dtype), b_r)
    p = softmax_rows(l)
    idx = select_topk(l, k)
    g = gates_from(p, idx)
    counts, offsets, perm, inv = permutation(idx, E)
    tok = (perm // k).astype(np.int64)  # token of every permuted row
    slot = (perm % k).astype(np.int64)
    y = np.zeros((T, d), dtype=dtype)
    R = T * k
    if keep:
        hg_all = np.empty((R, f), dtype=dtype)
        hu_all = np.empty((R, f), dtype=dtype)
        a_all = np.empty((R, f), dtype=dtype)
        o_all = np.empty((R, d), dtype=dtype)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        te = tok[r0:r1]
        hg, hu, a, o = expert_ffn(x[te], *expert_weights(e))
        # tokens within one expert are distinct, so this indexed add has no repeated index
        y[te] += g[te, slot[r0:r1]][:, None] * o
        if keep:
            hg_all[r0:r1], hu_all[r0:r1], a_all[r0:r1], o_all[r0:r1] = hg, hu, a, o
    out = {"logits": l, "p": p, "idx": idx, "gates": g, "counts": counts, "offsets": offsets, "perm": perm,
           "inv": inv, "y": y, "aux": aux_loss(p, counts, k), "k": k}
    if keep:
        out.update({"hg": hg_all, "hu": hu_all, "act": a_all, "o": o_all, "xp": x[tok]})
    return out


# --------------------------------------------------------------------------------------------- backward
def backward(fw: dict, dy_bits, d_aux: float, x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits,
             dtype=np.float64, has_bias: bool = False, expert_weights=None) -> dict:
    """Gradients of  L = <y, dy> + d_aux * aux  with the routing choice (idx, counts) held fixed.

    Returns dx[T,d], dW_r[d,E], db_r[E], dW_gate/dW_up[E,d,f], dW_down[E,f,d], plus the intermediates
    dg[T,k], dl[T,E] and the per-row d_o, dhg, dhu, dxp in permuted order."""
    if expert_weights is None:
        def expert_weights(e):
            return widen_bf16(Wg_bits[e], dtype), widen_bf16(Wu_bits[e], dtype), widen_bf16(Wd_bits[e], dtype)
    k = fw["k"]
    x = widen_bf16(x_bits, dtype)
    dy = widen_bf16(dy_bits, dtype)
    W_r = widen_bf16(Wr_bits, dtype)
    T, d = x.shape
    E, _, f = Wg_bits.shape
    idx, g, p, counts, offsets, perm = fw["idx"], fw["gates"], fw["p"], fw["counts"], fw["offsets"], fw["perm"]
    tok = (perm // k).astype(np.int64)
    slot = (perm % k).astype(np.int64)
    R = T * k
    dx = np.zeros((T, d), dtype=dtype)
    dg = np.zeros((T, k), dtype=dtype)
    dWg = np.zeros((E, d, f), dtype=dtype)
    dWu = np.zeros((E, d, f), dtype=dtype)
    dWd = np.zeros((E, f, d), dtype=dtype)
    d_o_all = np.empty((R, d), dtype=dtype)
    dhg_all = np.empty((R, f), dtype=dtype)
    dhu_all = np.empty((R, f), dtype=dtype)
    dxp_all = np.empty((R, d), dtype=dtype)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        te, se = tok[r0:r1], slot[r0:r1]
        Wg, Wu, Wd = expert_weights(e)
        hg, hu, a, o = fw["hg"][r0:r1], fw["hu"][r0:r1], fw["act"][r0:r1], fw["o"][r0:r1]
        # combine: y[t] = sum_j g[t,j] o[t,j]
        dg[te, se] = (dy[te] * o).sum(axis=1)
        d_o = g[te, se][:, None] * dy[te]
        # down projection o = a Wd
        dWd[e] = a.T @ d_o
        da = d_o @ Wd.T
        # a = silu(hg) * hu
        sig = 1.0 / (1.0 + np.exp(-hg))
        dhg = da * hu * sig * (1.0 + hg * (1.0 - sig))
        dhu = da * hg * sig
        # hg = x Wg, hu = x Wu
        dWg[e] = x[te].T @ dhg
        dWu[e] = x[te].T @ dhu
        dxp = dhg @ Wg.T + dhu @ Wu.T
        dx[te] += dxp
        d_o_all[r0:r1], dhg_all[r0:r1], dhu_all[r0:r1], dxp_all[r0:r1] = d_o, dhg, dhu, dxp
    # gates g = softmax over the selected logits: dl_sel[j] = g_j (dg_j - sum_j' g_j' dg_j')
    dl = np.zeros_like(p)
    inner = (g * dg).sum(axis=1, keepdims=True)
    np.put_along_axis(dl, idx.astype(np.int64), g * (dg - inner), axis=1)
    # auxiliary loss through P_e = mean_t p[t,e]; the counts are constants
    dp = d_aux * E * (counts.astype(dtype) / (T * k)) / T  # dL/dp[t,e], same for every t
    dl += p * (dp[None, :] - (p * dp[None, :]).sum(axis=1, keepdims=True))
    dW_r = x.T @ dl
    db_r = dl.sum(axis=0)
    dx += dl @ W_r.T
    return {"dx": dx, "dW_r": dW_r, "db_r": db_r, "dW_gate": dWg, "dW_up": dWu, "dW_down": dWd, "dg": dg,
            "dl": dl, "d_o": d_o_all, "dhg": dhg_all, "dhu": dhu_all, "dxp": dxp_all}


def loss_value(fw: dict, dy_bits, d_aux: float, dtype=np.float64) -> float:
    """The scalar whose gradient ``backward`` returns."""
    dy = widen_bf16(dy_bits, dtype)
    return float((fw["y"] * dy).sum()) + d_aux * fw["aux"]


# --------------------------------------------------------------------------------------------- sampled
def token_rows(t: int, fw_route: dict, x_bits, Wg_bits, Wu_bits, Wd_bits, dtype=np.float64) -> np.ndarray:
    """y[t,:] alone, from the routing of ``fw_route`` (used where the full layer is too large to run)."""
    x = widen_bf16(x_bits[t:t + 1], dtype)
    y = np.zeros(x.shape[1], dtype=dtype)
    for j in range(fw_route["idx"].shape[1]):
        e = int(fw_route["idx"][t, j])
        _, _, _, o = expert_ffn(x, widen_bf16(Wg_bits[e], dtype), widen_bf16(Wu_bits[e], dtype),
                                widen_bf16(Wd_bits[e], dtype))
        y += fw_route["gates"][t, j] * o[0]
    return y


def token_backward(t: int, fw_route: dict, dy_bits, d_aux: float, x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits,
                   dtype=np.float64):
    """dx[t,:] and dl[t,:] alone, from the routing of ``fw_route`` (used where the full layer is too large to run):
    the chain rule through the k experts of token t, its gates, and the auxiliary loss (whose counts come from the
    routing of all tokens)."""
    k = fw_route["idx"].shape[1]
    T, E = fw_route["p"].shape
    x = widen_bf16(x_bits[t:t + 1], dtype)
    dy = widen_bf16(dy_bits[t], dtype)
    g = fw_route["gates"][t]
    dg = np.zeros(k, dtype=dtype)
    dx = np.zeros(x.shape[1], dtype=dtype)
    for j in range(k):
        e = int(fw_route["idx"][t, j])
        Wg, Wu, Wd = widen_bf16(Wg_bits[e], dtype), widen_bf16(Wu_bits[e], dtype), widen_bf16(Wd_bits[e], dtype)
        hg, hu, a, o = expert_ffn(x, Wg, Wu, Wd)
        dg[j] = float(dy @ o[0])
        da = (g[j] * dy) @ Wd.T
        sig = 1.0 / (1.0 + np.exp(-hg[0]))
        dhg = da * hu[0] * sig * (1.0 + hg[0] * (1.0 - sig))
        dhu = da * hg[0] * sig
        dx += dhg @ Wg.T + dhu @ Wu.T
    p = fw_route["p"][t]
    dl = np.zeros(E, dtype=dtype)
    dl[fw_route["idx"][t].astype(np.int64)] = g * (dg - float((g * dg).sum()))
    dp = d_aux * E * (fw_route["counts"].astype(dtype) / (T * k)) / T
    dl += p * (dp - float((p * dp).sum()))
    dx += dl @ widen_bf16(Wr_bits, dtype).T
    return dx, dl


def route_only(x_bits, Wr_bits, k: int, E: int, b_r=None, logits_in=None, dtype=np.float64) -> dict:
    """Routing part of ``forward`` alone (logits, p, idx, gates, counts, offsets, perm, inv, aux)."""
    if logits_in is not None:
        l = np.asarray(logits_in).astype(dtype)
    else:
        l = router_logits(widen_bf16(x_bits, dtype), widen_bf16(Wr_bits, dtype), b_r)
    p = softmax_rows(l)
    idx = select_topk(l, k)
    g = gates_from(p, idx)
    counts, offsets, perm, inv = permutation(idx, E)
    return {"logits": l, "p": p, "idx": idx, "gates": g, "counts": counts, "offsets": offsets, "perm": perm,
            "inv": inv, "aux": aux_loss(p, counts, k), "k": k}


def expert_grads(e: int, fw_route: dict, dy_bits, x_bits, Wg_bits, Wu_bits, Wd_bits, dtype=np.float64):
    """Complete dW_gate[e], dW_up[e], dW_down[e] of one expert from the routing alone."""
    k = fw_route["k"]
    r0, r1 = int(fw_route["offsets"][e]), int(fw_route["offsets"][e + 1])
    d = x_bits.shape[1]
    f = Wg_bits.shape[2]
    if r1 == r0:
        return np.zeros((d, f), dtype), np.zeros((d, f), dtype), np.zeros((f, d), dtype)
    rows = fw_route["perm"][r0:r1].astype(np.int64)
    te, se = rows // k, rows % k
    x = widen_bf16(x_bits[te], dtype)
    dy = widen_bf16(dy_bits[te], dtype)
    Wg, Wu, Wd = widen_bf16(Wg_bits[e], dtype), widen_bf16(Wu_bits[e], dtype), widen_bf16(Wd_bits[e], dtype)
    hg, hu, a, _ = expert_ffn(x, Wg, Wu, Wd)
    d_o = fw_route["gates"][te, se][:, None] * dy
    da = d_o @ Wd.T
    sig = 1.0 / (1.0 + np.exp(-hg))
    dhg = da * hu * sig * (1.0 + hg * (1.0 - sig))
    dhu = da * hg * sig
    return x.T @ dhg, x.T @ dhu, a.T @ d_o


# --------------------------------------------------------------------------------------------- expert LoRA
# Low-rank adapters on the experts' fc1 (gate | up, one shared down-projection A1) and fc2, base weights frozen
# (the paper's "moe_experts" LoRA target group: experts.*.linear_fc1, experts.*.linear_fc2).  By definition the
# adapted layer is the plain layer evaluated with the effective weights
#     W_gate' = W_gate + s A1 B1_gate,   W_up' = W_up + s A1 B1_up,   W_down' = W_down + s A2 B2,
# and the adapter gradients follow from the gradient with respect to the effective weights by the chain rule:
#     dA1 = s (dW_gate' B1_gate^T + dW_up' B1_up^T),  dB1_gate = s A1^T dW_gate',  dB1_up = s A1^T dW_up',
#     dA2 = s dW_down' B2^T,  dB2 = s A2^T dW_down'.
def lora_expert_weights(Wg_bits, Wu_bits, Wd_bits, A1_bits, B1g_bits, B1u_bits, A2_bits, B2_bits, scale, dtype=np.float64):
    def get(e):
        A1 = widen_bf16(A1_bits[e], dtype)
        A2 = widen_bf16(A2_bits[e], dtype)
        return (widen_bf16(Wg_bits[e], dtype) + scale * A1 @ widen_bf16(B1g_bits[e], dtype),
                widen_bf16(Wu_bits[e], dtype) + scale * A1 @ widen_bf16(B1u_bits[e], dtype),
                widen_bf16(Wd_bits[e], dtype) + scale * A2 @ widen_bf16(B2_bits[e], dtype))
    return get


def lora_forward(x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits, A1_bits, B1g_bits, B1u_bits, A2_bits, B2_bits, scale,
                 k: int, b_r=None, dtype=np.float64) -> dict:
    ew = lora_expert_weights(Wg_bits, Wu_bits, Wd_bits, A1_bits, B1g_bits, B1u_bits, A2_bits, B2_bits, scale, dtype)
    return forward(x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits, k, b_r=b_r, dtype=dtype, expert_weights=ew)


def lora_backward(fw: dict, dy_bits, d_aux, x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits, A1_bits, B1g_bits, B1u_bits,
                  A2_bits, B2_bits, scale, dtype=np.float64) -> dict:
    ew = lora_expert_weights(Wg_bits, Wu_bits, Wd_bits, A1_bits, B1g_bits, B1u_bits, A2_bits, B2_bits, scale, dtype)
    bw = backward(fw, dy_bits, d_aux, x_bits, Wr_bits, Wg_bits, Wu_bits, Wd_bits, dtype=dtype, expert_weights=ew)
    E = Wg_bits.shape[0]
    A1, A2 = widen_bf16(A1_bits, dtype), widen_bf16(A2_bits, dtype)
    B1g, B1u, B2 = widen_bf16(B1g_bits, dtype), widen_bf16(B1u_bits, dtype), widen_bf16(B2_bits, dtype)
    out = {"dx": bw["dx"], "dW_r": bw["dW_r"], "db_r": bw["db_r"]}
    out["dA1"] = scale * np.stack([bw["dW_gate"][e] @ B1g[e].T + bw["dW_up"][e] @ B1u[e].T for e in range(E)])
    out["dB1_gate"] = scale * np.stack([A1[e].T @ bw["dW_gate"][e] for e in range(E)])
    out["dB1_up"] = scale * np.stack([A1[e].T @ bw["dW_up"][e] for e in range(E)])
    out["dA2"] = scale * np.stack([bw["dW_down"][e] @ B2[e].T for e in range(E)])
    out["dB2"] = scale * np.stack([A2[e].T @ bw["dW_down"][e] for e in range(E)])
    return out
