"""CPU oracle of the listwise training losses on grouped reranker scores.  TEST INFRASTRUCTURE ONLY.

Only the tests may import this file; the product never does, and this file imports nothing from the product.

What it computes (paper, paragraph "Contrastive and distillation losses").  A training step scores G passages per query;
the scores form a matrix s [n, G], one row per query.
* contrastive: the positive passage sits at position 0 of every row and the loss is the listwise cross-entropy of the row
  against that position, averaged over the rows:  L = (1/n) sum_g ( logsumexp(s_g) - s_g[0] ).
* distillation: the student distribution q_g = softmax(s_g / tau_s) is matched to the teacher distribution
  p_g = softmax(t_g / tau_t) of stored teacher scores t [n, G] with the KL divergence KL(p || q), averaged over the rows
  and multiplied by tau_s^2:  L = (tau_s^2 / n) sum_g sum_i p_gi ( log p_gi - log q_gi ).
Both have plain definitions, so the oracle is the definition in float64; the gradient with respect to s is the
derivative of that definition:  contrastive  dL/ds_g = ( softmax(s_g) - e_0 ) / n,   distillation
dL/ds_g = (tau_s / n) ( q_g - p_g )  (the teacher is a constant).

Readings where the paper is silent: the mean runs over the n rows (queries), not over the n G scores; a teacher
probability of exactly zero contributes nothing (0 log 0 = 0); temperatures are positive.

Pins (tests/test_listwise_pins.py): torch.nn.functional.cross_entropy and kl_div on the same numbers, closed forms
(equal scores give log G; a student equal to the teacher at equal temperatures gives 0 and a zero gradient; G = 1 gives
0), invariance under a shift of a row, gradient rows summing to zero, central finite differences in float64.
"""
from __future__ import annotations

import numpy as np


def log_softmax_rows(s: np.ndarray) -> np.ndarray:
    """log softmax over the last axis, the row maximum subtracted first."""
    z = s - s.max(axis=-1, keepdims=True)
    return z - np.log(np.exp(z).sum(axis=-1, keepdims=True))


def contrastive(scores: np.ndarray):
    """Listwise cross-entropy with the positive at position 0.  Returns (loss, dloss/dscores)."""
    s = np.asarray(scores, dtype=np.float64)
    n = s.shape[0]
    if n == 0:
        return 0.0, np.zeros_like(s)
    ls = log_softmax_rows(s)
    loss = float(-ls[:, 0].sum() / n)
    grad = np.exp(ls)
    grad[:, 0] -= 1.0
    return loss, grad / n


def distill(scores: np.ndarray, teacher: np.ndarray, s_temp: float, t_temp: float):
    """Listwise KL(teacher || student) at temperatures (s_temp, t_temp), times s_temp^2.  Returns (loss, dloss/dscores)."""
    s = np.asarray(scores, dtype=np.float64)
    t = np.asarray(teacher, dtype=np.float64)
    n = s.shape[0]
    if n == 0:
        return 0.0, np.zeros_like(s)
    lq = log_softmax_rows(s / s_temp)
    lp = log_softmax_rows(t / t_temp)
    p = np.exp(lp)
    terms = np.where(p > 0, p * (lp - lq), 0.0)
    loss = float(terms.sum() / n * s_temp * s_temp)
    grad = (np.exp(lq) - p) * (s_temp / n)
    return loss, grad
