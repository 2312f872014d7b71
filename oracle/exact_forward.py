"""Exact RNN-T sequence probabilities: the textbook forward recursion over the
(frame, token) lattice and a brute-force enumeration of every alignment.
Un-pruned, Algorithm 1 sums exactly these paths (Sec. 3.2: the segment maths
only amounts to summing the paths within a segment that lead to a given token
sequence), whatever the segment size."""
from typing import Sequence

import numpy as np

from . import rnnt_model as rm


def _lattice_log_probs(model: rm.RnntModel, enc: np.ndarray, y: Sequence[int], blank_threshold=None) -> np.ndarray:
    """log J(t, u, .) for every frame t and every prefix length u of y: [T, U+1, V].  With a blank threshold the
    lattice nodes whose blank probability exceeds it keep their blank arc only."""
    outs = []
    state, o = rm.predictor_init(model)
    outs.append(o)
    for k in y:
        state, o = rm.predictor_step(model, state, k)
        outs.append(o)
    logJ = rm.joiner_log_probs(model, np.asarray(enc, dtype=np.float64), np.stack(outs))  # [U+1, T, V]
    if blank_threshold is not None:
        logJ, _ = rm.apply_blank_threshold(logJ, blank_threshold, model.blank)
    return np.transpose(logJ, (1, 0, 2))


def forward_log_prob(model: rm.RnntModel, enc: np.ndarray, y: Sequence[int], blank_threshold=None) -> float:
    """alpha(t, u) = alpha(t-1, u) J(t-1, u, blank) + alpha(t, u-1) J(t, u-1, y_u);
    p(y|x) = alpha(T-1, U) J(T-1, U, blank)   (0-based frames)."""
    lj = _lattice_log_probs(model, enc, y, blank_threshold)
    T, U = lj.shape[0], len(y)
    blank = model.blank
    alpha = np.full((T, U + 1), -np.inf)
    alpha[0, 0] = 0.0
    for t in range(T):
        for u in range(U + 1):
            if t == 0 and u == 0:
                continue
            stay = alpha[t - 1, u] + lj[t - 1, u, blank] if t > 0 else -np.inf
            emit = alpha[t, u - 1] + lj[t, u - 1, y[u - 1]] if u > 0 else -np.inf
            alpha[t, u] = np.logaddexp(stay, emit)
    return float(alpha[T - 1, U] + lj[T - 1, U, blank])


def brute_force_log_prob(model: rm.RnntModel, enc: np.ndarray, y: Sequence[int], blank_threshold=None) -> float:
    """Sum, in the linear domain, over every monotone alignment: from (t, u) a
    blank moves to (t+1, u), token y_{u+1} moves to (t, u+1); an alignment is
    complete when the blank of the last frame has been taken with u = U."""
    lj = _lattice_log_probs(model, enc, y, blank_threshold)
    J = np.exp(lj)
    T, U = J.shape[0], len(y)
    blank = model.blank

    def walk(t: int, u: int, p: float) -> float:
        if t == T:
            return p if u == U else 0.0
        total = walk(t + 1, u, p * J[t, u, blank])
        if u < U:
            total += walk(t, u + 1, p * J[t, u, y[u]])
        return total

    return float(np.log(walk(0, 0, 1.0)))


def forward_log_prob_monotonic(model: rm.RnntModel, enc: np.ndarray, y: Sequence[int]) -> float:
    """Monotonic lattice (every output consumes a frame):
    alpha(t+1, u) = alpha(t, u) J(t, u, blank) + alpha(t, u-1) J(t, u-1, y_u);  p(y|x) = alpha(T, U)."""
    lj = _lattice_log_probs(model, enc, y)
    T, U = lj.shape[0], len(y)
    blank = model.blank
    alpha = np.full((T + 1, U + 1), -np.inf)
    alpha[0, 0] = 0.0
    for t in range(T):
        for u in range(U + 1):
            stay = alpha[t, u] + lj[t, u, blank]
            emit = alpha[t, u - 1] + lj[t, u - 1, y[u - 1]] if u > 0 else -np.inf
            alpha[t + 1, u] = np.logaddexp(stay, emit)
    return float(alpha[T, U])


def brute_force_log_prob_monotonic(model: rm.RnntModel, enc: np.ndarray, y: Sequence[int]) -> float:
    """Sum over every way to place the U tokens on distinct frames, in order; all other frames emit blank."""
    lj = _lattice_log_probs(model, enc, y)
    J = np.exp(lj)
    T, U = J.shape[0], len(y)
    blank = model.blank

    def walk(t: int, u: int, p: float) -> float:
        if t == T:
            return p if u == U else 0.0
        total = walk(t + 1, u, p * J[t, u, blank])
        if u < U:
            total += walk(t + 1, u + 1, p * J[t, u, y[u]])
        return total

    total = walk(0, 0, 1.0)
    return float(np.log(total)) if total > 0.0 else -np.inf
