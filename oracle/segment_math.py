"""Eq. 3-7: aggregated emission probabilities over a segment of S' frames, in
natural-log space and written as the explicit sums the equations state.
Frames t1, t2 are 1-based as in the paper; arrays carry an unused index 0."""
import numpy as np

NEG_INF = -np.inf


def logsumexp(a: np.ndarray, axis: int) -> np.ndarray:
    """log sum exp along `axis`; an all -inf slice gives -inf (log 0)."""
    a = np.asarray(a, dtype=np.float64)
    m = a.max(axis=axis, keepdims=True)
    safe = np.where(np.isfinite(m), m, 0.0)
    with np.errstate(divide="ignore"):
        out = safe + np.log(np.exp(a - safe).sum(axis=axis, keepdims=True))
    return np.squeeze(out, axis=axis)


def blank_product(logJ: np.ndarray, blank: int = 0) -> np.ndarray:
    """Eq. 3.  logJ [H, S', V] -> log Bl [H, S'+1, S'+2] indexed [h, t1, t2],
    t1 in 1..S', t2 in 1..S'+1:
      t1 <  t2: sum_{t'=t1}^{t2-1} log J(t', h, blank)
      t1 == t2: 0        t1 > t2: -inf."""
    H, S, _ = logJ.shape
    lBl = np.full((H, S + 1, S + 2), NEG_INF)
    for t1 in range(1, S + 1):
        for t2 in range(1, S + 2):
            if t1 < t2:
                acc = np.zeros(H)
                for tp in range(t1, t2):
                    acc = acc + logJ[:, tp - 1, blank]
                lBl[:, t1, t2] = acc
            elif t1 == t2:
                lBl[:, t1, t2] = 0.0
    return lBl


def nonblank_expansion_t(logJ: np.ndarray, lBl: np.ndarray, ld_old: np.ndarray, blank: int = 0) -> np.ndarray:
    """Eq. 4-5.  ld_old [H, S'] = log p(y_1..y_U(t1)) -> log d [H, V, S'] with
    d[h, k, t2] = sum_{t1=1}^{S'} d_old[h, t1] * Bl(h, t1, t2) * J(t2, h, k).
    The blank column is not an expansion token and is set to -inf."""
    H, S, V = logJ.shape
    ld = np.full((H, V, S), NEG_INF)
    for t2 in range(1, S + 1):
        terms = np.full((S, H, V), NEG_INF)
        for t1 in range(1, S + 1):
            # Eq. 4: p(y(t1), y_{U+1}(t2)) = p(y(t1)) * Bl(t1, t2) * J(t2, y_{U+1})
            terms[t1 - 1] = (ld_old[:, t1 - 1] + lBl[:, t1, t2])[:, None] + logJ[:, t2 - 1, :]
        ld[:, :, t2 - 1] = logsumexp(terms, axis=0)      # Eq. 5: sum over t1
    ld[:, blank, :] = NEG_INF
    return ld


def nonblank_expansion(ld: np.ndarray) -> np.ndarray:
    """Eq. 6.  delta_nb[h, k] = sum_{t2} d[h, k, t2]."""
    return logsumexp(ld, axis=2)


def blank_expansion(lBl: np.ndarray, ld_old: np.ndarray) -> np.ndarray:
    """Eq. 7.  delta_phi[h] = sum_{t1} d_old[h, t1] * Bl(h, t1, S'+1)."""
    H, S = ld_old.shape
    terms = np.stack([ld_old[:, t1 - 1] + lBl[:, t1, S + 1] for t1 in range(1, S + 1)], axis=0)
    return logsumexp(terms, axis=0)


# ---- monotonic variant (Sec. 2 and Sec. 5 name it as an easy adjustment; the equations below are this
# code's own derivation, pinned by brute force in the tests) --------------------------------------
# In a monotonic RNN-T every output, blank or token, consumes one frame.  A hypothesis that emits
# token k at frame t2 therefore continues at frame t2 + 1, and one that emits at the segment's last
# frame has left the segment.  Frame distributions get one more entry, index S'+1: "past the segment".


def nonblank_expansion_t_monotonic(logJ: np.ndarray, lBl: np.ndarray, ld_old: np.ndarray, blank: int = 0) -> np.ndarray:
    """Monotonic Eq. 4-5.  ld_old [H, S'+1] -> log d [H, V, S'+1] with
    d[h, k, t2 + 1] = sum_{t1=1}^{S'} d_old[h, t1] * Bl(h, t1, t2) * J(t2, h, k)   for t2 = 1..S',
    d[h, k, 1] = 0.  Mass already past the segment (d_old[h, S'+1]) cannot emit here."""
    H, S, V = logJ.shape
    assert ld_old.shape == (H, S + 1)
    ld = np.full((H, V, S + 1), NEG_INF)
    for t2 in range(1, S + 1):
        terms = np.full((S, H, V), NEG_INF)
        for t1 in range(1, S + 1):
            terms[t1 - 1] = (ld_old[:, t1 - 1] + lBl[:, t1, t2])[:, None] + logJ[:, t2 - 1, :]
        ld[:, :, t2] = logsumexp(terms, axis=0)          # lands on frame t2 + 1 (array index t2)
    ld[:, blank, :] = NEG_INF
    return ld


def blank_expansion_monotonic(lBl: np.ndarray, ld_old: np.ndarray) -> np.ndarray:
    """Monotonic Eq. 7.  delta_phi[h] = sum_{t1=1}^{S'} d_old[h, t1] * Bl(h, t1, S'+1) + d_old[h, S'+1]."""
    H, S1 = ld_old.shape
    S = S1 - 1
    terms = [ld_old[:, t1 - 1] + lBl[:, t1, S + 1] for t1 in range(1, S + 1)]
    terms.append(ld_old[:, S])
    return logsumexp(np.stack(terms, axis=0), axis=0)
