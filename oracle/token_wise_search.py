"""Algorithm 1: token-wise beam search for RNN-T, one utterance, fp64 log space.

`token_wise_beam_search` takes the steps of Algorithm 1 in the order the paper gives them and with its
names (lists A and B, ChooseNBest, AddAndMerge, ChooseNthScore, ChooseNBestExpansions,
UpdatePredictorOutput), so that it can be checked against the algorithm by eye; the code is written
from the algorithm's description, with Eq. 3-7 taken from segment_math.

Readings of points the paper leaves open (each mirrored by the CUDA path):
  * last segment when S does not divide the length: seg = enc[t:t+S] is a
    slice, so the final segment is simply shorter (S' = len - t);
  * ChooseNBest / ChooseNthScore / ChooseNBestExpansions order by score
    descending; equal scores fall back to insertion order (lists) or to the
    smaller hypothesis index, then the smaller token id (expansions);
  * expansions are over non-blank tokens only (Eq. 6 is defined for a new
    non-blank token);
  * the filter is the strict '>' Algorithm 1 prints, and is bypassed while
    Length(B) < N;
  * the inner loop has a safety cap `max_iters` per segment (the paper relies
    on the threshold alone); hitting it drops the rest of A and is reported;
  * merged hypotheses keep the predictor state of the entry inserted first;
  * an expansion of probability zero (log score -inf) is not a hypothesis and is
    never kept (it only arises in the monotonic variant, from a hypothesis whose
    whole mass has already left the segment).

`monotonic=True` runs the same loop for a monotonic RNN-T (every output consumes a
frame): frame distributions carry one more entry for "past the segment" and the
two monotonic formulas of segment_math replace Eq. 4-5 and Eq. 7.

`DecisionLog` records the score margin of every pruning decision and can
invert chosen ones, so a test can tell a legitimate near-tie flip of a lower
precision implementation from a real disagreement.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import rnnt_model as rm
from . import segment_math as sm

NEG_INF = -np.inf


class DecisionLog:
    """Margins of all cut decisions, numbered in the order they are taken."""

    def __init__(self, flips: Sequence[int] = ()):
        self.flips = set(int(i) for i in flips)
        self.margins: List[Tuple[int, str, float]] = []

    def decide(self, kind: str, margin: float) -> bool:
        """Log a decision with |score gap| `margin`; True if it must be inverted."""
        idx = len(self.margins)
        self.margins.append((idx, kind, float(margin)))
        return idx in self.flips

    def min_margin(self) -> float:
        return min((m for _, _, m in self.margins), default=np.inf)

    def below(self, tau: float) -> List[int]:
        return [i for i, _, m in self.margins if m < tau]


@dataclass
class Hypothesis:
    tok: Tuple[int, ...]
    ls: float                    # log score s
    state: rm.PredState          # predictor recurrent state
    o: Optional[np.ndarray]      # predictor output
    ld: Optional[np.ndarray]     # log of d: last-token frame distribution over the segment


@dataclass
class SearchStats:
    frames: int = 0
    calls: int = 0               # joiner invocations (Calls/Frame numerator)
    joins: int = 0               # frames fed to the joiner (Joins/Frame numerator)
    frame_rows: int = 0          # (hypothesis, frame) pairs fed to the joiner
    skipped: int = 0             # of those, pairs whose label part blank thresholding left out
    limit_hit: bool = False
    iters_per_segment: List[int] = field(default_factory=list)


def _ordered_top(scores: Sequence[float], n: int, log: Optional[DecisionLog], kind: str) -> List[int]:
    """Indices of the n highest scores, best first; ties keep list order."""
    order = sorted(range(len(scores)), key=lambda i: (-scores[i], i))
    if len(order) > n:
        if log is not None and n >= 1:
            # a cut below which everything has probability zero is no decision: its margin is infinite
            gap = scores[order[n - 1]] - scores[order[n]] if scores[order[n]] > NEG_INF else np.inf
            if log.decide(kind, gap):
                order[n - 1], order[n] = order[n], order[n - 1]
        order = order[:n]
    return order


def choose_n_best(hyps: List[Hypothesis], n: int, log=None, kind="nbest") -> List[Hypothesis]:
    return [hyps[i] for i in _ordered_top([h.ls for h in hyps], n, log, kind)]


def add_and_merge(B: List[Hypothesis], hyp: Hypothesis) -> bool:
    """Append hyp to B; if B already holds the same tokens, sum the scores."""
    for e in B:
        if e.tok == hyp.tok:
            e.ls = float(np.logaddexp(e.ls, hyp.ls))
            return True
    B.append(hyp)
    return False


def choose_nth_score(B: List[Hypothesis], n: int) -> float:
    return sorted((h.ls for h in B), reverse=True)[n - 1]


def choose_n_best_expansions(ldnb: np.ndarray, n: int, blank: int, log=None) -> List[Tuple[int, int]]:
    """Top-n (h, k) pairs, k != blank, by delta_nb; ties -> smaller h, then k."""
    H, V = ldnb.shape
    pairs = [(h, k) for h in range(H) for k in range(V) if k != blank]
    flat = [ldnb[h, k] for h, k in pairs]
    # a partial sort keeps this affordable at V in the thousands
    if len(flat) > 4 * n + 8:
        arr = np.asarray(flat)
        keep = np.argpartition(-arr, 2 * n + 4)[: 2 * n + 4]
        cut = arr[keep].min()
        keep = sorted(i for i in range(len(flat)) if flat[i] >= cut)
        pairs = [pairs[i] for i in keep]
        flat = [flat[i] for i in keep]
    return [pairs[i] for i in _ordered_top(flat, n, log, "expansion")]


def token_wise_beam_search(model: rm.RnntModel, enc: np.ndarray, N: int, S: int,
                           max_iters: Optional[int] = None,
                           max_len: Optional[int] = None,
                           log: Optional[DecisionLog] = None,
                           monotonic: bool = False,
                           blank_threshold: Optional[float] = None):
    """Algorithm 1.  enc [T, D_enc] -> (list of (tokens, log score) best first, stats).

    max_iters: safety cap on inner-loop passes per segment (None = uncapped).
    max_len:   test-only cap on hypothesis length; longer expansions are never
               created (used to make the un-pruned search finite).
    blank_threshold: blank thresholding for a model with the factorised output (rnnt_model.apply_blank_threshold):
               (hypothesis, frame) pairs whose blank probability exceeds it contribute their blank
               probability only; stats.skipped counts them.  None or 1: plain Algorithm 1."""
    enc = np.asarray(enc, dtype=np.float64)
    T = enc.shape[0]
    blank = model.blank
    stats = SearchStats(frames=T)

    state0, o0 = rm.predictor_init(model)
    B: List[Hypothesis] = [Hypothesis((), 0.0, state0, o0, None)]
    t = 0
    while t < T:
        seg = enc[t:t + S]
        Sp = seg.shape[0]
        A = choose_n_best(B, N, log, "segment_start")
        B = []
        t = t + S
        for hyp in A:
            ld = np.full(Sp + 1 if monotonic else Sp, NEG_INF)
            ld[0] = hyp.ls                       # all mass on the segment's first frame
            hyp.ld = ld
        it = 0
        while len(A) > 0:
            if max_iters is not None and it >= max_iters:
                stats.limit_hit = True
                break
            it += 1
            pred = np.stack([hyp.o for hyp in A])
            logJ = rm.joiner_log_probs(model, seg, pred)          # [H, S', V]
            stats.calls += 1
            stats.joins += Sp
            stats.frame_rows += Sp * len(A)
            if blank_threshold is not None:
                flip = (lambda gap: log.decide("skip", gap)) if log is not None else None
                logJ, skipped = rm.apply_blank_threshold(logJ, blank_threshold, blank, flip)
                stats.skipped += int(skipped.sum())

            ld_old = np.stack([hyp.ld for hyp in A])              # [H, S']
            lBl = sm.blank_product(logJ, blank)                   # Eq. 3
            if monotonic:
                ld_new = sm.nonblank_expansion_t_monotonic(logJ, lBl, ld_old, blank)
                ldphi = sm.blank_expansion_monotonic(lBl, ld_old)
            else:
                ld_new = sm.nonblank_expansion_t(logJ, lBl, ld_old, blank)  # Eq. 4-5
                ldphi = sm.blank_expansion(lBl, ld_old)           # Eq. 7
            ldnb = sm.nonblank_expansion(ld_new)                  # Eq. 6

            for h, hyp in enumerate(A):
                add_and_merge(B, Hypothesis(hyp.tok, float(ldphi[h]), hyp.state, hyp.o, None))

            A_prev = A
            A = []
            threshold = choose_nth_score(B, N) if len(B) >= N else None
            for (h, k) in choose_n_best_expansions(ldnb, N, blank, log):
                score = float(ldnb[h, k])
                if score == NEG_INF:
                    continue
                if max_len is not None and len(A_prev[h].tok) + 1 > max_len:
                    continue
                if len(B) < N:
                    keep = True
                else:
                    keep = score > threshold
                    if log is not None and log.decide("threshold", abs(score - threshold)):
                        keep = not keep
                if keep:
                    A.append(Hypothesis(A_prev[h].tok + (k,), score, A_prev[h].state, None,
                                        ld_new[h, k, :].copy()))
            for hyp in A:                                         # UpdatePredictorOutput
                hyp.state, hyp.o = rm.predictor_step(model, hyp.state, hyp.tok[-1])
        stats.iters_per_segment.append(it)

    final = choose_n_best(B, N, log, "final")
    return [(hyp.tok, hyp.ls) for hyp in final], stats
