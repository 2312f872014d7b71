"""Frame-wise breadth-first RNN-T beam search (Sec. 3.1, Eq. 1): the standard
algorithm the paper generalises.  Written separately from Algorithm 1 (no
segment machinery, dictionary-based merging) so that Algorithm 1 at S=1 can be
checked against it.

Per frame: hypotheses are extended by blank (they are then finished for this
frame) or by a non-blank token (Eq. 1); probabilities of alignments of the
same token sequence are summed; the best N non-blank extensions that beat
the N-th best finished hypothesis stay in the frame; the search moves to the
next frame when none does.
"""
from typing import Dict, Optional, Tuple

import numpy as np

from . import rnnt_model as rm


def standard_beam_search(model: rm.RnntModel, enc: np.ndarray, N: int,
                         max_iters: Optional[int] = None):
    enc = np.asarray(enc, dtype=np.float64)
    blank = model.blank
    # finished[tok] = [log prob, predictor state, predictor output]; dicts keep insertion order
    st0, o0 = rm.predictor_init(model)
    finished: Dict[Tuple[int, ...], list] = {(): [0.0, st0, o0]}
    calls = 0
    for t in range(enc.shape[0]):
        frame = enc[t:t + 1]
        ranked = sorted(enumerate(finished.items()), key=lambda e: (-e[1][1][0], e[0]))[:N]
        active = [(tok, v[0], v[1], v[2]) for _, (tok, v) in ranked]
        finished = {}
        it = 0
        while active:
            if max_iters is not None and it >= max_iters:
                break
            it += 1
            logJ = rm.joiner_log_probs(model, frame, np.stack([a[3] for a in active]))[:, 0, :]
            calls += 1
            # blank extensions end the frame for that hypothesis
            for h, (tok, lp, st, o) in enumerate(active):
                val = lp + logJ[h, blank]
                if tok in finished:
                    finished[tok][0] = float(np.logaddexp(finished[tok][0], val))
                else:
                    finished[tok] = [float(val), st, o]
            # Eq. 1 for every non-blank token
            cands = []
            for h, (tok, lp, st, o) in enumerate(active):
                for k in range(model.V):
                    if k != blank:
                        cands.append((-(lp + logJ[h, k]), h, k))
            cands.sort()
            cands = cands[:N]
            done_scores = sorted((v[0] for v in finished.values()), reverse=True)
            nxt = []
            for neg, h, k in cands:
                if len(done_scores) < N or -neg > done_scores[N - 1]:
                    tok, lp, st, o = active[h]
                    st2, o2 = rm.predictor_step(model, st, k)
                    nxt.append((tok + (k,), -neg, st2, o2))
            active = nxt
    ranked = sorted(enumerate(finished.items()), key=lambda e: (-e[1][1][0], e[0]))[:N]
    return [(tok, v[0]) for _, (tok, v) in ranked], calls


def monotonic_frame_search(model: rm.RnntModel, enc: np.ndarray, N: int):
    """Frame-synchronous beam search for a monotonic RNN-T: at every frame each of the N best
    hypotheses either emits blank or exactly one token, and both consume the frame.  Extensions
    that spell the same sequence are summed; only the N best token extensions of a frame are formed,
    and only those that beat the N-th best blank extension (when there are N) are kept."""
    enc = np.asarray(enc, dtype=np.float64)
    blank = model.blank
    st0, o0 = rm.predictor_init(model)
    beam: Dict[Tuple[int, ...], list] = {(): [0.0, st0, o0]}
    for t in range(enc.shape[0]):
        ranked = sorted(enumerate(beam.items()), key=lambda e: (-e[1][1][0], e[0]))[:N]
        active = [(tok, v[0], v[1], v[2]) for _, (tok, v) in ranked]
        logJ = rm.joiner_log_probs(model, enc[t:t + 1], np.stack([a[3] for a in active]))[:, 0, :]
        beam = {}
        for h, (tok, lp, st, o) in enumerate(active):
            beam[tok] = [float(lp + logJ[h, blank]), st, o]
        cands = sorted((-(lp + logJ[h, k]), h, k) for h, (tok, lp, st, o) in enumerate(active)
                       for k in range(model.V) if k != blank)[:N]
        stay = sorted((v[0] for v in beam.values()), reverse=True)
        for neg, h, k in cands:
            if len(stay) < N or -neg > stay[N - 1]:
                tok, lp, st, o = active[h]
                new = tok + (k,)
                if new in beam:
                    beam[new][0] = float(np.logaddexp(beam[new][0], -neg))
                else:
                    st2, o2 = rm.predictor_step(model, st, k)
                    beam[new] = [-neg, st2, o2]
    ranked = sorted(enumerate(beam.items()), key=lambda e: (-e[1][1][0], e[0]))[:N]
    return [(tok, v[0]) for _, (tok, v) in ranked]
