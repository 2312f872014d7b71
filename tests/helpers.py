"""Shared test helpers: build oracle models from synthetic tensors."""
import numpy as np

import tw_synth
from oracle import rnnt_model as rm


def oracle_model(m: "tw_synth.SyntheticModel") -> rm.RnntModel:
    return rm.RnntModel(m.W_e, m.W_p, m.W_out, m.b_out, m.emb, m.lstm_W_ih, m.lstm_W_hh, m.lstm_b,
                        activation=m.cfg.joiner_act, pred_init_state=m.pred_init_state, pred_init_out=m.pred_init_out,
                        normalisation=getattr(m.cfg, "joiner_norm", "softmax"))


def tiny_config(V=4, T=4, pred="stateless", seed=7, D_enc=5, J=6, emb=3, hidden=4, layers=1,
                blank_bias=1.0, N=2, S=2):
    return tw_synth.WorkloadConfig(
        name="tiny", batch=1, T=T, len_range=(T, T), D_enc=D_enc, pred_kind=pred, emb_dim=emb,
        lstm_layers=layers if pred == "lstm" else 0, lstm_hidden=hidden if pred == "lstm" else 0,
        J=J, V=V, blank_bias=blank_bias, N=N, S_values=(S,), dtype="f32", seed=seed)


def tiny_case(**kw):
    cfg = tiny_config(**kw)
    m = tw_synth.make_model(cfg)
    enc, _ = tw_synth.make_encoder_batch(cfg)
    # scale the logits up so that token probabilities differ clearly
    m.W_out *= 3.0
    return cfg, oracle_model(m), enc[0].astype(np.float64)


# ------------------------------------------------------------------------------------------------
# N-best comparison with the near-tie protocol
SCORE_TOL = 1e-4      # absolute tolerance on log-scores (fp32 mode)
TIE_TAU = 2e-5        # a pruning decision with a smaller score gap may legitimately flip in fp32


def _same_nbest(ref, got, tol, tau):
    """ref, got: lists of (tokens, score), best first.  Sequences must be the same set with scores
    within tol; the order must match except between neighbours closer than tau."""
    if len(ref) != len(got):
        return False
    gd = dict(got)
    if len(gd) != len(got) or set(gd) != set(t for t, _ in ref):
        return False
    for tok, s in ref:
        if not abs(gd[tok] - s) <= tol:
            return False
    for i, (tok, s) in enumerate(ref):
        if got[i][0] != tok:
            j = [t for t, _ in got].index(tok)
            if abs(ref[j][1] - s) > tau + 2 * tol:
                return False
    return True


def check_against_oracle(model, enc, N, S, max_iters, got, tol=SCORE_TOL, tau=TIE_TAU, max_flips=6, monotonic=False,
                         blank_threshold=None):
    """Runs Algorithm 1 in the oracle and compares with `got`.  Returns (ok, how, stats) where how is
    'exact' or 'near-tie' (the oracle reproduces `got` after inverting one or two pruning decisions
    whose score gap is below tau)."""
    import itertools
    from oracle import token_wise_search as tws
    log = tws.DecisionLog()
    ref, stats = tws.token_wise_beam_search(model, enc, N, S, max_iters=max_iters, log=log, monotonic=monotonic,
                                            blank_threshold=blank_threshold)
    if _same_nbest(ref, got, tol, tau):
        return True, "exact", stats
    close = log.below(tau)[:max_flips]
    for n in (1, 2):
        for flips in itertools.combinations(close, n):
            ref2, _ = tws.token_wise_beam_search(model, enc, N, S, max_iters=max_iters, log=tws.DecisionLog(flips),
                                                 monotonic=monotonic, blank_threshold=blank_threshold)
            if _same_nbest(ref2, got, tol, tau):
                return True, "near-tie", stats
    return False, "mismatch: oracle %r vs %r (min margin %.3g)" % (ref[:2], got[:2], log.min_margin()), stats


def nbest_from_arrays(tokens, lens, scores, b):
    out = []
    for i in range(lens.shape[1]):
        n = int(lens[b, i])
        if n >= 0:
            out.append((tuple(int(x) for x in tokens[b, i, :n]), float(scores[b, i])))
    return out
