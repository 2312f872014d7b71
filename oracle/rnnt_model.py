"""RNN-T model pieces the search calls (Sec. 3.1): joiner j(t,u,k) followed by
softmax normalisation J, and the prediction network g(u).  fp64 throughout.

Joiner form: z = W_out . act(W_e h_t + W_p g_u) + b_out with act = tanh (the synthetic benchmark
workloads) or ReLU (the joiner of the models in Sec. 4.1: one rectified hidden layer, then a linear map to
the vocabulary).
Predictor: either stateless (g = embedding of the last token; the empty
prefix uses the blank token's embedding) or a stack of LSTM layers with gate
order (input, forget, cell, output) and a single bias per layer, started by
feeding the blank token from an all-zero state (InitPredictor, Sec. 3.2).
"""
from typing import List, Optional, Sequence, Tuple

import numpy as np


def _f64(x):
    return np.asarray(x, dtype=np.float64)


class RnntModel:
    def __init__(self, W_e, W_p, W_out, b_out, emb,
                 lstm_W_ih: Sequence = (), lstm_W_hh: Sequence = (), lstm_b: Sequence = (),
                 blank: int = 0, activation: str = "tanh",
                 pred_init_state=None, pred_init_out=None, normalisation: str = "softmax"):
        self.W_e = _f64(W_e)        # [J, D_enc]
        self.W_p = _f64(W_p)        # [J, P]
        self.W_out = _f64(W_out)    # [V, J]
        self.b_out = _f64(b_out)    # [V]
        self.emb = _f64(emb)        # [V, emb_dim]
        self.lstm_W_ih = [_f64(w) for w in lstm_W_ih]   # [4Hd, in]
        self.lstm_W_hh = [_f64(w) for w in lstm_W_hh]   # [4Hd, Hd]
        self.lstm_b = [_f64(b) for b in lstm_b]         # [4Hd]
        self.blank = int(blank)
        assert activation in ("tanh", "relu")
        self.activation = activation
        # "softmax": J = softmax over the whole vocabulary (Sec. 3.1).  "hat": the factorised output that blank
        # thresholding needs (Sec. 2, Sec. 5): the blank logit goes through a sigmoid of its own and the
        # remaining probability is shared out by a softmax over the non-blank tokens.
        assert normalisation in ("softmax", "hat")
        self.normalisation = normalisation
        # InitPredictor() of Sec. 3.2 returns a learned initial state: optional here, as
        # pred_init_state [L, 2, Hd] (per layer h then c) and / or pred_init_out [P]
        self.pred_init_state = None if pred_init_state is None else _f64(pred_init_state)
        self.pred_init_out = None if pred_init_out is None else _f64(pred_init_out)
        self.V = self.W_out.shape[0]
        assert self.W_e.shape[0] == self.W_p.shape[0] == self.W_out.shape[1]
        assert len(self.lstm_W_ih) == len(self.lstm_W_hh) == len(self.lstm_b)

    @property
    def is_lstm(self) -> bool:
        return len(self.lstm_W_ih) > 0


def log_softmax(z: np.ndarray) -> np.ndarray:
    """log J = z - log sum_k exp z_k over the last axis (Sec. 3.1: J is the
    joiner output after softmax normalisation)."""
    m = z.max(axis=-1, keepdims=True)
    return z - (m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True)))


def joiner_log_probs(model: RnntModel, seg: np.ndarray, pred_out: np.ndarray) -> np.ndarray:
    """J = Softmax(Joiner(seg, pred)) of Algorithm 1, in log space.

    seg [S', D_enc] encoder frames, pred_out [H, P] predictor outputs
    -> log J [H, S', V] for every (hypothesis, frame) pair."""
    e = _f64(seg) @ model.W_e.T                     # [S', J]
    p = _f64(pred_out) @ model.W_p.T                # [H, J]
    pre = e[None, :, :] + p[:, None, :]             # [H, S', J]
    hidden = np.tanh(pre) if model.activation == "tanh" else np.maximum(pre, 0.0)
    z = hidden @ model.W_out.T + model.b_out        # [H, S', V]
    if model.normalisation == "hat":
        return log_hat(z, model.blank)
    return log_softmax(z)


def log_hat(z: np.ndarray, blank: int = 0) -> np.ndarray:
    """Factorised output distribution over the last axis, in log space:
      p(blank) = sigmoid(z_blank),   p(k) = (1 - p(blank)) * exp(z_k) / sum_{k' != blank} exp(z_k')   for k != blank."""
    zb = z[..., blank]
    log_pb = -np.logaddexp(0.0, -zb)                # log sigmoid(zb)
    log_rest = -np.logaddexp(0.0, zb)               # log (1 - sigmoid(zb))
    lab = np.delete(z, blank, axis=-1)
    m = lab.max(axis=-1, keepdims=True)
    lse = (m + np.log(np.exp(lab - m).sum(axis=-1, keepdims=True)))[..., 0]
    out = z - lse[..., None] + log_rest[..., None]
    out[..., blank] = log_pb
    return out


def apply_blank_threshold(logJ: np.ndarray, threshold: float, blank: int = 0, flip=None) -> np.ndarray:
    """Blank thresholding (Sec. 2: above a threshold on the blank probability the joiner is not invoked; Sec. 5
    names it as a later extension and prints no equations, so the rule here is this code's reading): at every
    (.., frame) whose blank probability exceeds `threshold` the label part of the output is not computed, i.e.
    the non-blank entries become probability 0 while the blank probability stays what the blank head gave.
    threshold = 1 changes nothing.  logJ [..., V] -> (thresholded copy, boolean mask of the skipped positions).
    `flip`, if given, is called with |log p(blank) - log threshold| per position (row-major order) and returns True
    where that decision is to be inverted."""
    lb = logJ[..., blank]
    with np.errstate(divide="ignore"):
        lt = np.log(threshold)
    skip = lb > lt
    if flip is not None:
        flat = skip.reshape(-1)
        for i, gap in enumerate(np.abs(lb - lt).reshape(-1)):
            if flip(float(gap)):
                flat[i] = not flat[i]
        skip = flat.reshape(skip.shape)
    out = logJ.copy()
    keep_blank = out[..., blank].copy()
    out[skip] = -np.inf
    out[..., blank] = keep_blank
    return out, skip


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


PredState = Optional[Tuple[List[np.ndarray], List[np.ndarray]]]


def lstm_step(model: RnntModel, state: PredState, token: int):
    """One predictor step on `token`.  state = (h[l], c[l]) per layer."""
    h_prev, c_prev = state
    x = model.emb[token]
    h_new, c_new = [], []
    for l in range(len(model.lstm_W_ih)):
        gates = model.lstm_W_ih[l] @ x + model.lstm_W_hh[l] @ h_prev[l] + model.lstm_b[l]
        Hd = gates.shape[0] // 4
        i, f, g, o = (gates[0:Hd], gates[Hd:2 * Hd], gates[2 * Hd:3 * Hd], gates[3 * Hd:4 * Hd])
        c = _sigmoid(f) * c_prev[l] + _sigmoid(i) * np.tanh(g)
        h = _sigmoid(o) * np.tanh(c)
        h_new.append(h)
        c_new.append(c)
        x = h
    return (h_new, c_new), x


def lstm_step_rows(model: RnntModel, h_prev: np.ndarray, c_prev: np.ndarray, tokens: Sequence[int]):
    """The same predictor step as lstm_step for R hypotheses at once (UpdatePredictorOutput of Algorithm 1
    runs the predictor for every new hypothesis; Sec. 4.1: a stack of LSTM layers).
    h_prev, c_prev [R, L, Hd], tokens [R] -> (h_new [R, L, Hd], c_new [R, L, Hd], out [R, Hd])."""
    h_prev, c_prev = _f64(h_prev), _f64(c_prev)
    x = model.emb[np.asarray(tokens, dtype=np.int64)]            # [R, emb_dim]
    h_new, c_new = np.empty_like(h_prev), np.empty_like(c_prev)
    for l in range(len(model.lstm_W_ih)):
        gates = x @ model.lstm_W_ih[l].T + h_prev[:, l] @ model.lstm_W_hh[l].T + model.lstm_b[l]
        Hd = gates.shape[1] // 4
        i, f, g, o = (gates[:, 0:Hd], gates[:, Hd:2 * Hd], gates[:, 2 * Hd:3 * Hd], gates[:, 3 * Hd:4 * Hd])
        c = _sigmoid(f) * c_prev[:, l] + _sigmoid(i) * np.tanh(g)
        h = _sigmoid(o) * np.tanh(c)
        h_new[:, l], c_new[:, l] = h, c
        x = h
    return h_new, c_new, x


def predictor_init(model: RnntModel):
    """InitPredictor(): (state, output) for the empty token prefix.  A model that carries a learned initial
    state (Sec. 3.2) returns it: the state as given (zeros without one), the output as given (the top layer's
    h without one).  Otherwise the blank token's embedding (stateless) or one step on the blank token from an
    all-zero state (LSTM)."""
    if not model.is_lstm:
        if model.pred_init_out is not None:
            return None, model.pred_init_out.copy()
        return None, model.emb[model.blank].copy()
    L = len(model.lstm_W_ih)
    Hd = model.lstm_W_hh[0].shape[1]
    zero = ([np.zeros(Hd) for _ in range(L)], [np.zeros(Hd) for _ in range(L)])
    if model.pred_init_state is not None or model.pred_init_out is not None:
        st = zero
        if model.pred_init_state is not None:
            st = ([model.pred_init_state[l, 0].copy() for l in range(L)], [model.pred_init_state[l, 1].copy() for l in range(L)])
        out = model.pred_init_out.copy() if model.pred_init_out is not None else st[0][L - 1].copy()
        return st, out
    return lstm_step(model, zero, model.blank)


def predictor_step(model: RnntModel, state: PredState, token: int):
    """UpdatePredictorOutput for one hypothesis: (new state, new output)."""
    if not model.is_lstm:
        return None, model.emb[token].copy()
    return lstm_step(model, state, token)


def predictor_for_tokens(model: RnntModel, tokens: Sequence[int]):
    """Predictor output after consuming a whole token prefix."""
    state, o = predictor_init(model)
    for k in tokens:
        state, o = predictor_step(model, state, k)
    return state, o
