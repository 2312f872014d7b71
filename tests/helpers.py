"""Shared test helpers: build oracle models from synthetic tensors."""
import numpy as np

import tw_synth
from oracle import rnnt_model as rm


def oracle_model(m: "tw_synth.SyntheticModel") -> rm.RnntModel:
    return rm.RnntModel(m.W_e, m.W_p, m.W_out, m.b_out, m.emb, m.lstm_W_ih, m.lstm_W_hh, m.lstm_b)


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
