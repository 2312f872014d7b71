"""Seeded tensors for a synthetic RNN-T: weights ~ N(0, 1/fan_in), embedding
rows ~ N(0, 1), encoder frames ~ N(0, 1), LSTM biases zero, output bias zero
except the blank entry.  Every tensor has its own Philox stream keyed by
(seed, tensor id), so a tensor's values do not depend on which other tensors
were drawn.  Values are float32; the "bf16" workloads round them to the
nearest bfloat16 (ties to even) and keep them in float32 storage."""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from .configs import WorkloadConfig

_TENSOR_IDS = {
    "W_e": 1, "W_p": 2, "W_out": 3, "emb": 4, "enc": 5, "lengths": 6,
    "lstm_W_ih": 16, "lstm_W_hh": 32,
}


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(tensor_id)]))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float32 values to bfloat16, returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def _normal(seed, tid, shape, std, dtype):
    w = _rng(seed, tid).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        w *= np.float32(std)
    if dtype == "bf16":
        w = round_to_bf16(w)
    return w


@dataclass
class SyntheticModel:
    cfg: WorkloadConfig
    W_e: np.ndarray            # [J, D_enc]
    W_p: np.ndarray            # [J, P]
    W_out: np.ndarray          # [V, J]
    b_out: np.ndarray          # [V]
    emb: np.ndarray            # [V, emb_dim]
    lstm_W_ih: List[np.ndarray] = field(default_factory=list)  # [4*Hd, in]
    lstm_W_hh: List[np.ndarray] = field(default_factory=list)  # [4*Hd, Hd]
    lstm_b: List[np.ndarray] = field(default_factory=list)     # [4*Hd]
    # a learned InitPredictor() result, when a test or a caller supplies one (the generators draw none)
    pred_init_state: Optional[np.ndarray] = None   # [L, 2, Hd]
    pred_init_out: Optional[np.ndarray] = None     # [P]


def make_model(cfg: WorkloadConfig) -> SyntheticModel:
    s, dt = cfg.seed, cfg.dtype
    P = cfg.P
    m = SyntheticModel(
        cfg=cfg,
        W_e=_normal(s, _TENSOR_IDS["W_e"], (cfg.J, cfg.D_enc), cfg.D_enc ** -0.5, dt),
        W_p=_normal(s, _TENSOR_IDS["W_p"], (cfg.J, P), P ** -0.5, dt),
        W_out=_normal(s, _TENSOR_IDS["W_out"], (cfg.V, cfg.J), cfg.J ** -0.5, dt),
        b_out=np.zeros(cfg.V, dtype=np.float32),
        emb=_normal(s, _TENSOR_IDS["emb"], (cfg.V, cfg.emb_dim), 1.0, dt),
    )
    m.b_out[0] = cfg.blank_bias
    if cfg.pred_kind == "lstm":
        Hd = cfg.lstm_hidden
        for l in range(cfg.lstm_layers):
            fan_in = cfg.emb_dim if l == 0 else Hd
            m.lstm_W_ih.append(_normal(s, _TENSOR_IDS["lstm_W_ih"] + l, (4 * Hd, fan_in), fan_in ** -0.5, dt))
            m.lstm_W_hh.append(_normal(s, _TENSOR_IDS["lstm_W_hh"] + l, (4 * Hd, Hd), Hd ** -0.5, dt))
            m.lstm_b.append(np.zeros(4 * Hd, dtype=np.float32))
    return m


def make_encoder_batch(cfg: WorkloadConfig, batch: Optional[int] = None):
    """Returns (enc [B, T, D_enc] float32, lengths [B] int32).  Frames past an
    utterance's length are still drawn (and must be ignored by a decoder)."""
    B = cfg.batch if batch is None else batch
    lo, hi = cfg.len_range
    lengths = _rng(cfg.seed, _TENSOR_IDS["lengths"]).integers(lo, hi + 1, size=cfg.batch).astype(np.int32)[:B]
    if B > cfg.batch:
        raise ValueError("batch exceeds the workload's batch")
    enc = _rng(cfg.seed, _TENSOR_IDS["enc"]).standard_normal(size=(B, cfg.T, cfg.D_enc), dtype=np.float32)
    if cfg.dtype == "bf16":
        enc = round_to_bf16(enc)
    return enc, lengths
