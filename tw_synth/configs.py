"""Named synthetic workloads, shaped like the RNN-T models the paper decodes
(Sec. 4.1: Emformer encoder output, LSTM predictor, single-layer joiner)."""
from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    batch: int                  # utterances per batch
    T: int                      # maximum encoder frames per utterance
    len_range: Tuple[int, int]  # utterance lengths drawn uniformly (inclusive)
    D_enc: int
    pred_kind: str              # "stateless" | "lstm"
    emb_dim: int
    lstm_layers: int
    lstm_hidden: int
    J: int                      # joiner hidden width
    V: int                      # vocabulary incl. blank (index 0)
    blank_bias: float
    N: int                      # beam
    S_values: Tuple[int, ...]   # segment sizes the workload sweeps
    dtype: str                  # "f32" | "bf16": storage precision of weights/inputs
    seed: int
    joiner_act: str = "tanh"   # "tanh" | "relu"
    joiner_norm: str = "softmax"   # "softmax" | "hat": factorised output, row 0 of W_out is the blank head

    @property
    def P(self) -> int:
        """Predictor output width."""
        return self.emb_dim if self.pred_kind == "stateless" else self.lstm_hidden

    def with_(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


CONFIGS = {
    # tiny, fp32 throughout, stateless predictor
    "c0": WorkloadConfig("c0", 1, 40, (40, 40), 64, "stateless", 64, 0, 0,
                         64, 32, 3.0, 2, (2,), "f32", 0),
    # Librispeech-shaped, variable lengths
    "c1": WorkloadConfig("c1", 32, 400, (200, 400), 512, "lstm", 640, 1, 640,
                         640, 1024, 4.0, 5, (1, 2, 3, 5), "bf16", 1),
    # same model, segment-size sweep
    "c2": WorkloadConfig("c2", 64, 400, (400, 400), 512, "lstm", 640, 1, 640,
                         640, 1024, 4.0, 10, (1, 2, 3, 5, 10, 20, 50), "bf16", 1),
    # large assistant-model shape
    "c3": WorkloadConfig("c3", 128, 600, (600, 600), 1024, "lstm", 1024, 2, 1024,
                         1024, 4096, 4.0, 10, (3,), "bf16", 2),
    # throughput stress on the c3 model
    "c4": WorkloadConfig("c4", 512, 1000, (500, 1000), 1024, "lstm", 1024, 2, 1024,
                         1024, 4096, 4.0, 10, (10,), "bf16", 2),
    # shaped like the paper's Librispeech model (Sec. 4.1): ReLU joiner, 500 sub-word units + blank,
    # 3-layer LSTM predictor; the vocabulary is not a multiple of anything
    "p1": WorkloadConfig("p1", 32, 300, (150, 300), 512, "lstm", 512, 3, 512,
                         512, 501, 4.0, 5, (1, 3, 5), "bf16", 3, "relu"),
    # the Librispeech-shaped model with a factorised (HAT) output for blank thresholding (Sec. 2, Sec. 5): the blank
    # head's bias makes the blank probability about 0.8 on most (hypothesis, frame) pairs
    "h1": WorkloadConfig("h1", 64, 400, (400, 400), 512, "lstm", 640, 1, 640,
                         640, 1024, 1.5, 10, (3,), "bf16", 4, "tanh", "hat"),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]
