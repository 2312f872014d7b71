"""Token-wise RNN-T beam search (Algorithm 1) on NVIDIA B200.

Thin Python binding over the C-ABI library libtw.so (see include/tw.h): every
step of the search runs in the library's CUDA kernels; this package only
marshals arguments.  There is no CPU fallback: importing `binding` without the
built library raises.
"""
from .binding import (TwDecoder, TwError, load_library, lib_path, MODE_F32, MODE_BF16,
                      PRED_STATELESS, PRED_LSTM, EXPORTED_SYMBOLS)

__all__ = ["TwDecoder", "TwError", "load_library", "lib_path", "MODE_F32", "MODE_BF16",
           "PRED_STATELESS", "PRED_LSTM", "EXPORTED_SYMBOLS"]
