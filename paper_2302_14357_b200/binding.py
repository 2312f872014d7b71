"""ctypes binding of libtw.so.  Names and argument order follow include/tw.h."""
import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

MODE_F32, MODE_BF16 = 0, 1
PRED_STATELESS, PRED_LSTM = 0, 1
ACT_TANH, ACT_RELU = 0, 1
DT_F32, DT_BF16 = 0, 1
NORM_SOFTMAX, NORM_HAT = 0, 1
TW_OK, TW_ERR_ARG, TW_ERR_ALLOC, TW_ERR_CUDA, TW_ERR_LIMIT, TW_ERR_STATE, TW_ERR_TIMEOUT = range(7)

EXPORTED_SYMBOLS = [
    "tw_init", "tw_destroy", "tw_decode", "tw_decode_host", "tw_max_tokens", "tw_project_encoder",
    "tw_joiner_segment", "tw_expand", "tw_joiner_expand", "tw_predictor_step", "tw_get_stats", "tw_set_profiling", "tw_set_fused", "tw_set_graph", "tw_set_lanes", "tw_set_monotonic", "tw_set_inline_gather", "tw_set_blank_threshold",
    "tw_stream_open", "tw_stream_push", "tw_stream_nbest", "tw_stream_close",
    "tw_joiner_expand_noalloc",
    "tw_last_cuda_error", "tw_strerror",
]

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class TwError(RuntimeError):
    def __init__(self, status: int, what: str, cuda: int = 0):
        self.status = status
        self.cuda = cuda
        super().__init__("%s: status %d (%s)%s" % (what, status, _strerror(status), " cudaError %d" % cuda if cuda else ""))


class _Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("D_enc", "P", "J", "V", "blank", "pred_kind", "emb_dim", "lstm_layers", "lstm_hidden", "joiner_act", "dtype", "joiner_norm")] + \
               [(n, C.c_void_p) for n in ("W_e", "W_p", "W_out", "b_out", "emb", "host_lstm_W_ih", "host_lstm_W_hh", "host_lstm_b",
                                          "pred_init_state", "pred_init_out")]


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "S", "mode", "max_batch", "max_T", "max_iters_per_segment", "max_tokens")]


class _Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("frames", "calls", "joins", "steps", "rows", "kernel_launches", "limit_hits", "joiner_frame_rows",
                                          "ns_prologue", "ns_predictor", "ns_joiner", "ns_scan", "ns_hyp", "joiner_launches", "fused_clusters", "fused_on",
                                          "frame_rows_skipped")]


def lib_path() -> str:
    return os.path.join(_PKG_DIR, "libtw.so")


def load_library() -> C.CDLL:
    """Loads libtw.so; raises if it has not been built (python -m paper_2302_14357_b200.build)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError("libtw.so is missing at %s: build it with `python -m paper_2302_14357_b200.build`; "
                           "there is no fallback path" % path)
    lib = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int32
    lib.tw_init.argtypes = [C.POINTER(_Model), C.POINTER(_Config), C.POINTER(vp)]
    lib.tw_destroy.argtypes = [vp]
    lib.tw_decode.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.tw_decode_host.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.tw_max_tokens.argtypes = [vp]
    lib.tw_project_encoder.argtypes = [vp, vp, i32, vp, vp]
    lib.tw_joiner_segment.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, vp]
    lib.tw_expand.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp]
    lib.tw_joiner_expand.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.tw_predictor_step.argtypes = [vp, vp, vp, i32, vp, vp, vp]
    lib.tw_get_stats.argtypes = [vp, C.POINTER(_Stats)]
    lib.tw_set_profiling.argtypes = [vp, C.c_int]
    lib.tw_set_fused.argtypes = [vp, C.c_int]
    lib.tw_set_graph.argtypes = [vp, C.c_int]
    lib.tw_set_lanes.argtypes = [vp, C.c_int]
    lib.tw_set_monotonic.argtypes = [vp, C.c_int]
    lib.tw_set_inline_gather.argtypes = [vp, C.c_int]
    lib.tw_set_blank_threshold.argtypes = [vp, C.c_float]
    lib.tw_stream_open.argtypes = [vp, i32, vp]
    lib.tw_stream_push.argtypes = [vp, vp, vp, i32, vp]
    lib.tw_stream_nbest.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.tw_stream_close.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.tw_joiner_expand_noalloc.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.tw_last_cuda_error.argtypes = [vp]
    lib.tw_strerror.argtypes = [C.c_int]
    lib.tw_strerror.restype = C.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name != "tw_strerror":
            getattr(lib, name).restype = C.c_int
    _LIB = lib
    return lib


def _strerror(status: int) -> str:
    try:
        return load_library().tw_strerror(status).decode()
    except Exception:
        return "?"


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


class TwDecoder:
    """A decoder handle (tw_init .. tw_destroy).  `weights` maps the tw_model field names to arrays or
    tensors ("lstm_W_ih", "lstm_W_hh", "lstm_b" are lists, one per layer; "pred_init_state" and "pred_init_out"
    are optional).  dtype "f32" or "bf16" is the element type in which the weights and, later, the encoder
    frames are handed to the library (tw_model::dtype); values are converted to it here."""

    def __init__(self, weights: Dict, N: int, S: int, mode: int = MODE_F32, max_batch: int = 1, max_T: int = 1,
                 max_iters_per_segment: int = 0, max_tokens: int = 0, blank: int = 0, joiner_act: str = "tanh",
                 dtype: str = "f32", joiner_norm: str = "softmax"):
        import torch
        self._torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("TwDecoder needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", torch.cuda.current_device())

        self.dtype = dtype
        self._tdtype = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]

        def dev(x):
            t = torch.as_tensor(x) if not isinstance(x, np.ndarray) else torch.from_numpy(np.ascontiguousarray(x))
            return t.to(self.device).to(self._tdtype).contiguous()
        weights = dict(weights)
        joiner_act = weights.pop("joiner_act", None) or joiner_act
        joiner_norm = weights.pop("joiner_norm", None) or joiner_norm
        w = {k: ([dev(a) for a in v] if isinstance(v, (list, tuple)) else dev(v)) for k, v in weights.items() if v is not None}
        self._keep = w
        layers = len(w.get("lstm_W_ih", []))
        J, D_enc = w["W_e"].shape
        V = w["W_out"].shape[0]
        P = w["W_p"].shape[1]
        emb_dim = w["emb"].shape[1]
        m = _Model()
        m.D_enc, m.P, m.J, m.V, m.blank = D_enc, P, J, V, blank
        m.pred_kind = PRED_LSTM if layers else PRED_STATELESS
        m.emb_dim, m.lstm_layers = emb_dim, layers
        m.lstm_hidden = w["lstm_W_hh"][0].shape[1] if layers else 0
        m.joiner_act = {"tanh": ACT_TANH, "relu": ACT_RELU}[joiner_act]
        m.dtype = {"f32": DT_F32, "bf16": DT_BF16}[dtype]
        m.joiner_norm = {"softmax": NORM_SOFTMAX, "hat": NORM_HAT}[joiner_norm]
        for name in ("pred_init_state", "pred_init_out"):
            setattr(m, name, w[name].data_ptr() if name in w else None)
        for name in ("W_e", "W_p", "W_out", "b_out", "emb"):
            setattr(m, name, w[name].data_ptr())
        self._tables = []
        for name in ("lstm_W_ih", "lstm_W_hh", "lstm_b"):
            arr = (C.c_void_p * max(layers, 1))(*[t.data_ptr() for t in w.get(name, [])])
            self._tables.append(arr)
            setattr(m, "host_" + name, C.cast(arr, C.c_void_p).value if layers else None)
        c = _Config(N, S, mode, max_batch, max_T, max_iters_per_segment, max_tokens)
        h = C.c_void_p()
        st = self.lib.tw_init(C.byref(m), C.byref(c), C.byref(h))
        if st != TW_OK:
            raise TwError(st, "tw_init")
        self.h = h
        self.N, self.S, self.V, self.J, self.D_enc, self.P = N, S, V, J, D_enc, P
        self.L, self.Hd = layers, m.lstm_hidden
        self.mode = mode
        self.U_cap = self.lib.tw_max_tokens(self.h)
        self.Vp = (V + 255) // 256 * 256      # row pitch of delta_nb on the fused path (vocabulary padded to 256 columns)

    # -- helpers -------------------------------------------------------------------------------
    def _stream(self):
        return self._torch.cuda.current_stream().cuda_stream

    def _check(self, st: int, what: str, allow_limit: bool = False):
        if st == TW_OK or (allow_limit and st == TW_ERR_LIMIT):
            return st
        raise TwError(st, what, self.lib.tw_last_cuda_error(self.h))

    def _f32(self, x):
        return self._torch.as_tensor(x, dtype=self._torch.float32, device=self.device).contiguous()

    def _frames(self, x):
        """Encoder frames on the device in the handle's element type."""
        t = self._torch.as_tensor(x) if not isinstance(x, np.ndarray) else self._torch.from_numpy(np.ascontiguousarray(x))
        return t.to(self.device).to(self._tdtype).contiguous()

    def _i32(self, x):
        return None if x is None else self._torch.as_tensor(x, dtype=self._torch.int32, device=self.device).contiguous()

    def close(self):
        if getattr(self, "h", None):
            self.lib.tw_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the calls of include/tw.h ------------------------------------------------------------
    def decode(self, enc, lengths):
        """tw_decode: enc [B, T, D_enc], lengths [B] -> (tokens, lens, scores, status, rc)."""
        torch = self._torch
        enc, lengths = self._frames(enc), self._i32(lengths)
        B, T = enc.shape[0], enc.shape[1]
        tokens = torch.empty((B, self.N, self.U_cap), dtype=torch.int32, device=self.device)
        lens = torch.empty((B, self.N), dtype=torch.int32, device=self.device)
        scores = torch.empty((B, self.N), dtype=torch.float64, device=self.device)
        status = torch.empty((B,), dtype=torch.int32, device=self.device)
        rc = self.lib.tw_decode(self.h, enc.data_ptr(), lengths.data_ptr(), B, T, tokens.data_ptr(), lens.data_ptr(),
                                scores.data_ptr(), status.data_ptr(), self._stream())
        self._check(rc, "tw_decode", allow_limit=True)
        return tokens, lens, scores, status, rc

    def decode_host(self, enc, lengths: np.ndarray, out=None):
        """tw_decode_host: host buffers in, host buffers out (copies are part of the call).  enc: a float32 numpy
        array, or a CPU torch tensor of the handle's element type (numpy has no bfloat16)."""
        if isinstance(enc, np.ndarray):
            if self.dtype != "f32":
                raise TypeError("a bf16 handle takes its host frames as a torch.bfloat16 CPU tensor")
            enc = np.ascontiguousarray(enc, dtype=np.float32)
            enc_ptr = enc.ctypes.data
        else:
            if enc.dtype != self._tdtype or enc.device.type != "cpu" or not enc.is_contiguous():
                raise TypeError("host frames must be a contiguous CPU tensor of the handle's element type")
            enc_ptr = enc.data_ptr()
        lengths = np.ascontiguousarray(lengths, dtype=np.int32)
        B, T = enc.shape[0], enc.shape[1]
        if out is None:
            out = (np.empty((B, self.N, self.U_cap), np.int32), np.empty((B, self.N), np.int32),
                   np.empty((B, self.N), np.float64), np.empty((B,), np.int32))
        tokens, lens, scores, status = out
        rc = self.lib.tw_decode_host(self.h, enc_ptr, lengths.ctypes.data, B, T, tokens.ctypes.data,
                                     lens.ctypes.data, scores.ctypes.data, status.ctypes.data, self._stream())
        self._check(rc, "tw_decode_host", allow_limit=True)
        return tokens, lens, scores, status, rc

    def _nbest_buffers(self, B):
        torch = self._torch
        return (torch.empty((B, self.N, self.U_cap), dtype=torch.int32, device=self.device),
                torch.empty((B, self.N), dtype=torch.int32, device=self.device),
                torch.empty((B, self.N), dtype=torch.float64, device=self.device),
                torch.empty((B,), dtype=torch.int32, device=self.device))

    def stream_open(self, B: int):
        self._check(self.lib.tw_stream_open(self.h, B, self._stream()), "tw_stream_open")
        self._stream_B = B

    def stream_push(self, enc_chunk, chunk_lens):
        """tw_stream_push: enc_chunk [B, Tc, D_enc], chunk_lens [B] valid frames of the chunk per utterance."""
        enc_chunk, chunk_lens = self._frames(enc_chunk), self._i32(chunk_lens)
        self._check(self.lib.tw_stream_push(self.h, enc_chunk.data_ptr(), chunk_lens.data_ptr(), enc_chunk.shape[1],
                                            self._stream()), "tw_stream_push", allow_limit=True)

    def stream_nbest(self):
        out = self._nbest_buffers(self._stream_B)
        self._check(self.lib.tw_stream_nbest(self.h, *[t.data_ptr() for t in out], self._stream()), "tw_stream_nbest")
        return out

    def stream_close(self):
        out = self._nbest_buffers(self._stream_B)
        rc = self.lib.tw_stream_close(self.h, *[t.data_ptr() for t in out], self._stream())
        self._check(rc, "tw_stream_close", allow_limit=True)
        return out + (rc,)

    def project_encoder(self, enc):
        enc = self._frames(enc).reshape(-1, self.D_enc)
        out = self._torch.empty((enc.shape[0], self.J), dtype=self._torch.float32, device=self.device)
        self._check(self.lib.tw_project_encoder(self.h, enc.data_ptr(), enc.shape[0], out.data_ptr(), self._stream()), "tw_project_encoder")
        return out

    def joiner_segment(self, E_seg, Pp, row_group, seg_len=None):
        E_seg, Pp, row_group, seg_len = self._f32(E_seg), self._f32(Pp), self._i32(row_group), self._i32(seg_len)
        G, R = E_seg.shape[0], Pp.shape[0]
        out = self._torch.empty((R, self.S, self.V), dtype=self._torch.float32, device=self.device)
        self._check(self.lib.tw_joiner_segment(self.h, E_seg.data_ptr(), Pp.data_ptr(), row_group.data_ptr(), _ptr(seg_len),
                                               G, R, out.data_ptr(), self._stream()), "tw_joiner_segment")
        return out

    def _expand_outputs(self, R):
        t = self._torch
        return (t.empty((R,), dtype=t.float32, device=self.device), t.empty((R, self.V), dtype=t.float32, device=self.device),
                t.empty((R, self.S), dtype=t.float32, device=self.device))

    def expand(self, logp, ld_old, seg_len_row=None):
        logp, ld_old, seg_len_row = self._f32(logp), self._f32(ld_old), self._i32(seg_len_row)
        R = ld_old.shape[0]
        ldphi, ldnb, la = self._expand_outputs(R)
        self._check(self.lib.tw_expand(self.h, logp.data_ptr(), ld_old.data_ptr(), _ptr(seg_len_row), R, ldphi.data_ptr(),
                                       ldnb.data_ptr(), la.data_ptr(), self._stream()), "tw_expand")
        return ldphi, ldnb, la

    def joiner_expand(self, E_seg, Pp, row_group, seg_len, ld_old):
        E_seg, Pp, ld_old = self._f32(E_seg), self._f32(Pp), self._f32(ld_old)
        row_group, seg_len = self._i32(row_group), self._i32(seg_len)
        G, R = E_seg.shape[0], Pp.shape[0]
        ldphi, ldnb, la = self._expand_outputs(R)
        self._check(self.lib.tw_joiner_expand(self.h, E_seg.data_ptr(), Pp.data_ptr(), row_group.data_ptr(), _ptr(seg_len),
                                              ld_old.data_ptr(), G, R, ldphi.data_ptr(), ldnb.data_ptr(), la.data_ptr(),
                                              self._stream()), "tw_joiner_expand")
        return ldphi, ldnb, la

    def predictor_step(self, tokens, state_in=None):
        t = self._torch
        tokens = self._i32(tokens)
        R = tokens.shape[0]
        state_out = None
        if self.L:
            state_in = self._f32(state_in)
            state_out = t.empty((R, self.L, 2, self.Hd), dtype=t.float32, device=self.device)
        Pp = t.empty((R, self.J), dtype=t.float32, device=self.device)
        self._check(self.lib.tw_predictor_step(self.h, tokens.data_ptr(), _ptr(state_in), R, _ptr(state_out), Pp.data_ptr(),
                                               self._stream()), "tw_predictor_step")
        return state_out, Pp

    def set_fused(self, on: bool) -> bool:
        """tw_set_fused; returns False when the fused kernel is not available for this handle."""
        return self.lib.tw_set_fused(self.h, int(bool(on))) == TW_OK

    def set_graph(self, on: bool):
        self._check(self.lib.tw_set_graph(self.h, int(bool(on))), "tw_set_graph")

    def set_monotonic(self, on: bool):
        """tw_set_monotonic: the monotonic RNN-T variant (every output consumes a frame) for later decodes."""
        self._check(self.lib.tw_set_monotonic(self.h, int(bool(on))), "tw_set_monotonic")

    def set_inline_gather(self, on: bool):
        """tw_set_inline_gather: who builds the predictor's work list in a fused bf16 decode step."""
        self._check(self.lib.tw_set_inline_gather(self.h, int(bool(on))), "tw_set_inline_gather")

    def set_blank_threshold(self, threshold: float) -> int:
        """tw_set_blank_threshold (factorised-output models only); returns the status."""
        return self.lib.tw_set_blank_threshold(self.h, float(threshold))

    def set_lanes(self, on: bool):
        self._check(self.lib.tw_set_lanes(self.h, int(bool(on))), "tw_set_lanes")

    def set_profiling(self, on: bool):
        self._check(self.lib.tw_set_profiling(self.h, int(bool(on))), "tw_set_profiling")

    def stats(self) -> Dict[str, int]:
        s = _Stats()
        self._check(self.lib.tw_get_stats(self.h, C.byref(s)), "tw_get_stats")
        return {n: getattr(s, n) for n, _ in _Stats._fields_}


def weights_from_synth(m) -> Dict:
    """tw_model fields from a tw_synth.SyntheticModel (plain attribute access, no arithmetic)."""
    return dict(W_e=m.W_e, W_p=m.W_p, W_out=m.W_out, b_out=m.b_out, emb=m.emb,
                lstm_W_ih=list(m.lstm_W_ih), lstm_W_hh=list(m.lstm_W_hh), lstm_b=list(m.lstm_b),
                joiner_act=m.cfg.joiner_act, joiner_norm=getattr(m.cfg, "joiner_norm", "softmax"), pred_init_state=getattr(m, "pred_init_state", None),
                pred_init_out=getattr(m, "pred_init_out", None))


NOALLOC_MAX_ROWS = 4096
NOALLOC_MAX_ELEMS = 4 * 1024 * 1024


def joiner_expand_noalloc(W_out, b_out, S, blank, E_seg, Pp, row_group, seg_len, ld_old, joiner_act="tanh"):
    """tw_joiner_expand_noalloc: joiner + softmax + Eq. 3-7 without a handle and without any device
    allocation inside the library (its scratch is a fixed array in the library image).  All arguments
    are CUDA tensors the caller already owns (float32, int32 for row_group / seg_len); the three
    outputs are allocated here, by the caller's side, before the call.  Returns (status, ldphi, ldnb, la)."""
    import torch
    lib = load_library()
    V, J = W_out.shape
    G, R = E_seg.shape[0], Pp.shape[0]
    dev = W_out.device
    ldphi = torch.empty((R,), dtype=torch.float32, device=dev)
    ldnb = torch.empty((R, V), dtype=torch.float32, device=dev)
    la = torch.empty((R, S), dtype=torch.float32, device=dev)
    act = joiner_act if isinstance(joiner_act, int) else {"tanh": ACT_TANH, "relu": ACT_RELU}[joiner_act]
    st = lib.tw_joiner_expand_noalloc(W_out.data_ptr(), b_out.data_ptr(), J, V, S, blank, act, E_seg.data_ptr(), Pp.data_ptr(),
                                      row_group.data_ptr(), _ptr(seg_len), ld_old.data_ptr(), G, R, ldphi.data_ptr(),
                                      ldnb.data_ptr(), la.data_ptr(), torch.cuda.current_stream().cuda_stream)
    return st, ldphi, ldnb, la
