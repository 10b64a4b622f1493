"""ctypes front end of the CPU oracle (``wind_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg may import this; the CUDA package never does.  The C file is
compiled on first use with ``gcc -O2 -fopenmp`` into ``oracle/_build/``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wind_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libwind_oracle.so")
_lib = None

f32p = C.POINTER(C.c_float)
f64p = C.POINTER(C.c_double)
i32p = C.POINTER(C.c_int32)
i64p = C.POINTER(C.c_int64)


class OracleModel(C.Structure):
    _fields_ = [
        ("D", C.c_int32), ("E", C.c_int32), ("P", C.c_int32), ("L", C.c_int32),
        ("H", C.c_int32), ("V", C.c_int32), ("blank_id", C.c_int32), ("act", C.c_int32),
        ("emb", f32p),
        ("w_ih", C.POINTER(f32p)), ("w_hh", C.POINTER(f32p)),
        ("b_ih", C.POINTER(f32p)), ("b_hh", C.POINTER(f32p)),
        ("w_enc", f32p), ("b_enc", f32p),
        ("w_pred", f32p), ("b_pred", f32p),
        ("w_out", f32p), ("b_out", f32p),
        ("round_bf16", C.c_int32),
    ]


class OracleStats(C.Structure):
    _fields_ = [
        ("steps", C.c_int64), ("joint_rows", C.c_int64), ("pred_updates", C.c_int64),
        ("forced", C.c_int64), ("low_margin", C.c_int64), ("decisions", C.c_int64),
        ("emit_frames", C.c_int64), ("jump_hist", C.c_int64 * 65),
    ]

    def as_dict(self) -> Dict[str, object]:
        d = {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "jump_hist"}
        d["jump_hist"] = [int(x) for x in self.jump_hist]
        return d


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    if (not force) and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        mp = C.POINTER(OracleModel)
        L.oracle_linear.argtypes = [f32p, f32p, f64p, C.c_int, C.c_int, f64p]
        L.oracle_linear.restype = None
        L.oracle_bf16_round.argtypes = [C.c_double]
        L.oracle_bf16_round.restype = C.c_double
        L.oracle_lstm_step.argtypes = [mp, C.c_int32, f64p, f64p]
        L.oracle_lstm_step.restype = None
        L.oracle_pred_proj.argtypes = [mp, f64p, f64p]
        L.oracle_pred_proj.restype = None
        L.oracle_enc_proj.argtypes = [mp, f32p, C.c_int, f64p]
        L.oracle_enc_proj.restype = None
        L.oracle_joint_logits.argtypes = [mp, f64p, f64p, f64p, f64p]
        L.oracle_joint_logits.restype = None
        L.oracle_decode_seq.argtypes = [mp, f32p, C.c_int32, C.c_int32, C.c_double, i32p, i32p, C.c_int32,
                                        C.POINTER(OracleStats)]
        L.oracle_decode_seq.restype = C.c_int32
        L.oracle_decode_wind.argtypes = [mp, f32p, C.c_int32, C.c_int32, C.c_int32, C.c_double, i32p, i32p,
                                         C.c_int32, C.POINTER(OracleStats)]
        L.oracle_decode_wind.restype = C.c_int32
        L.oracle_decode_batch.argtypes = [mp, f32p, i32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_double,
                                          i32p, i32p, i32p, C.c_int32, C.POINTER(OracleStats)]
        L.oracle_decode_batch.restype = None
        L.oracle_replay_verify.argtypes = [mp, f32p, C.c_int32, C.c_int32, C.c_double, i32p, i32p, C.c_int32,
                                           i64p, i64p, i64p, i32p]
        L.oracle_replay_verify.restype = C.c_int32
        L.oracle_eval_joint_window.argtypes = [mp, f32p, C.c_int32, i32p, C.c_int32, C.c_int32, C.c_int32, f64p,
                                               f64p, f64p, f64p]
        L.oracle_eval_joint_window.restype = C.c_int32
        L.oracle_first_output_logprobs.argtypes = [mp, f32p, C.c_int32, i32p, C.c_int32, C.c_int32, C.c_int32, f64p]
        L.oracle_first_output_logprobs.restype = C.c_int32
        L.oracle_decode_window_greedy_batch.argtypes = L.oracle_decode_batch.argtypes
        L.oracle_decode_window_greedy_batch.restype = None
        L.oracle_replay_verify_window.argtypes = [mp, f32p, C.c_int32, C.c_int32, C.c_int32, C.c_double, i32p, i32p,
                                                  C.c_int32, i64p, i64p, i64p, i32p]
        L.oracle_replay_verify_window.restype = C.c_int32
        L.oracle_beam_search.argtypes = [mp, f32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                         C.c_int32, i32p, i32p, i32p, f64p, f64p, i64p]
        L.oracle_beam_search.restype = C.c_int32
        L.oracle_beam_prefix_step.argtypes = [mp, f32p, C.c_int32, C.c_int32, i32p, i32p, f64p, i32p]
        L.oracle_beam_prefix_step.restype = None
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: np.ndarray, t):
    return a.ctypes.data_as(t)


class Model:
    """Holds fp32 copies of the weights and the C struct that points at them."""

    def __init__(self, w: Dict[str, object], round_bf16: bool = False):
        """round_bf16: enc_proj, the LSTM hidden state and the joint's activations are rounded to bf16 where they are
        produced (the places a bf16 implementation rounds its matrix operands); the default keeps fp64 throughout."""
        self.dims = {k: int(w[k]) for k in ("D", "E", "P", "L", "H", "V", "blank_id", "act")}
        L = self.dims["L"]
        self._keep = []

        def keep(a):
            a = _f32(a)
            self._keep.append(a)
            return _ptr(a, f32p)

        def keep_list(lst: Sequence[np.ndarray]):
            arr = (f32p * L)(*[keep(a) for a in lst])
            self._keep.append(arr)
            return arr

        self.c = OracleModel(
            D=self.dims["D"], E=self.dims["E"], P=self.dims["P"], L=L, H=self.dims["H"], V=self.dims["V"],
            blank_id=self.dims["blank_id"], act=self.dims["act"],
            emb=keep(w["emb"]),
            w_ih=keep_list(w["w_ih"]), w_hh=keep_list(w["w_hh"]),
            b_ih=keep_list(w["b_ih"]), b_hh=keep_list(w["b_hh"]),
            w_enc=keep(w["w_enc"]), b_enc=keep(w["b_enc"]),
            w_pred=keep(w["w_pred"]), b_pred=keep(w["b_pred"]),
            w_out=keep(w["w_out"]), b_out=keep(w["b_out"]),
            round_bf16=int(bool(round_bf16)),
        )

    @property
    def ref(self):
        return C.byref(self.c)


def decode_batch(model: Model, enc: np.ndarray, enc_len: np.ndarray, W: int, S: int,
                 max_out: Optional[int] = None, margin_thr: float = 0.05):
    """W == 0: Algorithm 1 (sequential).  W >= 1: Algorithm 2.  Returns (tokens, frames, out_len, stats)."""
    enc = _f32(enc)
    B, T, D = enc.shape
    assert D == model.dims["D"]
    enc_len = np.ascontiguousarray(enc_len, dtype=np.int32)
    if max_out is None:
        max_out = max(1, T * S)
    tokens = np.full((B, max_out), -1, np.int32)
    frames = np.full((B, max_out), -1, np.int32)
    out_len = np.zeros(B, np.int32)
    st = OracleStats()
    lib().oracle_decode_batch(model.ref, _ptr(enc, f32p), _ptr(enc_len, i32p), B, T, W, S, margin_thr,
                              _ptr(tokens, i32p), _ptr(frames, i32p), _ptr(out_len, i32p), max_out, C.byref(st))
    return tokens, frames, out_len, st.as_dict()


def decode_window_greedy_batch(model: Model, enc: np.ndarray, enc_len: np.ndarray, W: int, S: int,
                               max_out: Optional[int] = None, margin_thr: float = 0.05):
    """Window-based greedy decoding (the best (label, offset) pair of Eq. (1) at every step)."""
    enc = _f32(enc)
    B, T, D = enc.shape
    assert D == model.dims["D"]
    enc_len = np.ascontiguousarray(enc_len, dtype=np.int32)
    if max_out is None:
        max_out = max(1, T * S)
    tokens = np.full((B, max_out), -1, np.int32)
    frames = np.full((B, max_out), -1, np.int32)
    out_len = np.zeros(B, np.int32)
    st = OracleStats()
    lib().oracle_decode_window_greedy_batch(model.ref, _ptr(enc, f32p), _ptr(enc_len, i32p), B, T, W, S, margin_thr,
                                            _ptr(tokens, i32p), _ptr(frames, i32p), _ptr(out_len, i32p), max_out,
                                            C.byref(st))
    return tokens, frames, out_len, st.as_dict()


def beam_search(model: Model, enc_b: np.ndarray, T: int, W: int, K: int, S: int, max_hyps: int = 64,
                max_out: Optional[int] = None, prefix_search: bool = False):
    """Algorithm 3 for one utterance.  Returns (list of (tokens, frames, score) most probable first, min_gap, steps)."""
    enc_b = _f32(enc_b)
    if max_out is None:
        max_out = max(1, int(T) * S)
    tok = np.full((max_hyps, max_out), -1, np.int32)
    frm = np.full((max_hyps, max_out), -1, np.int32)
    ln = np.zeros(max_hyps, np.int32)
    sc = np.zeros(max_hyps, np.float64)
    gap = C.c_double(0.0)
    steps = C.c_int64(0)
    n = lib().oracle_beam_search(model.ref, _ptr(enc_b, f32p), int(T), int(W), int(K), int(S), int(bool(prefix_search)),
                                 max_hyps, max_out,
                                 _ptr(tok, i32p), _ptr(frm, i32p), _ptr(ln, i32p), _ptr(sc, f64p), C.byref(gap),
                                 C.byref(steps))
    assert n >= 0
    hyps = [(tok[a, : ln[a]].copy(), frm[a, : ln[a]].copy(), float(sc[a])) for a in range(n)]
    return hyps, gap.value, steps.value


def beam_prefix_step(model: Model, enc_t: np.ndarray, hyps: Sequence[Sequence[int]], scores: Sequence[float]):
    """Step (2) of Algorithm 3's recombination on its own.  Returns (new scores, removed flags)."""
    enc_t = _f32(enc_t)
    n = len(hyps)
    ml = max(1, max((len(h) for h in hyps), default=1))
    tok = np.zeros((n, ml), np.int32)
    for i, h in enumerate(hyps):
        tok[i, : len(h)] = h
    lens = np.array([len(h) for h in hyps], np.int32)
    sc = np.array(scores, np.float64)
    gone = np.zeros(n, np.int32)
    lib().oracle_beam_prefix_step(model.ref, _ptr(enc_t, f32p), n, ml, _ptr(tok, i32p), _ptr(lens, i32p), _ptr(sc, f64p),
                                  _ptr(gone, i32p))
    return sc, gone.astype(bool)


def replay_verify_window(model: Model, enc_b: np.ndarray, T: int, W: int, S: int, tokens: np.ndarray,
                         frames: np.ndarray, margin_thr: float = 0.05):
    """Check one utterance's (token, frame) list against window-based greedy decoding with the same W and S."""
    enc_b = _f32(enc_b)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    frames = np.ascontiguousarray(frames, dtype=np.int32)
    nd, nl, nn = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    bad = C.c_int32(-1)
    rc = lib().oracle_replay_verify_window(model.ref, _ptr(enc_b, f32p), int(T), int(W), int(S), margin_thr,
                                           _ptr(tokens, i32p), _ptr(frames, i32p), len(tokens),
                                           C.byref(nd), C.byref(nl), C.byref(nn), C.byref(bad))
    return dict(rc=int(rc), decisions=nd.value, low_margin=nl.value, not_argmax=nn.value, bad_pos=bad.value)


def replay_verify(model: Model, enc_b: np.ndarray, T: int, S: int, tokens: np.ndarray, frames: np.ndarray,
                  margin_thr: float = 0.05):
    """Check one utterance's (token, frame) list against the sequential definition.

    Returns dict(rc, decisions, low_margin, not_argmax, bad_pos); rc == 0 means consistent.
    """
    enc_b = _f32(enc_b)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    frames = np.ascontiguousarray(frames, dtype=np.int32)
    nd, nl, nn = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    bad = C.c_int32(-1)
    rc = lib().oracle_replay_verify(model.ref, _ptr(enc_b, f32p), int(T), int(S), margin_thr,
                                    _ptr(tokens, i32p), _ptr(frames, i32p), len(tokens),
                                    C.byref(nd), C.byref(nl), C.byref(nn), C.byref(bad))
    return dict(rc=int(rc), decisions=nd.value, low_margin=nl.value, not_argmax=nn.value, bad_pos=bad.value)


def eval_joint_window(model: Model, enc_b: np.ndarray, T: int, prefix: Sequence[int], t0: int, W: int):
    """Teacher-forced logits [n, V+1] (fp64) at frames t0..t0+n-1, plus pred_proj, h, c."""
    enc_b = _f32(enc_b)
    d = model.dims
    prefix = np.ascontiguousarray(prefix, dtype=np.int32)
    logits = np.zeros((W, d["V"] + 1), np.float64)
    g = np.zeros(d["H"], np.float64)
    h = np.zeros((d["L"], d["P"]), np.float64)
    c = np.zeros((d["L"], d["P"]), np.float64)
    n = lib().oracle_eval_joint_window(model.ref, _ptr(enc_b, f32p), int(T), _ptr(prefix, i32p), len(prefix),
                                       int(t0), int(W), _ptr(logits, f64p), _ptr(g, f64p), _ptr(h, f64p),
                                       _ptr(c, f64p))
    return logits[:n], g, h, c


def first_output_logprobs(model: Model, enc_b: np.ndarray, T: int, prefix: Sequence[int], t0: int, W: int) -> np.ndarray:
    """Eq. (1): log P'(v, t) for the window starting at t0, [n, V+1] fp64 (-inf where P' is zero)."""
    enc_b = _f32(enc_b)
    prefix = np.ascontiguousarray(prefix, dtype=np.int32)
    out = np.zeros((max(W, 1), model.dims["V"] + 1), np.float64)
    n = lib().oracle_first_output_logprobs(model.ref, _ptr(enc_b, f32p), int(T), _ptr(prefix, i32p), len(prefix),
                                           int(t0), int(W), _ptr(out, f64p))
    return out[:n]


def linear(Wm: np.ndarray, b: Optional[np.ndarray], x: np.ndarray) -> np.ndarray:
    Wm = _f32(Wm)
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.zeros(Wm.shape[0], np.float64)
    bp = _ptr(_f32(b), f32p) if b is not None else None
    lib().oracle_linear(_ptr(Wm, f32p), bp, _ptr(x, f64p), Wm.shape[0], Wm.shape[1], _ptr(y, f64p))
    return y


def bf16_round(x: float) -> float:
    """The oracle's own rounding of one value to bf16 (what Model(round_bf16=True) applies)."""
    return float(lib().oracle_bf16_round(float(x)))


def lstm_step(model: Model, tok: int, h: np.ndarray, c: np.ndarray):
    h = np.array(h, dtype=np.float64, order="C")
    c = np.array(c, dtype=np.float64, order="C")
    lib().oracle_lstm_step(model.ref, int(tok), _ptr(h, f64p), _ptr(c, f64p))
    return h, c


def pred_proj(model: Model, h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.float64)
    g = np.zeros(model.dims["H"], np.float64)
    lib().oracle_pred_proj(model.ref, _ptr(h, f64p), _ptr(g, f64p))
    return g


def enc_proj(model: Model, enc_b: np.ndarray) -> np.ndarray:
    enc_b = _f32(enc_b)
    out = np.zeros((enc_b.shape[0], model.dims["H"]), np.float64)
    lib().oracle_enc_proj(model.ref, _ptr(enc_b, f32p), enc_b.shape[0], _ptr(out, f64p))
    return out


def joint_logits(model: Model, encp_row: np.ndarray, g: np.ndarray) -> np.ndarray:
    encp_row = np.ascontiguousarray(encp_row, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    z = np.zeros(model.dims["H"], np.float64)
    out = np.zeros(model.dims["V"] + 1, np.float64)
    lib().oracle_joint_logits(model.ref, _ptr(encp_row, f64p), _ptr(g, f64p), _ptr(z, f64p), _ptr(out, f64p))
    return out
