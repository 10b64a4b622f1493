"""Thin ctypes binding of ``libwind_b200.so`` (declared in ``include/wind.h``).

Argument marshalling only: every step of the decoding path runs inside the
library's CUDA kernels.  PyTorch is used for device memory and streams.  There
is no CPU fallback: if the shared library is missing or no CUDA device is
present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwind_b200.so")

WIND_OK = 0
WIND_ERR_INVALID_ARG = 1
WIND_ERR_UNSUPPORTED = 2
WIND_ERR_CUDA = 3
WIND_ERR_OUTPUT_OVERFLOW = 4
WIND_ERR_TIMEOUT = 5
WIND_ERR_INTERNAL = 6
WIND_ERR_WORKSPACE = 7
WIND_ACT_RELU, WIND_ACT_TANH = 0, 1
WIND_DT_F32, WIND_DT_BF16 = 0, 1
WIND_KERNELS_AUTO, WIND_KERNELS_SIMT, WIND_KERNELS_TENSOR = 0, 1, 2

EXPORTS = [
    "wind_workspace_bytes", "wind_decode_greedy", "wind_decode_window_greedy", "wind_host_staging_bytes", "wind_decode_greedy_host",
    "wind_eval_joint_window", "wind_window_first_output", "wind_eval_joint_window_static", "wind_profile_decode", "wind_beam_workspace_bytes", "wind_beam_search", "wind_plan_batches", "wind_read_stats", "wind_set_trace", "wind_read_trace", "wind_debug_stall_barrier", "wind_set_kernels", "wind_status_string", "wind_last_cuda_error",
    "wind_set_loop_options", "wind_debug_plan", "wind_bench_joint", "wind_refill_workspace_bytes", "wind_decode_greedy_refill",
]

_vp = C.c_void_p


class wind_model_t(C.Structure):
    _fields_ = [
        ("D", C.c_int32), ("E", C.c_int32), ("P", C.c_int32), ("L", C.c_int32), ("H", C.c_int32), ("V", C.c_int32),
        ("blank_id", C.c_int32), ("act", C.c_int32), ("dtype", C.c_int32), ("reserved", C.c_int32),
        ("emb", _vp), ("w_ih", C.POINTER(_vp)), ("w_hh", C.POINTER(_vp)), ("b_ih", C.POINTER(_vp)),
        ("b_hh", C.POINTER(_vp)),
        ("w_enc", _vp), ("b_enc", _vp), ("w_pred", _vp), ("b_pred", _vp), ("w_out", _vp), ("b_out", _vp),
    ]


class wind_stats_t(C.Structure):
    _fields_ = [
        ("steps", C.c_int64), ("joint_rows", C.c_int64), ("tokens", C.c_int64), ("forced", C.c_int64),
        ("frames", C.c_int64), ("jump_hist", C.c_int64 * 65), ("status", C.c_int32),
        ("launches_per_step", C.c_int32), ("launches_setup", C.c_int32), ("kernels", C.c_int32),
        ("timeout_site", C.c_int32), ("timeout_cta", C.c_int32),
    ]

    def as_dict(self) -> Dict[str, object]:
        d = {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "jump_hist"}
        d["jump_hist"] = [int(x) for x in self.jump_hist]
        return d


class wind_profile_t(C.Structure):
    _fields_ = [
        ("enc_proj_ms", C.c_double), ("joint_ms", C.c_double), ("control_ms", C.c_double), ("pred_ms", C.c_double),
        ("enc_proj_launches", C.c_int64), ("joint_launches", C.c_int64), ("control_launches", C.c_int64),
        ("pred_launches", C.c_int64),
        ("loop_ms", C.c_double), ("lstm_ms", C.c_double), ("proj_ms", C.c_double), ("gate_table_ms", C.c_double),
    ]


class wind_plan_t(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "grid", "resident", "dataflow", "smem_bytes", "nj", "vt_count", "rg_count", "rg_stride", "j_mode", "tm_j", "tm_l", "tm_p",
        "nl", "np", "ut_count", "ht_count", "ql_count", "qp_count", "l_items", "p_items", "w_first", "w_count", "l_sets",
        "tile_bytes", "buf_off", "z_off", "z_off_p", "stage_off",
        "slots", "ul", "ug_count", "mt_count", "hg_count", "stages_lp", "stages_j", "stage_lp", "stage_j")]

    def as_dict(self) -> Dict[str, int]:
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class wind_joint_bench_t(C.Structure):
    _fields_ = [("ms", C.c_double), ("rows", C.c_int64), ("rows_issued", C.c_int64), ("labels_issued", C.c_int64),
                ("iters", C.c_int32), ("resident", C.c_int32), ("ctas", C.c_int32), ("reserved", C.c_int32)]


class wind_trace_event_t(C.Structure):
    _fields_ = [("role", C.c_int32), ("phase", C.c_int32), ("event", C.c_int32), ("step", C.c_int32), ("clock", C.c_int64)]


_lib = None


def load_library():
    """Load the shared library (works without a GPU; compute calls need one)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2505_13765_b200.build` "
            "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    mp = C.POINTER(wind_model_t)
    i32 = C.c_int32
    L.wind_workspace_bytes.argtypes = [mp, i32, i32, i32, C.POINTER(C.c_size_t)]
    L.wind_workspace_bytes.restype = i32
    L.wind_host_staging_bytes.argtypes = [mp, i32, i32, i32, C.POINTER(C.c_size_t)]
    L.wind_host_staging_bytes.restype = i32
    dec = [mp, _vp, _vp, i32, i32, i32, i32, _vp, _vp, _vp, i32, _vp, C.c_size_t, _vp]
    L.wind_decode_greedy.argtypes = dec
    L.wind_decode_window_greedy.argtypes = dec
    L.wind_decode_window_greedy.restype = i32
    L.wind_decode_greedy.restype = i32
    L.wind_decode_greedy_host.argtypes = dec
    L.wind_refill_workspace_bytes.argtypes = [mp, i32, i32, i32, i32, C.POINTER(C.c_size_t)]
    L.wind_refill_workspace_bytes.restype = i32
    L.wind_decode_greedy_refill.argtypes = [mp, _vp, _vp, i32, i32, i32, i32, i32, _vp, _vp, _vp, i32, _vp, C.c_size_t, _vp]
    L.wind_decode_greedy_refill.restype = i32
    L.wind_decode_greedy_host.restype = i32
    L.wind_profile_decode.argtypes = dec + [C.POINTER(wind_profile_t)]
    L.wind_profile_decode.restype = i32
    L.wind_eval_joint_window.argtypes = [mp, _vp, _vp, i32, i32, i32, _vp, i32, _vp, _vp, _vp, _vp, C.c_size_t, _vp]
    L.wind_eval_joint_window.restype = i32
    L.wind_window_first_output.argtypes = [mp, _vp, _vp, i32, i32, i32, _vp, i32, _vp, _vp, _vp, i32, _vp, _vp, _vp, _vp, C.c_size_t, _vp]
    L.wind_window_first_output.restype = i32
    L.wind_eval_joint_window_static.argtypes = [mp, _vp, _vp, i32, i32, i32, _vp, i32, _vp, _vp, _vp, _vp]
    L.wind_eval_joint_window_static.restype = i32
    L.wind_beam_workspace_bytes.argtypes = [mp, i32, i32, i32, i32, C.POINTER(C.c_size_t)]
    L.wind_beam_workspace_bytes.restype = i32
    L.wind_beam_search.argtypes = [mp, _vp, i32, i32, i32, i32, i32, i32, i32, _vp, _vp, _vp, _vp, C.POINTER(i32),
                                   C.POINTER(C.c_int64), _vp, C.c_size_t, _vp]
    L.wind_beam_search.restype = i32
    L.wind_plan_batches.argtypes = [_vp, i32, i32, _vp, _vp, C.POINTER(i32)]
    L.wind_plan_batches.restype = i32
    L.wind_read_stats.argtypes = [_vp, _vp, C.POINTER(wind_stats_t)]
    L.wind_read_stats.restype = i32
    L.wind_set_trace.argtypes = [i32]
    L.wind_set_trace.restype = i32
    L.wind_read_trace.argtypes = [mp, i32, i32, i32, _vp, _vp, C.POINTER(wind_trace_event_t), i32, C.POINTER(i32)]
    L.wind_read_trace.restype = i32
    L.wind_debug_stall_barrier.argtypes = [i32]
    L.wind_debug_stall_barrier.restype = i32
    L.wind_set_kernels.argtypes = [i32]
    L.wind_set_kernels.restype = i32
    L.wind_set_loop_options.argtypes = [i32, i32, i32, i32]
    L.wind_set_loop_options.restype = None
    L.wind_debug_plan.argtypes = [mp, i32, i32, i32, i32, C.POINTER(wind_plan_t)]
    L.wind_debug_plan.restype = i32
    L.wind_bench_joint.argtypes = [mp, i32, i32, i32, _vp, C.c_size_t, _vp, C.POINTER(wind_joint_bench_t)]
    L.wind_bench_joint.restype = i32
    L.wind_status_string.argtypes = [i32]
    L.wind_status_string.restype = C.c_char_p
    L.wind_last_cuda_error.argtypes = []
    L.wind_last_cuda_error.restype = C.c_char_p
    _lib = L
    return L


class WindError(RuntimeError):
    def __init__(self, status: int):
        L = load_library()
        self.status = status
        msg = L.wind_status_string(status).decode()
        if status == WIND_ERR_CUDA:
            msg += ": " + L.wind_last_cuda_error().decode()
        super().__init__(msg)


def wind_status_string(status: int) -> str:
    return load_library().wind_status_string(status).decode()


def wind_set_loop_options(resident: bool = True, joint_placement: int = -1, max_joint_waves: int = 4, dataflow: int = -1) -> None:
    """Options of the loop kernels' tile planner (process-wide); the defaults restore normal operation."""
    load_library().wind_set_loop_options(int(bool(resident)), int(joint_placement), int(max_joint_waves), int(dataflow))


def wind_debug_plan(dims: Dict[str, int], B: int, W: int, sms: int = 148, smem_optin: int = 232448):
    """The tile plan for bf16 model dimensions `dims` (D, E, P, L, H, V) on a device with the given SM count and
    opt-in shared memory: host arithmetic only (no GPU needed).  Returns (status, dict of the plan's fields)."""
    m = wind_model_t()
    for k in ("D", "E", "P", "L", "H", "V"):
        setattr(m, k, int(dims[k]))
    m.blank_id = int(dims.get("blank_id", dims["V"]))
    m.act = 0
    m.dtype = WIND_DT_BF16
    out = wind_plan_t()
    st = load_library().wind_debug_plan(C.byref(m), B, W, sms, smem_optin, C.byref(out))
    return st, out.as_dict()


def wind_bench_joint(model: "WindModel", B: int, W: int, iters: int, workspace, stream=None) -> Dict[str, float]:
    """The loop kernel's joint phase alone, `iters` times back to back on fixed activations (see wind.h)."""
    out = wind_joint_bench_t()
    st = load_library().wind_bench_joint(model.ref, B, W, iters, _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream),
                                         C.byref(out))
    if st != WIND_OK:
        raise WindError(st)
    return {k: getattr(out, k) for k, _ in out._fields_ if k != "reserved"}


def wind_set_trace(first_step: int) -> int:
    """Record the loop kernel's timeline for lock steps first_step and first_step + 1 (< -1: off)."""
    return load_library().wind_set_trace(first_step)


def wind_read_trace(model: "WindModel", B: int, T: int, W: int, workspace, stream=None) -> List[Dict[str, int]]:
    L = load_library()
    cap = 24 * 512
    buf = (wind_trace_event_t * cap)()
    n = C.c_int32(0)
    st = L.wind_read_trace(model.ref, B, T, W, _ws_ptr(workspace), _stream_ptr(stream), buf, cap, C.byref(n))
    if st != WIND_OK:
        raise WindError(st)
    return [dict(role=e.role, phase=e.phase, event=e.event, step=e.step, clock=e.clock) for e in buf[: n.value]]


def wind_debug_stall_barrier(extra_arrivals: int) -> int:
    """Test hook: make the loop kernel's grid barrier unfillable (see wind.h); 0 restores normal operation."""
    return load_library().wind_debug_stall_barrier(extra_arrivals)


def wind_set_kernels(kernels: int) -> int:
    return load_library().wind_set_kernels(kernels)


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2505_13765_b200 needs a CUDA device (sm_100a); there is no CPU path")
    return torch


def _stream_ptr(stream=None) -> int:
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


class WindModel:
    """Device copies of the weights plus the C struct pointing at them.

    ``weights`` is the dict produced by ``wind_synth.make_model`` (fp32 numpy
    arrays; bf16-representable when ``dtype == 'bf16'``).
    """

    def __init__(self, weights: Dict[str, object], device="cuda:0"):
        torch = _torch()
        self.device = torch.device(device)
        self.dims = {k: int(weights[k]) for k in ("D", "E", "P", "L", "H", "V", "blank_id", "act")}
        self.dtype = WIND_DT_BF16 if weights["dtype"] == "bf16" else WIND_DT_F32
        self._keep: List[object] = []
        tdt = torch.bfloat16 if self.dtype == WIND_DT_BF16 else torch.float32

        def mat(a):
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device).to(tdt).contiguous()
            self._keep.append(t)
            return t.data_ptr()

        def vec(a):
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device).contiguous()
            self._keep.append(t)
            return t.data_ptr()

        L = self.dims["L"]

        def ptr_array(ptrs: Sequence[int]):
            arr = (_vp * L)(*ptrs)
            self._keep.append(arr)
            return arr

        self.c = wind_model_t(
            D=self.dims["D"], E=self.dims["E"], P=self.dims["P"], L=L, H=self.dims["H"], V=self.dims["V"],
            blank_id=self.dims["blank_id"], act=self.dims["act"], dtype=self.dtype, reserved=0,
            emb=mat(weights["emb"]),
            w_ih=ptr_array([mat(a) for a in weights["w_ih"]]), w_hh=ptr_array([mat(a) for a in weights["w_hh"]]),
            b_ih=ptr_array([vec(a) for a in weights["b_ih"]]), b_hh=ptr_array([vec(a) for a in weights["b_hh"]]),
            w_enc=mat(weights["w_enc"]), b_enc=vec(weights["b_enc"]),
            w_pred=mat(weights["w_pred"]), b_pred=vec(weights["b_pred"]),
            w_out=mat(weights["w_out"]), b_out=vec(weights["b_out"]),
        )

    @property
    def ref(self):
        return C.byref(self.c)

    @property
    def torch_dtype(self):
        torch = _torch()
        return torch.bfloat16 if self.dtype == WIND_DT_BF16 else torch.float32


def wind_workspace_bytes(model, B: int, T: int, W: int) -> int:
    """``model`` is a WindModel or a bare ``wind_model_t`` (no GPU needed for the latter)."""
    L = load_library()
    n = C.c_size_t(0)
    ref = model.ref if isinstance(model, WindModel) else C.byref(model)
    st = L.wind_workspace_bytes(ref, B, T, W, C.byref(n))
    if st != WIND_OK:
        raise WindError(st)
    return int(n.value)


def wind_host_staging_bytes(model, B: int, T: int, max_out: int) -> int:
    L = load_library()
    n = C.c_size_t(0)
    ref = model.ref if isinstance(model, WindModel) else C.byref(model)
    st = L.wind_host_staging_bytes(ref, B, T, max_out, C.byref(n))
    if st != WIND_OK:
        raise WindError(st)
    return int(n.value)


def alloc_workspace(model: WindModel, B: int, T: int, W: int, host_staging_max_out: int = 0):
    torch = _torch()
    n = wind_workspace_bytes(model, B, T, W)
    if host_staging_max_out:
        n += wind_host_staging_bytes(model, B, T, host_staging_max_out)
    return torch.empty(n + 256, dtype=torch.uint8, device=model.device)


def _ws_ptr(ws) -> int:
    p = ws.data_ptr()
    return (p + 255) // 256 * 256


def _ws_bytes(ws) -> int:
    return ws.numel() - (_ws_ptr(ws) - ws.data_ptr())


def wind_decode_greedy(model: WindModel, enc, enc_len, W: int, max_symbols: int, out_tokens, out_frames, out_len,
                       workspace, stream=None, check: bool = True) -> int:
    """enc [B,T,D] device tensor of the model's dtype; enc_len/out_* int32 device tensors."""
    L = load_library()
    B, T, D = enc.shape
    assert enc.is_contiguous() and enc.dtype == model.torch_dtype and D == model.dims["D"]
    max_out = out_tokens.shape[1]
    st = L.wind_decode_greedy(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W, max_symbols,
                              out_tokens.data_ptr(), out_frames.data_ptr(), out_len.data_ptr(), max_out,
                              _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_refill_workspace_bytes(model, N: int, T: int, B: int, W: int) -> int:
    L = load_library()
    n = C.c_size_t(0)
    ref = model.ref if isinstance(model, WindModel) else C.byref(model)
    st = L.wind_refill_workspace_bytes(ref, N, T, B, W, C.byref(n))
    if st != WIND_OK:
        raise WindError(st)
    return int(n.value)


def wind_decode_greedy_refill(model: WindModel, enc, enc_len, B: int, W: int, max_symbols: int, out_tokens, out_frames,
                              out_len, workspace, stream=None, check: bool = True) -> int:
    """N utterances on B batch rows, rows refilled inside the loop.  enc [N,T,D]; enc_len/out_* int32 device tensors [N...]."""
    L = load_library()
    N, T, D = enc.shape
    assert enc.is_contiguous() and enc.dtype == model.torch_dtype and D == model.dims["D"]
    max_out = out_tokens.shape[1]
    st = L.wind_decode_greedy_refill(model.ref, enc.data_ptr(), enc_len.data_ptr(), N, T, B, W, max_symbols,
                                     out_tokens.data_ptr(), out_frames.data_ptr(), out_len.data_ptr(), max_out,
                                     _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_decode_window_greedy(model: WindModel, enc, enc_len, W: int, max_symbols: int, out_tokens, out_frames, out_len,
                              workspace, stream=None, check: bool = True) -> int:
    """Window-based greedy decoding; arguments as wind_decode_greedy."""
    L = load_library()
    B, T, D = enc.shape
    assert enc.is_contiguous() and enc.dtype == model.torch_dtype and D == model.dims["D"]
    max_out = out_tokens.shape[1]
    st = L.wind_decode_window_greedy(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W, max_symbols,
                                     out_tokens.data_ptr(), out_frames.data_ptr(), out_len.data_ptr(), max_out,
                                     _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_decode_greedy_host(model: WindModel, enc_host, enc_len_host, W: int, max_symbols: int, out_tokens_host,
                            out_frames_host, out_len_host, workspace, stream=None, check: bool = True) -> int:
    """Same as wind_decode_greedy with HOST (ideally pinned) torch tensors for enc, enc_len and the outputs."""
    L = load_library()
    B, T, D = enc_host.shape
    assert enc_host.is_contiguous() and enc_host.dtype == model.torch_dtype and not enc_host.is_cuda
    max_out = out_tokens_host.shape[1]
    st = L.wind_decode_greedy_host(model.ref, enc_host.data_ptr(), enc_len_host.data_ptr(), B, T, W, max_symbols,
                                   out_tokens_host.data_ptr(), out_frames_host.data_ptr(), out_len_host.data_ptr(),
                                   max_out, _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_profile_decode(model: WindModel, enc, enc_len, W: int, max_symbols: int, out_tokens, out_frames, out_len,
                        workspace, stream=None) -> Dict[str, float]:
    """Per-kernel CUDA-event times of one decode (measurement aid, host-driven loop)."""
    L = load_library()
    B, T, D = enc.shape
    prof = wind_profile_t()
    st = L.wind_profile_decode(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W, max_symbols,
                               out_tokens.data_ptr(), out_frames.data_ptr(), out_len.data_ptr(), out_tokens.shape[1],
                               _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream), C.byref(prof))
    if st != WIND_OK:
        raise WindError(st)
    return {k: getattr(prof, k) for k, _ in prof._fields_}


def wind_eval_joint_window(model: WindModel, enc, enc_len, W: int, prefix, prefix_len, t0, logits, workspace,
                           stream=None, check: bool = True) -> int:
    L = load_library()
    B, T, D = enc.shape
    U = prefix.shape[1] if prefix is not None and prefix.numel() else 0
    st = L.wind_eval_joint_window(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W,
                                  prefix.data_ptr() if U else None, U, prefix_len.data_ptr(), t0.data_ptr(),
                                  logits.data_ptr(), _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_window_first_output(model: WindModel, enc, enc_len, W: int, prefix, prefix_len, t0, logp, workspace, K: int = 0,
                             top_label=None, top_jump=None, top_logp=None, stream=None) -> int:
    """Eq. (1): log P'(v, t) of each utterance's window into ``logp`` [B, W, V+1]; optionally the K best (label, offset)."""
    L = load_library()
    B, T, D = enc.shape
    U = prefix.shape[1] if prefix is not None and prefix.numel() else 0
    st = L.wind_window_first_output(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W,
                                    prefix.data_ptr() if U else None, U, prefix_len.data_ptr(), t0.data_ptr(),
                                    logp.data_ptr(), K, top_label.data_ptr() if K else None, top_jump.data_ptr() if K else None,
                                    top_logp.data_ptr() if K else None, _ws_ptr(workspace), _ws_bytes(workspace), _stream_ptr(stream))
    if st != WIND_OK:
        raise WindError(st)
    return st


WIND_STATIC_WORKSPACE_BYTES = 16 * 1024 * 1024


def wind_eval_joint_window_static(model: WindModel, enc, enc_len, W: int, prefix, prefix_len, t0, logits, stream=None,
                                  check: bool = True) -> int:
    """wind_eval_joint_window without a caller workspace: for callers that cannot allocate device
    memory.  Scratch is the library's built-in array of WIND_STATIC_WORKSPACE_BYTES; larger problems
    are rejected with WIND_ERR_WORKSPACE.  Calls sharing a device must not overlap on the GPU."""
    L = load_library()
    B, T, D = enc.shape
    U = prefix.shape[1] if prefix is not None and prefix.numel() else 0
    st = L.wind_eval_joint_window_static(model.ref, enc.data_ptr(), enc_len.data_ptr(), B, T, W,
                                         prefix.data_ptr() if U else None, U, prefix_len.data_ptr(), t0.data_ptr(),
                                         logits.data_ptr(), _stream_ptr(stream))
    if check and st != WIND_OK:
        raise WindError(st)
    return st


def wind_read_stats(workspace, stream=None) -> Dict[str, object]:
    L = load_library()
    s = wind_stats_t()
    st = L.wind_read_stats(_ws_ptr(workspace), _stream_ptr(stream), C.byref(s))
    if st != WIND_OK:
        raise WindError(st)
    return s.as_dict()


# ---------------------------------------------------------------------------
# convenience wrapper used by the tests and the benchmark
# ---------------------------------------------------------------------------
def to_device_enc(model: WindModel, enc_np: np.ndarray):
    torch = _torch()
    t = torch.from_numpy(np.ascontiguousarray(enc_np, dtype=np.float32))
    return t.to(model.torch_dtype).to(model.device).contiguous()


def wind_beam_search(model: WindModel, enc_np: np.ndarray, W: int, K: int, S: int, max_hyps: int = 64,
                     max_out: Optional[int] = None, check: bool = True, prefix_search: bool = False):
    """Algorithm 3 for one utterance [T, D] (numpy).  Returns (list of (tokens, frames, score) best first, steps, status)."""
    torch = _torch()
    L = load_library()
    T = int(enc_np.shape[0])
    enc = to_device_enc(model, enc_np[None])[0].contiguous()
    if max_out is None:
        max_out = max(1, T * S)
    n = C.c_size_t(0)
    st = L.wind_beam_workspace_bytes(model.ref, T, W, K, S, C.byref(n))
    if st != WIND_OK:
        if check:
            raise WindError(st)
        return [], 0, st
    ws = torch.empty(n.value + 256, dtype=torch.uint8, device=model.device)
    off = (-ws.data_ptr()) % 256
    tok = np.full((max_hyps, max_out), -1, np.int32)
    frm = np.full((max_hyps, max_out), -1, np.int32)
    ln = np.zeros(max_hyps, np.int32)
    sc = np.zeros(max_hyps, np.float64)
    nh, steps = C.c_int32(0), C.c_int64(0)
    st = L.wind_beam_search(model.ref, enc.data_ptr(), T, W, K, S, int(bool(prefix_search)), max_hyps, max_out,
                            tok.ctypes.data, frm.ctypes.data,
                            ln.ctypes.data, sc.ctypes.data, C.byref(nh), C.byref(steps), ws.data_ptr() + off, n.value,
                            _stream_ptr(None))
    if check and st != WIND_OK:
        raise WindError(st)
    hyps = [(tok[a, : min(ln[a], max_out)].copy(), frm[a, : min(ln[a], max_out)].copy(), float(sc[a])) for a in range(nh.value)]
    return hyps, steps.value, st


def wind_plan_batches(lens_np: np.ndarray, B: int):
    """Length-aware batching plan: (order [N], batch_T [n_batches]); batch k = order[k*B : (k+1)*B]."""
    L = load_library()
    lens = np.ascontiguousarray(lens_np, dtype=np.int32)
    N = int(lens.shape[0])
    order = np.zeros(max(N, 1), np.int32)
    batch_T = np.zeros(max((N + B - 1) // max(B, 1), 1), np.int32)
    nb = C.c_int32(0)
    st = L.wind_plan_batches(lens.ctypes.data, N, B, order.ctypes.data, batch_T.ctypes.data, C.byref(nb))
    if st != WIND_OK:
        raise WindError(st)
    return order[:N], batch_T[: nb.value]


def decode_dataset(model: WindModel, utterances, W: int, S: int, B: int, plan: bool = True, window_greedy: bool = False,
                   refill: bool = False):
    """Decodes a list of [T_i, D] numpy arrays on B batch rows; results come back in the list's order.

    plan=True groups utterances of similar length (wind_plan_batches); plan=False keeps the arrival order.  Packing the
    batches is marshalling; every batch is one call of the decode entry point.  refill=True hands the whole list to
    wind_decode_greedy_refill in ONE call (longest first when plan=True): a row takes the next utterance as soon as its
    own is finished; models and shapes that entry point does not cover fall back to the batches.  Returns (list of token
    arrays, list of frame arrays, total lock steps).
    """
    lens = np.array([u.shape[0] for u in utterances], np.int32)
    N = len(utterances)
    if refill and not window_greedy and N > 0:
        order = wind_plan_batches(lens, B)[0] if plan else np.arange(N, dtype=np.int32)
        T = max(1, int(lens.max()))
        enc = np.zeros((N, T, model.dims["D"]), np.float32)
        for r, i in enumerate(order):
            enc[r, : lens[i]] = utterances[i]
        tok, frm, olen, stats, st = decode_refill(model, enc, lens[order], B, W, S, check=False)
        if st == WIND_OK:
            toks, frms = [None] * N, [None] * N
            for r, i in enumerate(order):
                toks[i], frms[i] = tok[r, : olen[r]].copy(), frm[r, : olen[r]].copy()
            return toks, frms, stats["steps"]
        if st != WIND_ERR_UNSUPPORTED:
            raise WindError(st)
    if plan:
        order, _ = wind_plan_batches(lens, B)
    else:
        order = np.arange(N, dtype=np.int32)
    toks, frms, steps = [None] * N, [None] * N, 0
    D = model.dims["D"]
    for k in range(0, N, B):
        idx = order[k: k + B]
        T = max(1, int(lens[idx].max()))
        enc = np.zeros((len(idx), T, D), np.float32)
        for r, i in enumerate(idx):
            enc[r, : lens[i]] = utterances[i]
        tok, frm, olen, stats, _ = decode(model, enc, lens[idx], W, S, window_greedy=window_greedy)
        steps += stats["steps"]
        for r, i in enumerate(idx):
            toks[i], frms[i] = tok[r, : olen[r]].copy(), frm[r, : olen[r]].copy()
    return toks, frms, steps


def decode_refill(model: WindModel, enc_np: np.ndarray, lens_np: np.ndarray, B: int, W: int, S: int,
                  max_out: Optional[int] = None, check: bool = True):
    """All N utterances of enc_np [N,T,D] on B batch rows that are refilled inside the loop (wind_decode_greedy_refill);
    returns numpy (tokens [N, max_out], frames, out_len [N], stats, status)."""
    torch = _torch()
    N, T, _ = enc_np.shape
    enc = to_device_enc(model, enc_np)
    lens = torch.from_numpy(np.ascontiguousarray(lens_np, dtype=np.int32)).to(model.device)
    if max_out is None:
        max_out = max(1, T * S)
    tok = torch.full((N, max_out), -1, dtype=torch.int32, device=model.device)
    frm = torch.full((N, max_out), -1, dtype=torch.int32, device=model.device)
    olen = torch.zeros(N, dtype=torch.int32, device=model.device)
    ws = torch.empty(wind_refill_workspace_bytes(model, N, T, B, W) + 256, dtype=torch.uint8, device=model.device)
    st = wind_decode_greedy_refill(model, enc, lens, B, W, S, tok, frm, olen, ws, check=check)
    stats = wind_read_stats(ws)
    return tok.cpu().numpy(), frm.cpu().numpy(), olen.cpu().numpy(), stats, st


def decode(model: WindModel, enc_np: np.ndarray, lens_np: np.ndarray, W: int, S: int, max_out: Optional[int] = None,
           check: bool = True, window_greedy: bool = False):
    """Marshals numpy inputs to the device, decodes, returns numpy (tokens, frames, out_len, stats, status)."""
    torch = _torch()
    B, T, _ = enc_np.shape
    enc = to_device_enc(model, enc_np)
    lens = torch.from_numpy(np.ascontiguousarray(lens_np, dtype=np.int32)).to(model.device)
    if max_out is None:
        max_out = max(1, T * S)
    tok = torch.full((B, max_out), -1, dtype=torch.int32, device=model.device)
    frm = torch.full((B, max_out), -1, dtype=torch.int32, device=model.device)
    olen = torch.zeros(B, dtype=torch.int32, device=model.device)
    ws = alloc_workspace(model, B, T, W)
    call = wind_decode_window_greedy if window_greedy else wind_decode_greedy
    st = call(model, enc, lens, W, S, tok, frm, olen, ws, check=check)
    stats = wind_read_stats(ws)
    return tok.cpu().numpy(), frm.cpu().numpy(), olen.cpu().numpy(), stats, st
