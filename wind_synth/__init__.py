"""Seeded synthetic inputs for batched greedy RNN-T / WIND decoding.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no projection, LSTM, joint, argmax or decoding loop).
Both the CPU oracle's tests and the CUDA path's tests/bench take their inputs
from here so that the two sides see identical bytes.

Recipe (shapes follow the workloads named in the paper's experiments section:
BPE vocabulary of 1024 labels plus blank, window sizes 1..16; the remaining
dimensions are the configured FastConformer-Large / XL decoder shapes):

* weight matrices, PyTorch ``[out, in]`` row-major, i.i.d. N(0, 1/fan_in);
* embedding rows N(0, 1), the blank/start-of-sequence row all zeros;
* all biases zero except ``b_out[blank]``, which is a calibrated constant read
  from ``blank_bias.json`` (written by ``oracle/calibrate_blank_bias.py``);
* encoder frames i.i.d. N(0, 1); utterance lengths uniform integers in the
  configured range; frames beyond an utterance's length are NaN (parity runs,
  a poison that must never be decoded) or zero (timing runs);
* on the bf16 path every weight matrix and the encoder frames are rounded to
  bf16 (round-to-nearest-even) exactly once here; both sides consume those
  rounded values, so only on-chip rounding differs between them.

Random numbers come from numpy's counter-based Philox generator keyed by
``seed`` and a per-tensor stream id, so a tensor's values do not depend on the
order in which tensors are requested.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np

ACT_RELU = 0
ACT_TANH = 1

BASE_SEED = 20250513
_BIAS_FILE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "blank_bias.json")


@dataclass(frozen=True)
class WindConfig:
    name: str
    index: int              # seed offset
    B: int                  # utterances
    len_lo: int             # shortest utterance, frames
    len_hi: int             # longest utterance, frames (= padded T)
    D: int                  # encoder dim
    E: int                  # embedding dim
    P: int                  # pred-net LSTM hidden
    L: int                  # LSTM layers
    H: int                  # joint hidden
    V: int                  # labels (logits are V+1 wide)
    act: int                # ACT_RELU / ACT_TANH
    W: int                  # default window
    S: int                  # max symbols per frame
    dtype: str              # "f32" or "bf16"
    rate: float             # target non-blank frame rate
    rate_tol: float = 0.02

    @property
    def blank_id(self) -> int:
        return self.V

    @property
    def T(self) -> int:
        return self.len_hi

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


CONFIGS: Dict[str, WindConfig] = {
    c.name: c
    for c in [
        WindConfig("cfg1_tiny", 1, 1, 100, 100, 64, 64, 64, 1, 64, 32, ACT_RELU, 4, 5, "f32", 0.30),
        WindConfig("cfg2_large_b1", 2, 1, 1250, 1250, 512, 640, 640, 1, 640, 1024, ACT_RELU, 8, 10, "bf16", 0.35),
        WindConfig("cfg3_large_b128", 3, 128, 125, 2500, 512, 640, 640, 1, 640, 1024, ACT_RELU, 8, 10, "bf16", 0.35),
        WindConfig("cfg4_xl_r25", 4, 64, 500, 5000, 1024, 640, 640, 2, 640, 1024, ACT_RELU, 8, 10, "bf16", 0.25),
        WindConfig("cfg4_xl_r50", 4, 64, 500, 5000, 1024, 640, 640, 2, 640, 1024, ACT_RELU, 8, 10, "bf16", 0.50),
        WindConfig("cfg5_bigvocab", 5, 32, 250, 3000, 1024, 1024, 1024, 1, 1024, 8192, ACT_TANH, 16, 10, "bf16", 0.40),
    ]
}


def small_variant(cfg: WindConfig, B: int, len_lo: int, len_hi: int) -> WindConfig:
    """Same model shapes and seed (hence the same weights), fewer/shorter utterances."""
    return replace(cfg, B=B, len_lo=len_lo, len_hi=len_hi)


# ---------------------------------------------------------------------------
# bf16 helpers (pure bit manipulation)
# ---------------------------------------------------------------------------
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result is fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    nan = np.isnan(a)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    out = r.view(np.float32).copy()
    out[nan] = np.nan
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 array whose values are already bf16-representable -> uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# ---------------------------------------------------------------------------
# generators
# ---------------------------------------------------------------------------
def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(stream)]))


def _normal(seed: int, stream: int, shape, std: float) -> np.ndarray:
    a = _rng(seed, stream).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def load_blank_bias(name: str) -> Optional[float]:
    if not os.path.exists(_BIAS_FILE):
        return None
    with open(_BIAS_FILE) as f:
        table = json.load(f)
    ent = table.get(name)
    return None if ent is None else float(ent["b_out_blank"])


def make_model(cfg: WindConfig, blank_bias: Optional[float] = None) -> Dict[str, object]:
    """Weights as fp32 numpy arrays (bf16-representable when cfg.dtype == 'bf16').

    ``w_ih``, ``w_hh``, ``b_ih``, ``b_hh`` are lists of length L.  Gate order in
    the 4P axis is (input, forget, cell, output).
    """
    s = cfg.seed
    rnd = bf16_round if cfg.dtype == "bf16" else (lambda x: x)
    emb = _normal(s, 1, (cfg.V + 1, cfg.E), 1.0)
    emb[cfg.blank_id, :] = 0.0
    w_ih, w_hh, b_ih, b_hh = [], [], [], []
    for l in range(cfg.L):
        fan = cfg.E if l == 0 else cfg.P
        w_ih.append(rnd(_normal(s, 10 + 4 * l, (4 * cfg.P, fan), fan ** -0.5)))
        w_hh.append(rnd(_normal(s, 11 + 4 * l, (4 * cfg.P, cfg.P), cfg.P ** -0.5)))
        b_ih.append(np.zeros(4 * cfg.P, np.float32))
        b_hh.append(np.zeros(4 * cfg.P, np.float32))
    w_enc = rnd(_normal(s, 2, (cfg.H, cfg.D), cfg.D ** -0.5))
    w_pred = rnd(_normal(s, 3, (cfg.H, cfg.P), cfg.P ** -0.5))
    w_out = rnd(_normal(s, 4, (cfg.V + 1, cfg.H), cfg.H ** -0.5))
    b_out = np.zeros(cfg.V + 1, np.float32)
    if blank_bias is None:
        blank_bias = load_blank_bias(cfg.name)
    if blank_bias is None:
        blank_bias = 0.0
    b_out[cfg.blank_id] = np.float32(blank_bias)
    return dict(
        D=cfg.D, E=cfg.E, P=cfg.P, L=cfg.L, H=cfg.H, V=cfg.V,
        blank_id=cfg.blank_id, act=cfg.act, dtype=cfg.dtype,
        emb=rnd(emb), w_ih=w_ih, w_hh=w_hh, b_ih=b_ih, b_hh=b_hh,
        w_enc=w_enc, b_enc=np.zeros(cfg.H, np.float32),
        w_pred=w_pred, b_pred=np.zeros(cfg.H, np.float32),
        w_out=w_out, b_out=b_out,
    )


def make_lengths(cfg: WindConfig, seed_offset: int = 0) -> np.ndarray:
    g = _rng(cfg.seed + seed_offset, 100)
    return g.integers(cfg.len_lo, cfg.len_hi + 1, size=cfg.B, dtype=np.int64).astype(np.int32)


def make_enc(cfg: WindConfig, pad: str = "nan", seed_offset: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Encoder outputs ``[B, T, D]`` fp32 and lengths ``[B]`` int32.

    ``seed_offset=1000`` gives the separate calibration sample.
    """
    lens = make_lengths(cfg, seed_offset)
    fill = {"nan": np.nan, "zero": 0.0}[pad]
    enc = np.full((cfg.B, cfg.T, cfg.D), fill, dtype=np.float32)
    for b in range(cfg.B):
        enc[b, : int(lens[b])] = make_utterance(cfg, b, int(lens[b]), seed_offset)
    return enc, lens


def make_utterance(cfg: WindConfig, b: int, n: int, seed_offset: int = 0) -> np.ndarray:
    """The ``n`` valid frames ``[n, D]`` of utterance ``b`` (the rows ``make_enc`` puts at ``enc[b, :n]``)."""
    x = _normal(cfg.seed + seed_offset, 1000 + b, (n, cfg.D), 1.0)
    return bf16_round(x) if cfg.dtype == "bf16" else x
