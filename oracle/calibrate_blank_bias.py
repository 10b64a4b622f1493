"""Calibrate the blank output bias of every synthetic configuration.

For each configuration the blank logit's bias is bisected in [-20, 20] on a
separate seeded calibration sample (same weights, encoder frames drawn with
seed + 1000) until the oracle's non-blank frame rate -- the fraction of valid
frames on which sequential greedy decoding (Algorithm 1) emits at least one
token -- is within 0.005 of the configured target.  The result is written to
``wind_synth/blank_bias.json``; the input generator only reads that file.

This script calls nothing but the oracle and the input generator.

    python -m oracle.calibrate_blank_bias [config ...]
"""
from __future__ import annotations

import json
import os
import sys
import time

import numpy as np

import oracle
import wind_synth as ws

OUT = os.path.join(os.path.dirname(os.path.abspath(ws.__file__)), "blank_bias.json")

# calibration sample per config: (utterances, frames each)
CAL_SHAPE = {
    "cfg1_tiny": (16, 250),
    "cfg2_large_b1": (8, 500),
    "cfg3_large_b128": (8, 500),
    "cfg4_xl_r25": (8, 500),
    "cfg4_xl_r50": (8, 500),
    "cfg5_bigvocab": (8, 250),
}


def rate_for_bias(cfg, weights, enc, lens, bias):
    weights = dict(weights)
    b_out = np.array(weights["b_out"], copy=True)
    b_out[cfg.blank_id] = np.float32(bias)
    weights["b_out"] = b_out
    model = oracle.Model(weights)
    _, _, out_len, st = oracle.decode_batch(model, enc, lens, W=0, S=cfg.S)
    frames = int(lens.sum())
    return st["emit_frames"] / frames, float(out_len.sum()) / frames


def calibrate(name: str):
    cfg = ws.CONFIGS[name]
    nb, nt = CAL_SHAPE[name]
    cal = ws.small_variant(cfg, nb, nt, nt)
    weights = ws.make_model(cal, blank_bias=0.0)
    enc, lens = ws.make_enc(cal, pad="zero", seed_offset=1000)
    lo, hi = -20.0, 20.0
    best = None
    for it in range(24):
        mid = 0.5 * (lo + hi)
        rate, tpf = rate_for_bias(cal, weights, enc, lens, mid)
        print(f"  {name}: bias {mid:+.5f} -> non-blank frame rate {rate:.4f}, tokens/frame {tpf:.3f}", flush=True)
        if best is None or abs(rate - cfg.rate) < abs(best[1] - cfg.rate):
            best = (mid, rate, tpf)
        if abs(rate - cfg.rate) <= 0.005:
            break
        # a larger blank bias makes blank win more often -> lower rate
        if rate > cfg.rate:
            lo = mid
        else:
            hi = mid
    bias = float(np.float32(best[0]))
    return dict(b_out_blank=bias, target_rate=cfg.rate, calibration_rate=best[1], calibration_tokens_per_frame=best[2],
                calibration_sample=f"{nb}x{nt} frames, seed {cal.seed}+1000", iterations=it + 1)


def main(argv):
    names = argv or list(ws.CONFIGS)
    table = {}
    if os.path.exists(OUT):
        with open(OUT) as f:
            table = json.load(f)
    for n in names:
        t = time.time()
        table[n] = calibrate(n)
        print(f"{n}: {table[n]} ({time.time() - t:.1f}s)", flush=True)
        with open(OUT, "w") as f:
            json.dump(table, f, indent=1, sort_keys=True)
            f.write("\n")


if __name__ == "__main__":
    main(sys.argv[1:])
