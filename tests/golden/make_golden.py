"""Writes tests/golden/cfg1_tiny_oracle.json: the CPU oracle's own result on the tiny configuration.

The paper prints no worked numeric example (its numbers need its checkpoints and test sets), so this file
is not a value from the paper: it freezes the oracle's sequential-greedy output (Algorithm 1) on the seeded
tiny workload, so that a later change to the oracle's arithmetic or to the input generator shows up as a
diff of this file.  It calls nothing but the oracle and the input generator.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
import wind_synth as ws  # noqa: E402


def main():
    cfg = ws.CONFIGS["cfg1_tiny"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    om = oracle.Model(weights)
    tok, frm, n, st = oracle.decode_batch(om, enc, lens, W=0, S=cfg.S)
    out = {
        "source": "oracle.decode_batch(W=0) on wind_synth cfg1_tiny (Algorithm 1, sequential greedy)",
        "config": cfg.name, "seed": cfg.seed, "S": cfg.S, "lens": [int(x) for x in lens],
        "b_out_blank": float(weights["b_out"][cfg.blank_id]),
        "tokens": [[int(x) for x in tok[b, : n[b]]] for b in range(cfg.B)],
        "frames": [[int(x) for x in frm[b, : n[b]]] for b in range(cfg.B)],
        "decisions": st["decisions"], "low_margin": st["low_margin"], "emit_frames": st["emit_frames"],
    }
    with open(os.path.join(HERE, "cfg1_tiny_oracle.json"), "w") as f:
        json.dump(out, f)
        f.write("\n")
    print("tokens", sum(len(t) for t in out["tokens"]), "decisions", out["decisions"])


if __name__ == "__main__":
    main()
