"""Writes the stored oracle results under tests/golden/.  Calls nothing but the oracle and the input generator.

cfg1_tiny_oracle.json: the CPU oracle's own result on the tiny configuration.  The paper prints no worked numeric
example (its numbers need its checkpoints and test sets), so this file is not a value from the paper: it freezes the
oracle's sequential-greedy output (Algorithm 1) on the seeded tiny workload, so that a later change to the oracle's
arithmetic or to the input generator shows up as a diff of this file.

fullsize_oracle.json (--fullsize): for the batched configurations at their stated sizes, the oracle's sequential-greedy
result on a sample of utterances (the shortest few, one from the middle of the length order, for two of them the
longest), stored as
the transcript length, a SHA-256 digest of the (token, frame) arrays and the decision statistics.  The GPU tests at
full size compare the library's transcripts of those utterances with the digests before they replay them through the
oracle, so the oracle's own decode of them is not repeated at every test run.

    python tests/golden/make_golden.py [--fullsize]
"""
import hashlib
import json
import os
import sys
from concurrent.futures import ThreadPoolExecutor

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
import wind_synth as ws  # noqa: E402

# configuration -> (how many of the shortest utterances, whether the longest is taken too); the utterance at the middle
# of the length order is always in.  (The longest of the two costliest configurations would take the oracle minutes
# at every test run; the longest of the other two covers the end of a decode, when every other row has finished.)
FULLSIZE = {"cfg3_large_b128": (8, True), "cfg4_xl_r25": (4, True), "cfg4_xl_r50": (4, False), "cfg5_bigvocab": (4, False)}


def transcript_digest(tokens, frames) -> str:
    """SHA-256 over the int32 token array followed by the int32 frame array."""
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(tokens, dtype=np.int32).tobytes())
    h.update(np.ascontiguousarray(frames, dtype=np.int32).tobytes())
    return h.hexdigest()


def fullsize_sample(lens, n_short, with_longest):
    order = np.argsort(lens, kind="stable")
    picked = [int(i) for i in order[:n_short]] + [int(order[len(order) // 2])] + ([int(order[-1])] if with_longest else [])
    return sorted(set(picked))


def tiny():
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


def fullsize():
    out = {"source": "oracle.decode_batch(W=0) (Algorithm 1) on sampled utterances of the wind_synth configurations at "
                     "their stated sizes; digest = SHA-256 of int32 tokens then int32 frames"}
    for name, (n_short, with_longest) in FULLSIZE.items():
        cfg = ws.CONFIGS[name]
        weights = ws.make_model(cfg)
        lens = ws.make_lengths(cfg)
        sample = fullsize_sample(lens, n_short, with_longest)
        om = oracle.Model(weights)

        def one(b):
            n = int(lens[b])
            x = ws.make_utterance(cfg, b, n)
            tok, frm, cnt, st = oracle.decode_batch(om, x[None], lens[b: b + 1], W=0, S=cfg.S, max_out=n * cfg.S)
            return dict(len=n, n=int(cnt[0]), sha256=transcript_digest(tok[0, : cnt[0]], frm[0, : cnt[0]]),
                        decisions=st["decisions"], low_margin=st["low_margin"], emit_frames=st["emit_frames"])

        with ThreadPoolExecutor(min(8, len(sample))) as ex:
            res = list(ex.map(one, sample))
        out[name] = {"seed": cfg.seed, "S": cfg.S, "b_out_blank": float(weights["b_out"][cfg.blank_id]),
                     "utterances": {str(b): r for b, r in zip(sample, res)}}
        print(name, {b: (r["len"], r["n"]) for b, r in zip(sample, res)}, flush=True)
    with open(os.path.join(HERE, "fullsize_oracle.json"), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")


if __name__ == "__main__":
    if "--fullsize" in sys.argv:
        fullsize()
    else:
        tiny()
