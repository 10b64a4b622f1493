"""GPU parity at the stated size of every batched configuration, in the launch configuration the benchmark times.

The library decodes the whole batch (B = 128 / 64 / 32 utterances of up to 2500 / 5000 / 3000 frames).  Every
transcript gets the checks that hold at any size (frames non-decreasing and inside the utterance, at most S tokens per
frame, labels in range, counters consistent).  A sample of utterances -- the shortest few, one from the middle of the
length order and (configurations 3 and 4 at rate 0.25) the longest, listed in tests/golden/fullsize_oracle.json together with a digest of the oracle's own
transcript (written by tests/golden/make_golden.py --fullsize, which calls only the oracle and the input generator) --
is compared with the oracle under the margin rule: the transcript is replayed through the oracle, every implied
decision must be the oracle's argmax or lie within 0.05 of its maximum, and a transcript whose decisions are all the
argmax must equal the oracle's bit for bit.  For the configuration with a window sweep the transcripts of all window
sizes must be equal on the GPU (Algorithm 2 gives Algorithm 1's result for every W).
"""
import hashlib
import json
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import oracle
import wind_synth as ws

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden", "fullsize_oracle.json")
MARGIN = 0.05


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_13765_b200 as p
    p.load_library()
    return p


def digest(tokens, frames) -> str:
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(tokens, dtype=np.int32).tobytes())
    h.update(np.ascontiguousarray(frames, dtype=np.int32).tobytes())
    return h.hexdigest()


def structural_checks(cfg, lens, tok, frm, olen, stats, W):
    for b in range(cfg.B):
        f, k = frm[b, : olen[b]], tok[b, : olen[b]]
        assert np.all(np.diff(f) >= 0)
        if len(f):
            assert f.min() >= 0 and f.max() < lens[b] and np.bincount(f).max() <= cfg.S
        assert np.all((k >= 0) & (k < cfg.V))
        assert np.all(tok[b, olen[b]:] == -1)
    assert stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
    hist = np.array(stats["jump_hist"])
    assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum())
    assert hist[W + 1:].sum() == 0


def fullsize_case(pkg, name, windows, replay_windows):
    g = json.load(open(GOLDEN))[name]
    cfg = ws.CONFIGS[name]
    weights = ws.make_model(cfg)
    assert cfg.seed == g["seed"] and cfg.S == g["S"] and float(weights["b_out"][cfg.blank_id]) == g["b_out_blank"]
    enc, lens = ws.make_enc(cfg, pad="nan")
    model = pkg.WindModel(weights)
    om = oracle.Model(weights)
    sample = sorted(int(b) for b in g["utterances"])
    outs = {}
    for W in windows:
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, cfg.S)
        assert st == 0 and stats["kernels"] == 2, (W, st, stats["kernels"])
        structural_checks(cfg, lens, tok, frm, olen, stats, W)
        outs[W] = (tok, frm, olen)
        print(f"[{name}] W={W}: {stats['steps']} lock steps, {int(olen.sum())} tokens over {int(lens.sum())} frames")
    # Algorithm 2 gives the same transcripts for every window (bit for bit on the GPU path by itself)
    first = outs[windows[0]]
    for W in windows[1:]:
        for a, b in zip(outs[W], first):
            assert np.array_equal(a, b), f"window {W} differs from window {windows[0]}"
    for W in replay_windows:
        tok, frm, olen = outs[W]

        def replay(b):
            return oracle.replay_verify(om, enc[b], int(lens[b]), cfg.S, tok[b, : olen[b]], frm[b, : olen[b]], MARGIN)

        with ThreadPoolExecutor(min(8, len(sample))) as ex:
            reps = list(ex.map(replay, sample))
        exact = off = 0
        for b, r in zip(sample, reps):
            ref = g["utterances"][str(b)]
            assert ref["len"] == int(lens[b])
            assert r["rc"] == 0, f"{name} W={W} utterance {b}: replay failed {r}"
            same = int(olen[b]) == ref["n"] and digest(tok[b, : olen[b]], frm[b, : olen[b]]) == ref["sha256"]
            exact += same
            off += r["not_argmax"]
            if r["not_argmax"] == 0:
                assert same, f"{name} W={W} utterance {b}: every decision is the oracle argmax yet the transcripts differ"
        print(f"[{name}] W={W}: {exact}/{len(sample)} sampled utterances equal to the oracle's transcript, {off} decisions "
              f"off the oracle argmax (all inside {MARGIN})")


def test_cfg3_at_its_stated_size(pkg):
    fullsize_case(pkg, "cfg3_large_b128", windows=[8, 1], replay_windows=[8])


def test_cfg4_rate25_at_its_stated_size_window_sweep(pkg):
    fullsize_case(pkg, "cfg4_xl_r25", windows=[8, 1, 4, 16], replay_windows=[8])


def test_cfg4_rate50_at_its_stated_size(pkg):
    fullsize_case(pkg, "cfg4_xl_r50", windows=[16, 8], replay_windows=[16])


def test_cfg5_at_its_stated_size(pkg):
    fullsize_case(pkg, "cfg5_bigvocab", windows=[16, 1], replay_windows=[16])
