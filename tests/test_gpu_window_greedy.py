"""GPU parity of window-based greedy decoding (the most probable (label, offset) pair of Eq. (1) per step) against
the oracle: every decision of the GPU's output must be the oracle's pick or lie within the margin of it in log P',
and utterances without such near-ties must match the oracle's own output token for token."""
import os
import sys
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

from conftest import LOOP_MODES, set_loop_mode
import torch

sys.path.insert(0, os.path.join(os.path.dirname(__file__), ".."))
sys.path.insert(0, os.path.dirname(__file__))

import oracle
import wind_synth as ws
from naive_model import random_weights
from test_gpu_parity import ragged_case, MARGIN
from test_oracle_pins import table_model

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_13765_b200 as p
    p.load_library()
    return p


def check_window_greedy(pkg, weights, enc, lens, W, S, kernels=0):
    prev = pkg.wind_set_kernels(kernels)
    try:
        model = pkg.WindModel(weights)
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, S, window_greedy=True)
    finally:
        pkg.wind_set_kernels(prev)
    assert st == 0
    om = oracle.Model(weights)
    B = enc.shape[0]
    otok, ofrm, on, ost = oracle.decode_window_greedy_batch(om, enc, lens, W=W, S=S, max_out=tok.shape[1])

    def replay(b):
        return oracle.replay_verify_window(om, enc[b], int(lens[b]), W, S, tok[b, : olen[b]], frm[b, : olen[b]], MARGIN)

    with ThreadPoolExecutor(8) as ex:
        reps = list(ex.map(replay, range(B)))
    exact = off = 0
    for b in range(B):
        r = reps[b]
        assert r["rc"] == 0, f"utterance {b}: replay failed {r}"
        off += r["not_argmax"]
        same = on[b] == olen[b] and np.array_equal(otok[b, : on[b]], tok[b, : olen[b]]) and \
            np.array_equal(ofrm[b, : on[b]], frm[b, : olen[b]])
        exact += bool(same)
        if r["not_argmax"] == 0:
            assert same, f"utterance {b}: every decision is the oracle's pick yet the sequences differ"
        f = frm[b, : olen[b]]
        assert np.all(np.diff(f) >= 0)
        if len(f):
            assert f.max() < lens[b] and np.bincount(f).max() <= S
        assert np.all(tok[b, olen[b]:] == -1)
    assert stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
    hist = np.array(stats["jump_hist"])
    assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum()) and hist[W + 1:].sum() == 0
    print(f"[window-greedy] W={W} S={S} exact {exact}/{B} utterances, {off} decisions off the oracle's pick (all inside "
          f"{MARGIN}); oracle low-margin decisions {ost['low_margin']}/{ost['decisions']}")
    return dict(exact=exact, off=off, stats=stats), (tok, frm, olen)


def test_worked_example_fp32(pkg):
    # frame types A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1), C = (x .02, y .03, blank .95); utterance
    # A B C C, S = 1.  W = 2: P'(x,0) = .45 beats P'(y,1) = .4 -> x at 0, then y at 1.  Algorithm 2: only y at 1.
    w = table_model([[.45, .05, .5], [.1, .8, .1], [.02, .03, .95]])
    enc = np.eye(3, dtype=np.float32)[[0, 1, 2, 2]][None]
    lens = np.array([4], np.int32)
    model = pkg.WindModel(w)
    for W, want_t, want_f in ((2, [0, 1], [0, 1]), (3, [0, 1], [0, 1]), (1, [1], [1])):
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, 1, window_greedy=True)
        assert st == 0 and list(tok[0, : olen[0]]) == want_t and list(frm[0, : olen[0]]) == want_f
    tok, frm, olen, stats, st = pkg.decode(model, enc, lens, 2, 1)
    assert list(tok[0, : olen[0]]) == [1] and list(frm[0, : olen[0]]) == [1]
    w2 = table_model([[.3, .1, .6], [.1, .8, .1], [.02, .03, .95]])
    tok, frm, olen, stats, st = pkg.decode(pkg.WindModel(w2), enc, lens, 2, 1, window_greedy=True)
    assert list(tok[0, : olen[0]]) == [1] and list(frm[0, : olen[0]]) == [1] and stats["jump_hist"][1] == 1


@pytest.mark.parametrize("seed,W,S,act,blank0,L,bias", [
    (0, 4, 3, 0, False, 1, 1.0), (1, 8, 2, 1, True, 2, 0.5), (2, 1, 5, 0, False, 1, 0.0), (3, 13, 1, 1, False, 2, 1.5),
    (4, 64, 10, 0, True, 1, 2.5)])
def test_fp32_ragged_shapes(pkg, seed, W, S, act, blank0, L, bias):
    w, enc, lens = ragged_case(500 + seed, B=7, T=50, D=24, E=20, P=24, L=L, H=40, V=37, act=act,
                               blank_id=0 if blank0 else None, bias=bias)
    rep, _ = check_window_greedy(pkg, w, enc, lens, W, S)
    assert rep["exact"] >= 5


def test_fp32_one_frame_window_equals_greedy_decoding_on_the_gpu(pkg):
    w, enc, lens = ragged_case(510, B=6, T=40, D=24, E=20, P=24, L=1, H=40, V=37, bias=1.0)
    model = pkg.WindModel(w)
    a = pkg.decode(model, enc, lens, 1, 3, window_greedy=True)
    b = pkg.decode(model, enc, lens, 1, 3)
    assert np.array_equal(a[2], b[2]) and np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("kernels", [1, 2])
@pytest.mark.parametrize("L,W,B", [(1, 4, 9), (2, 8, 33), (1, 16, 70)])
def test_bf16_both_kernel_sets(pkg, kernels, L, W, B):
    w, enc, lens = ragged_case(520 + L + W, B=B, T=40, D=64, E=64, P=128, L=L, H=128, V=300, act=L % 2, bias=1.5, dtype="bf16")
    rep, _ = check_window_greedy(pkg, w, enc, lens, W, 3, kernels=kernels)
    assert rep["stats"]["kernels"] == kernels


def test_bf16_streaming_mode_of_the_loop_kernel(pkg, monkeypatch):
    pkg.wind_set_loop_options(resident=False)
    w, enc, lens = ragged_case(531, B=150, T=30, D=64, E=64, P=64, L=1, H=128, V=257, act=0, bias=1.5, dtype="bf16")
    rep, _ = check_window_greedy(pkg, w, enc, lens, 8, 3, kernels=2)
    assert rep["stats"]["kernels"] == 2


def test_cfg3_full_batch_sampled_utterances(pkg):
    # the benchmark's workload and launch configuration; the oracle replays a sample of the utterances
    cfg = ws.CONFIGS["cfg3_large_b128"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights)
    tok, frm, olen, stats, st = pkg.decode(model, enc, lens, cfg.W, cfg.S, window_greedy=True)
    assert st == 0 and stats["kernels"] == 2 and stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
    hist = np.array(stats["jump_hist"])
    assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum())
    om = oracle.Model(weights)
    order = np.argsort(lens)
    sample = [int(order[0]), int(order[len(order) // 4]), int(order[len(order) // 2])]   # the oracle's replay of the longest one alone takes two minutes

    def replay(b):
        return oracle.replay_verify_window(om, enc[b], int(lens[b]), cfg.W, cfg.S, tok[b, : olen[b]], frm[b, : olen[b]], MARGIN)

    with ThreadPoolExecutor(3) as ex:
        reps = list(ex.map(replay, sample))
    for b, r in zip(sample, reps):
        assert r["rc"] == 0, f"utterance {b}: {r}"
    print("[window-greedy cfg3]", [(b, int(lens[b]), r["decisions"], r["not_argmax"]) for b, r in zip(sample, reps)])


@pytest.mark.parametrize("mode", LOOP_MODES)
def test_bf16_tensor_path_wide_window_and_overflow(pkg, mode):
    # W = 40: more window rows than lanes in the decision warp; then an output buffer that is too small
    set_loop_mode(pkg, mode)
    w, enc, lens = ragged_case(540, B=6, T=70, D=64, E=64, P=64, L=1, H=128, V=150, act=1, bias=3.0, dtype="bf16")
    rep, (tok, frm, olen) = check_window_greedy(pkg, w, enc, lens, 40, 2, kernels=2)
    assert rep["stats"]["kernels"] == 2 and olen.max() > 4
    model = pkg.WindModel(w)
    prev = pkg.wind_set_kernels(2)
    try:
        t2, f2, o2, _, st = pkg.decode(model, enc, lens, 40, 2, max_out=4, check=False, window_greedy=True)
    finally:
        pkg.wind_set_kernels(prev)
    assert st == pkg.binding.WIND_ERR_OUTPUT_OVERFLOW and o2.max() == 4
    for b in range(6):
        n = min(4, olen[b])
        assert o2[b] == n and np.array_equal(t2[b, :n], tok[b, :n]) and np.array_equal(f2[b, :n], frm[b, :n])


def test_bf16_resident_joint_in_waves(pkg):
    # 33 vocabulary tiles leave four CTAs per tile: 480 window rows take two waves of 96-row groups per CTA
    w, enc, lens = ragged_case(550, B=60, T=24, D=64, E=64, P=64, L=1, H=64, V=4099, act=0, bias=2.0, dtype="bf16")
    rep, _ = check_window_greedy(pkg, w, enc, lens, 8, 3, kernels=2)
    assert rep["stats"]["kernels"] == 2
