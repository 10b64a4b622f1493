"""GPU parity of WIND beam search (Algorithm 3, one utterance) against the oracle.

The search takes discrete decisions (which K entries of P', which K hypotheses survive) on log-probabilities that the
GPU computes in fp32 and the oracle in fp64.  The oracle reports the smallest log-probability difference that decided
anything in its own run (min_gap); when it is well above the GPU's arithmetic error the two searches must agree
exactly (tokens and frames of every final hypothesis, scores within the accumulated rounding), otherwise the case is
only counted.  Most cases must be decidable."""
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.join(os.path.dirname(__file__), ".."))
sys.path.insert(0, os.path.dirname(__file__))

import oracle
import wind_synth as ws
from naive_model import random_weights
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


def small_model(seed, dtype="f32", V=37, L=1, act=0, blank0=False, bias=1.5):
    r = np.random.default_rng(7000 + seed)
    w = random_weights(r, 24, 20, 24, L, 40, V, blank_id=0 if blank0 else None, act=act, blank_bias=bias, bias_scale=0.1)
    w["dtype"] = dtype
    if dtype == "bf16":
        for k in ("emb", "w_enc", "w_pred", "w_out"):
            w[k] = ws.bf16_round(w[k])
        w["w_ih"] = [ws.bf16_round(a) for a in w["w_ih"]]
        w["w_hh"] = [ws.bf16_round(a) for a in w["w_hh"]]
    return w, r


def compare(pkg, w, enc, W, K, S, gap_needed, tol, prefix_search=False, round_bf16=False):
    """Returns True when the case was decidable and the GPU agreed with the oracle (round_bf16: the oracle that rounds
    enc_proj, the hidden state and the joint's activations to bf16 where the bf16 kernels do)."""
    T = enc.shape[0]
    want, gap, steps = oracle.beam_search(oracle.Model(w, round_bf16=round_bf16), enc, T, W, K, S, max_hyps=256,
                                          prefix_search=prefix_search)
    got, gsteps, st = pkg.wind_beam_search(pkg.WindModel(w), enc, W, K, S, max_hyps=256, prefix_search=prefix_search)
    assert st == 0 and len(got) >= 1
    for tok, frm, sc in got:                      # always: well-formed hypotheses
        assert len(tok) == len(frm) and np.all(np.diff(frm) >= 0) and (len(frm) == 0 or frm.max() < T)
        assert len(frm) == 0 or np.bincount(frm).max() <= S
        assert np.all(tok != w["blank_id"]) and np.isfinite(sc) and sc <= 1e-6
    assert [g[2] for g in got] == sorted([g[2] for g in got], reverse=True)
    if gap < gap_needed:
        return False
    assert gsteps == steps
    assert list(got[0][0]) == list(want[0][0]) and list(got[0][1]) == list(want[0][1])
    a = {tuple(int(x) for x in h[0]): h for h in want}
    b = {tuple(int(x) for x in h[0]): h for h in got}
    assert set(a) == set(b)
    worst = 0.0
    for k in a:
        assert abs(a[k][2] - b[k][2]) < tol, (k, a[k][2], b[k][2])
        assert list(a[k][1]) == list(b[k][1])
        worst = max(worst, abs(a[k][2] - b[k][2]))
    print(f"[beam case] W={W} K={K} T={T} steps={steps} oracle min gap {gap:.2e}, worst score difference {worst:.2e}")
    return True


def test_worked_example_fp32(pkg):
    # A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1); utterance A B, W = 2, S = 1, K = 2:
    # [] -> {[x] .45, [y] .4}; [x] at frame 1 -> {[x,y] .36, [x,x] .045} (x before blank on the .1 tie); final [y] .4 wins.
    w = table_model([[.45, .05, .5], [.1, .8, .1]])
    enc = np.eye(2, dtype=np.float32)[[0, 1]]
    hyps, steps, st = pkg.wind_beam_search(pkg.WindModel(w), enc, 2, 2, 1)
    assert st == 0 and steps == 2
    assert [list(h[0]) for h in hyps] == [[1], [0, 1], [0, 0]] and [list(h[1]) for h in hyps] == [[1], [0, 1], [0, 1]]
    assert np.allclose([h[2] for h in hyps], np.log([.4, .36, .045]), atol=1e-5)
    one, _, _ = pkg.wind_beam_search(pkg.WindModel(w), enc, 2, 1, 1)
    assert list(one[0][0]) == [0, 1] and abs(one[0][2] - np.log(.36)) < 1e-5


@pytest.mark.parametrize("W,K,S,L,blank0,act", [(1, 2, 3, 1, False, 0), (4, 3, 3, 1, True, 1), (8, 4, 2, 2, False, 0), (3, 2, 10, 1, False, 1),
                                               (16, 4, 4, 1, True, 0)])
def test_fp32_matches_the_oracle_when_the_search_is_decidable(pkg, W, K, S, L, blank0, act):
    # fp32 arithmetic: measured score differences against the oracle are 1e-6 .. 3e-6 over 30 .. 180 iterations; a case
    # counts as decidable when the oracle's smallest deciding difference is 25 times that
    decided = 0
    for seed in range(8):
        w, r = small_model(seed + 10 * W, L=L, act=act, blank0=blank0, bias=2.5)
        T = int(r.integers(12, 24))
        enc = r.standard_normal((T, 24)).astype(np.float32)
        decided += compare(pkg, w, enc, W, K, S, gap_needed=5e-5, tol=1e-4)
    print(f"[beam] W={W} K={K} S={S}: {decided}/8 cases decidable and equal to the oracle")
    assert decided >= 4


def test_prefix_step_worked_example_fp32(pkg):
    # A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1); utterance A B, W = 1, S = 2, K = 2 (derivation: the
    # oracle's pin of the same example): at t = 1 the list {[] .5, [x,x] .2025, [x] .225} becomes {[x,x] .23}
    w = table_model([[.45, .05, .5], [.1, .8, .1]])
    enc = np.eye(2, dtype=np.float32)[[0, 1]]
    hyps, steps, st = pkg.wind_beam_search(pkg.WindModel(w), enc, 1, 2, 2, prefix_search=True)
    assert st == 0 and steps == 4
    assert [list(h[0]) for h in hyps] == [[0, 0, 1, 1], [0, 0, 1, 0], [0, 0, 0, 1], [0, 0, 0, 0]]
    assert np.allclose(np.exp([h[2] for h in hyps]), [.1472, .0184, .0184, .0023], atol=1e-6)


@pytest.mark.parametrize("W,K,S,L,bias", [(1, 2, 3, 1, 2.5), (1, 4, 2, 2, 1.5), (8, 4, 2, 1, 2.5)])
def test_fp32_with_the_prefix_step_matches_the_oracle_when_decidable(pkg, W, K, S, L, bias):
    decided = changed = 0
    for seed in range(8):
        w, r = small_model(400 + seed + 10 * W, L=L, bias=bias)
        T = int(r.integers(12, 24))
        enc = r.standard_normal((T, 24)).astype(np.float32)
        decided += compare(pkg, w, enc, W, K, S, gap_needed=5e-5, tol=1e-4, prefix_search=True)
        a, _, _ = oracle.beam_search(oracle.Model(w), enc, T, W, K, S, max_hyps=256)
        b, _, _ = oracle.beam_search(oracle.Model(w), enc, T, W, K, S, max_hyps=256, prefix_search=True)
        da = {tuple(int(x) for x in h[0]): h[2] for h in a}
        db = {tuple(int(x) for x in h[0]): h[2] for h in b}
        changed += set(da) != set(db) or any(abs(da[k] - db[k]) > 1e-9 for k in da)
    print(f"[beam] prefix step, W={W} K={K} S={S}: {decided}/8 cases decidable and equal to the oracle; "
          f"the step changes the final hypotheses in {changed}/8")
    assert decided >= 3 and changed >= 3       # the cases do contain prefix pairs


def test_bf16_best_score_is_close_to_the_oracle(pkg):
    # bf16 weights: the kernels also round activations to bf16, so logits differ from the oracle's by about 1e-2 and
    # the discrete search is hardly ever decidable at that error; what must hold is that the hypotheses are well
    # formed (checked in compare) and that the best score is close to the oracle's
    same = 0
    for seed in range(6):
        w, r = small_model(100 + seed, dtype="bf16", bias=2.5)
        T = int(r.integers(12, 20))
        enc = ws.bf16_round(r.standard_normal((T, 24)).astype(np.float32))
        compare(pkg, w, enc, 4, 2, 3, gap_needed=1e9, tol=0.0)
        want, gap, _ = oracle.beam_search(oracle.Model(w), enc, T, 4, 2, 3)
        got, _, _ = pkg.wind_beam_search(pkg.WindModel(w), enc, 4, 2, 3)
        assert abs(got[0][2] - want[0][2]) < 0.02 * (len(want[0][0]) + T), (got[0][2], want[0][2])
        same += list(got[0][0]) == list(want[0][0])
    print(f"[beam bf16] best hypothesis equal to the oracle's in {same}/6 cases")


@pytest.mark.parametrize("W,K,S,L,blank0,act,prefix", [(1, 2, 3, 1, False, 0, False), (4, 3, 3, 1, True, 1, False),
                                                      (8, 4, 2, 2, False, 0, False), (4, 2, 3, 1, False, 0, True),
                                                      (16, 4, 4, 1, True, 0, False)])
def test_bf16_matches_the_oracle_that_rounds_where_the_kernels_do(pkg, W, K, S, L, blank0, act, prefix):
    # bf16 weights: the kernels round enc_proj, the hidden state and the joint's activations to bf16.  Against the oracle
    # in the same precision (Model(round_bf16=True): fp64 sums, the same three roundings) what is left is the kernels' fp32
    # accumulation: scores agree to about 1e-6, except where an fp32 sum falls on the other side of a bf16 rounding
    # boundary than the fp64 sum (one last-place step of one value: up to about 1e-3 in a score).  A case is decidable
    # when the oracle's smallest deciding difference is four times the largest score difference measured in it; then
    # every final hypothesis (tokens, frames) and the number of iterations must be the oracle's.
    decided = 0
    for seed in range(8):
        w, r = small_model(500 + seed + 10 * W, dtype="bf16", L=L, act=act, blank0=blank0, bias=2.5)
        T = int(r.integers(12, 24))
        enc = ws.bf16_round(r.standard_normal((T, 24)).astype(np.float32))
        want, gap, steps = oracle.beam_search(oracle.Model(w, round_bf16=True), enc, T, W, K, S, max_hyps=256, prefix_search=prefix)
        got, gsteps, st = pkg.wind_beam_search(pkg.WindModel(w), enc, W, K, S, max_hyps=256, prefix_search=prefix)
        assert st == 0 and len(got) >= 1
        a = {tuple(int(x) for x in h[0]): h for h in want}
        b = {tuple(int(x) for x in h[0]): h for h in got}
        worst = max((abs(a[k][2] - b[k][2]) for k in a if k in b), default=0.0)
        assert worst < 5e-3, (seed, worst)
        if gap >= 4 * max(worst, 1e-6):
            assert gsteps == steps and set(a) == set(b), (seed, gap, worst)
            assert all(list(a[k][1]) == list(b[k][1]) for k in a)
            assert list(got[0][0]) == list(want[0][0])
            decided += 1
    print(f"[beam bf16] W={W} K={K} S={S} prefix={prefix}: {decided}/8 cases decidable and equal to the rounding oracle")
    assert decided >= 5


def test_beam_one_equals_window_based_greedy_on_the_gpu(pkg):
    w, r = small_model(200)
    T = 30
    enc = r.standard_normal((T, 24)).astype(np.float32)
    model = pkg.WindModel(w)
    hyps, steps, st = pkg.wind_beam_search(model, enc, 4, 1, 3)
    want, gap, osteps = oracle.beam_search(oracle.Model(w), enc, T, 4, 1, 3)
    if gap > 2e-3:
        tok, frm, olen, stats, _ = pkg.decode(model, enc[None], np.array([T], np.int32), 4, 3, window_greedy=True)
        assert list(hyps[0][0]) == list(tok[0, : olen[0]]) and list(hyps[0][1]) == list(frm[0, : olen[0]])
        assert steps == stats["steps"]


def test_arguments(pkg):
    w, r = small_model(300)
    model = pkg.WindModel(w)
    enc = r.standard_normal((10, 24)).astype(np.float32)
    assert pkg.wind_beam_search(model, enc, 4, 17, 3, check=False)[2] == pkg.binding.WIND_ERR_UNSUPPORTED
    assert pkg.wind_beam_search(model, enc, 65, 2, 3, check=False)[2] == pkg.binding.WIND_ERR_UNSUPPORTED
    hyps, _, st = pkg.wind_beam_search(model, enc, 4, 2, 3, max_hyps=1)
    assert st == 0 and len(hyps) == 1
