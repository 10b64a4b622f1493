"""Randomised shapes against the oracle (fixed seeds): the tile planner of the loop kernel has many branches (which
mode, how many utterances per decoder / projection CTA, where the W_out tile lives, who records the steps), and the
shapes of the named configs reach only a few of them.  Every case is a full decode (Algorithm 2 or window-based
greedy) or a teacher-forced logits comparison on the tensor-core path."""
import os
import sys

import numpy as np
import pytest

from conftest import LOOP_MODES, set_loop_mode
import torch

sys.path.insert(0, os.path.join(os.path.dirname(__file__), ".."))
sys.path.insert(0, os.path.dirname(__file__))

import test_gpu_parity as tp
import test_gpu_window_greedy as tw

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


@pytest.mark.parametrize("seed", [1, 3])
def test_small_dimensions_many_utterances(pkg, monkeypatch, seed):
    r = np.random.default_rng(seed)
    for i in range(20):
        P = int(r.choice([64, 128, 192, 256, 320])); H = int(r.choice([64, 128, 192, 256, 320, 640]))
        V = int(r.integers(127, 700)); B = int(r.choice([1, 2, 7, 31, 64, 65, 128, 129, 200, 333]))
        W = int(r.choice([1, 2, 3, 5, 8, 13, 16, 24, 40])); L = int(r.choice([1, 1, 2, 2, 3])); S = int(r.integers(1, 6))
        act = int(r.integers(0, 2)); blank0 = bool(r.integers(0, 2)); res = int(r.integers(0, 2)); T = int(r.integers(8, 40))
        mode = LOOP_MODES[(2 * res + i) % 3]
        win = bool(r.integers(0, 3) == 0)
        set_loop_mode(pkg, mode)
        w, enc, lens = tp.ragged_case(9000 + i, B=B, T=T, D=64, E=int(r.choice([64, 128])), P=P, L=L, H=H, V=V, act=act,
                                      blank_id=0 if blank0 else None, bias=float(r.uniform(0.5, 3.0)), dtype="bf16")
        print(f"case {i}: B={B} T={T} W={W} S={S} P={P} H={H} V={V} L={L} mode={mode} window={win}", flush=True)
        if win:
            tw.check_window_greedy(pkg, w, enc, lens, W, S, kernels=2)
        else:
            tp.check_against_oracle(pkg, w, enc, lens, W, S, kernels=2)


def test_large_dimensions(pkg, monkeypatch):
    r = np.random.default_rng(11)
    for i in range(16):
        P = int(r.choice([64, 320, 512, 640, 1024])); H = int(r.choice([64, 256, 512, 640, 1024]))
        V = int(r.choice([127, 128, 255, 256, 257, 1024, 2000, 4099])); B = int(r.choice([1, 3, 16, 32, 64, 100, 128, 160]))
        W = int(r.choice([1, 2, 4, 8, 16, 32, 64])); L = int(r.choice([1, 2])); S = int(r.integers(1, 11)); act = int(r.integers(0, 2))
        res = int(r.integers(0, 2)); T = int(r.integers(4, 16)); kind = int(r.integers(0, 4)); D = int(r.choice([64, 512]))
        E = int(r.choice([64, 640]))
        mode = LOOP_MODES[(2 * res + i) % 3]
        set_loop_mode(pkg, mode)
        w, enc, lens = tp.ragged_case(9500 + i, B=B, T=T, D=D, E=E, P=P, L=L, H=H, V=V, act=act, blank_id=0 if i % 3 == 0 else None,
                                      bias=float(r.uniform(0.5, 3.0)), dtype="bf16")
        print(f"case {i}: kind={kind} B={B} T={T} W={W} S={S} D={D} E={E} P={P} H={H} V={V} L={L} mode={mode}", flush=True)
        if kind == 0:
            tw.check_window_greedy(pkg, w, enc, lens, W, S, kernels=2)
        elif kind == 1:
            tp.logits_parity(pkg, w, enc, lens, W=W, S=S, tol=tp.TOL["bf16"], n_windows=B, kernels=2)
        else:
            tp.check_against_oracle(pkg, w, enc, lens, W, S, kernels=2)


def refill_case(pkg, r, i, seed_base):
    """One random (model, utterances, rows) case: refilled rows against one batch of all utterances, same loop mode."""
    P = int(r.choice([64, 128, 192, 256, 640])); H = int(r.choice([64, 128, 256, 640]))
    V = int(r.choice([127, 140, 300, 1024, 2100])); N = int(r.choice([1, 2, 9, 40, 77, 130, 200]))
    B = int(r.choice([1, 2, 5, 16, 33, 64, 128, 150])); W = int(r.choice([1, 2, 4, 8, 13, 16, 32])); L = int(r.choice([1, 1, 2, 3]))
    S = int(r.integers(1, 6)); act = int(r.integers(0, 2)); T = int(r.integers(4, 30))
    mode = ["barriers", "streaming"][i % 2]
    set_loop_mode(pkg, mode)
    w, enc, lens = tp.ragged_case(seed_base + i, B=N, T=T, D=64, E=64, P=P, L=L, H=H, V=V, act=act,
                                  blank_id=0 if i % 3 == 0 else None, bias=float(r.uniform(0.5, 3.0)), dtype="bf16")
    enc = np.nan_to_num(enc)
    print(f"refill case {i}: N={N} rows={B} T={T} W={W} S={S} P={P} H={H} V={V} L={L} mode={mode}", flush=True)
    model = pkg.WindModel(w)
    # the reference decodes the utterances in fixed batches of exactly B rows (the last one padded with empty utterances),
    # so that both sides run the same tile plan, hence the same kernel and arithmetic
    tok1 = np.full((N, max(1, T * S)), -1, np.int32); frm1 = tok1.copy(); olen1 = np.zeros(N, np.int32)
    for k in range(0, N, B):
        m = min(B, N - k)
        e = np.zeros((B,) + enc.shape[1:], enc.dtype); l = np.zeros(B, np.int32)
        e[:m], l[:m] = enc[k: k + m], lens[k: k + m]
        t_, f_, o_, _, st1 = pkg.decode(model, e, l, W, S)
        assert st1 == 0
        tok1[k: k + m], frm1[k: k + m], olen1[k: k + m] = t_[:m], f_[:m], o_[:m]
    tok, frm, olen, stats, st = pkg.decode_refill(model, enc, lens, B, W, S)
    assert st == 0 and stats["kernels"] == 2
    assert np.array_equal(olen, olen1)
    for u in range(N):
        assert np.array_equal(tok[u, : olen[u]], tok1[u, : olen1[u]]) and np.array_equal(frm[u, : olen[u]], frm1[u, : olen1[u]]), u
    assert stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
    hist = np.array(stats["jump_hist"])
    assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum())


def test_refilled_rows_random_shapes(pkg):
    r = np.random.default_rng(21)
    for i in range(24):
        refill_case(pkg, r, i, 9700)
