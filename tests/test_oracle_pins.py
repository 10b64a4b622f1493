"""Pins for the CPU oracle: closed forms, library fp64 routines, brute force, invariants.

The paper prints no worked numeric example, so the oracle is fixed by what the
paper and the mathematics fix instead:
  * Algorithm 2 returns exactly Algorithm 1's result for every window size
    (results section: identical accuracy at every W; method section: frames
    skipped by a jump are blank under the same decoder state);
  * the blank / non-blank rules of the background section, checked by brute
    force with an independent evaluator that re-runs a library LSTM over the
    whole prefix;
  * linear layers and the LSTM cell against library fp64 routines and closed forms.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from naive_model import NaiveModel, random_weights, tie_expected, tie_model, tie_utterances


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------------------
# linear layers, LSTM cell, joint: library routines and closed forms
# ---------------------------------------------------------------------------
def test_linear_matches_fp64_matmul():
    r = rng(1)
    W = r.standard_normal((37, 53)).astype(np.float32)
    b = r.standard_normal(37).astype(np.float32)
    x = r.standard_normal(53)
    y = oracle.linear(W, b, x)
    ref = W.astype(np.float64) @ x + b.astype(np.float64)
    assert np.max(np.abs(y - ref)) < 1e-12
    # a transposed operand or a dropped bias must show
    assert np.max(np.abs(y - (W.astype(np.float64) @ x))) > 1e-3
    y0 = oracle.linear(W, None, x)
    assert np.max(np.abs(y0 - W.astype(np.float64) @ x)) < 1e-12


def test_linear_unit_vectors_pick_columns():
    W = np.arange(12, dtype=np.float32).reshape(3, 4)
    for k in range(4):
        x = np.zeros(4)
        x[k] = 1.0
        assert np.array_equal(oracle.linear(W, None, x), W[:, k].astype(np.float64))


def test_lstm_zero_weights_closed_form():
    # all matrices zero: gates are the bias sums; from zero state
    # c = sigma(bi) * tanh(bg), h = sigma(bo) * tanh(c); f plays no role at step 1,
    # at step 2 c2 = sigma(bf) * c + sigma(bi) * tanh(bg).
    P, E, V = 3, 2, 4
    w = random_weights(rng(2), 2, E, P, 1, 2, V)
    w["w_ih"] = [np.zeros((4 * P, E), np.float32)]
    w["w_hh"] = [np.zeros((4 * P, P), np.float32)]
    bi, bf, bg, bo = 0.3, -0.7, 1.1, 0.4
    b = np.concatenate([np.full(P, v, np.float32) for v in (bi, bf, bg, bo)])
    w["b_ih"] = [b / 2]
    w["b_hh"] = [b / 2]
    m = oracle.Model(w)
    sig = lambda v: 1.0 / (1.0 + np.exp(-np.float64(np.float32(v))))
    bg64 = np.float64(np.float32(bg))
    h, c = oracle.lstm_step(m, 1, np.zeros((1, P)), np.zeros((1, P)))
    c1 = sig(bi) * np.tanh(bg64)
    assert np.allclose(c, c1, atol=1e-7) and np.allclose(h, sig(bo) * np.tanh(c1), atol=1e-7)
    h, c = oracle.lstm_step(m, 2, h, c)
    c2 = sig(bf) * c1 + sig(bi) * np.tanh(bg64)
    assert np.allclose(c, c2, atol=1e-7) and np.allclose(h, sig(bo) * np.tanh(c2), atol=1e-7)


def test_lstm_all_zero_gives_zero_state():
    P, E, V = 4, 3, 5
    w = random_weights(rng(3), 2, E, P, 2, 2, V)
    for k in ("w_ih", "w_hh", "b_ih", "b_hh"):
        w[k] = [np.zeros_like(a) for a in w[k]]
    m = oracle.Model(w)
    h, c = oracle.lstm_step(m, 2, np.zeros((2, P)), np.zeros((2, P)))
    assert np.all(h == 0) and np.all(c == 0)


@pytest.mark.parametrize("L", [1, 2, 3])
def test_lstm_matches_torch_lstm(L):
    r = rng(10 + L)
    D, E, P, H, V = 5, 7, 6, 4, 9
    w = random_weights(r, D, E, P, L, H, V, bias_scale=0.5, emb_zero_blank=False)
    m = oracle.Model(w)
    nm = NaiveModel(w)
    prefix = [3, 0, 8, 8, 1]
    h = np.zeros((L, P))
    c = np.zeros((L, P))
    h, c = oracle.lstm_step(m, w["blank_id"], h, c)
    for k, tok in enumerate(prefix):
        h, c = oracle.lstm_step(m, tok, h, c)
        h_top, hn, cn = nm.decoder(prefix[: k + 1])
        assert np.max(np.abs(h - hn.numpy())) < 1e-12
        assert np.max(np.abs(c - cn.numpy())) < 1e-12
    g = oracle.pred_proj(m, h)
    ref = w["w_pred"].astype(np.float64) @ h[-1] + w["b_pred"].astype(np.float64)
    assert np.max(np.abs(g - ref)) < 1e-12


def to_bf16(a):
    """Library rounding to bf16 (torch), as fp64 numpy."""
    return torch.as_tensor(np.asarray(a, np.float64)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def test_bf16_rounding_matches_the_library_conversion():
    r = rng(31)
    xs = np.concatenate([r.standard_normal(2000), r.standard_normal(500) * 1e-3, r.standard_normal(500) * 1e4,
                         # exact ties between two bf16 neighbours (even and odd), and values that are already bf16
                         np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 1.0, -2.5, 3.140625])])
    ref = to_bf16(xs)
    got = np.array([oracle.bf16_round(x) for x in xs])
    assert np.array_equal(got, ref)
    assert oracle.bf16_round(1.00390625) == 1.0 and oracle.bf16_round(1.01171875) == 1.015625    # ties go to the even pattern


@pytest.mark.parametrize("L,act", [(1, 0), (2, 1)])
def test_rounding_mode_rounds_enc_proj_hidden_state_and_activations_and_nothing_else(L, act):
    # Model(round_bf16=True): the three quantities a bf16 implementation keeps as matrix operands are rounded where they
    # are produced.  Recomputed here step by step with library fp64 routines and the library's bf16 conversion.
    r = rng(40 + L)
    D, E, P, H, V = 6, 5, 7, 8, 9
    w = random_weights(r, D, E, P, L, H, V, act=act, bias_scale=0.4, emb_zero_blank=False)
    m = oracle.Model(w, round_bf16=True)
    m0 = oracle.Model(w)
    f64 = lambda a: np.asarray(a, np.float64)
    enc = r.standard_normal((5, D)).astype(np.float32)
    ep = oracle.enc_proj(m, enc)
    ref_ep = to_bf16(f64(enc) @ f64(w["w_enc"]).T + f64(w["b_enc"]))
    assert np.array_equal(ep, ref_ep)
    assert np.max(np.abs(ep - oracle.enc_proj(m0, enc))) > 1e-4          # the flag does something
    # LSTM: the rounded h is what feeds the next layer and the next update; c is not rounded
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    h = np.zeros((L, P)); c = np.zeros((L, P)); hr = np.zeros((L, P)); cr = np.zeros((L, P))
    for tok in [w["blank_id"], 3, 8, 8, 0, 1]:
        h, c = oracle.lstm_step(m, tok, h, c)
        x = f64(w["emb"][tok])
        for l in range(L):
            g = f64(w["w_ih"][l]) @ x + f64(w["b_ih"][l]) + f64(w["w_hh"][l]) @ hr[l] + f64(w["b_hh"][l])
            gi, gf, gg, go = sig(g[:P]), sig(g[P:2 * P]), np.tanh(g[2 * P:3 * P]), sig(g[3 * P:])
            cr[l] = gf * cr[l] + gi * gg
            hr[l] = to_bf16(go * np.tanh(cr[l]))
            x = hr[l]
        assert np.array_equal(h, hr)
        assert np.max(np.abs(c - cr)) < 1e-12
    assert np.max(np.abs(c - to_bf16(c))) > 1e-6                           # c keeps its precision
    # pred_proj is not rounded; the joint's activations are
    g = oracle.pred_proj(m, h)
    ref_g = f64(w["w_pred"]) @ hr[-1] + f64(w["b_pred"])
    assert np.max(np.abs(g - ref_g)) < 1e-12 and np.max(np.abs(g - to_bf16(g))) > 1e-6
    lg = oracle.joint_logits(m, ep[2], g)
    sgm = ref_ep[2] + ref_g
    z = to_bf16(np.maximum(sgm, 0) if act == 0 else np.tanh(sgm))
    assert np.max(np.abs(lg - (f64(w["w_out"]) @ z + f64(w["b_out"])))) < 1e-12
    # and the decoding entry points go through the same functions: a decode with the flag differs from one without it only
    # through these roundings (same code path: W-invariance still holds)
    enc_b = r.standard_normal((2, 30, D)).astype(np.float32)
    lens = np.array([30, 17], np.int32)
    a = oracle.decode_batch(m, enc_b, lens, W=0, S=3)
    b = oracle.decode_batch(m, enc_b, lens, W=5, S=3)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])


@pytest.mark.parametrize("act", [0, 1])
def test_enc_proj_and_joint_match_fp64(act):
    r = rng(20 + act)
    D, E, P, H, V = 6, 4, 5, 8, 7
    w = random_weights(r, D, E, P, 1, H, V, act=act, bias_scale=0.3)
    m = oracle.Model(w)
    enc = r.standard_normal((9, D)).astype(np.float32)
    ep = oracle.enc_proj(m, enc)
    ref = enc.astype(np.float64) @ w["w_enc"].astype(np.float64).T + w["b_enc"].astype(np.float64)
    assert np.max(np.abs(ep - ref)) < 1e-12
    g = r.standard_normal(H)
    lg = oracle.joint_logits(m, ep[4], g)
    s = ref[4] + g
    z = np.maximum(s, 0) if act == 0 else np.tanh(s)
    ref_l = w["w_out"].astype(np.float64) @ z + w["b_out"].astype(np.float64)
    assert np.max(np.abs(lg - ref_l)) < 1e-12
    # the other activation must differ (guards against an ignored act flag)
    z2 = np.tanh(s) if act == 0 else np.maximum(s, 0)
    assert np.max(np.abs(lg - (w["w_out"].astype(np.float64) @ z2 + w["b_out"]))) > 1e-3


def test_eval_joint_window_matches_independent_evaluator():
    r = rng(30)
    D, E, P, H, V = 5, 4, 6, 7, 6
    w = random_weights(r, D, E, P, 2, H, V, act=1, bias_scale=0.2, blank_id=2)
    m = oracle.Model(w)
    nm = NaiveModel(w)
    T = 11
    enc = r.standard_normal((T, D)).astype(np.float32)
    prefix = [0, 5, 1, 1]
    for t0, W in [(0, 4), (9, 4), (3, 1), (10, 16)]:
        lg, g, h, c = oracle.eval_joint_window(m, enc, T, prefix, t0, W)
        assert lg.shape[0] == min(W, T - t0)
        for k in range(lg.shape[0]):
            assert np.max(np.abs(lg[k] - nm.logits(enc[t0 + k], prefix))) < 1e-11


# ---------------------------------------------------------------------------
# brute force: tabulate argmax joint(t, prefix) with the independent evaluator
# ---------------------------------------------------------------------------
def brute_force_greedy(nm, enc, S):
    """Algorithm 1's rules walked on independently evaluated logits.

    Background-section rules: a non-blank label is appended and the frame is kept;
    blank advances the frame and keeps the decoder input.  The S cap forces an
    advance after the S-th consecutive emission on one frame.
    """
    T = enc.shape[0]
    hyp, frames, t, count = [], [], 0, 0
    while t < T:
        lg = nm.logits(enc[t], hyp)
        label = int(np.argmax(lg))  # numpy argmax returns the first maximum
        if label != nm.blank:
            hyp.append(label)
            frames.append(t)
            count += 1
            if count == S:
                t += 1
                count = 0
        else:
            t += 1
            count = 0
    return hyp, frames


@pytest.mark.parametrize("seed,blank_id,act,S,bias", [
    (0, None, 0, 2, 0.0), (1, 0, 1, 3, 0.5), (2, 1, 0, 1, -0.5), (3, None, 1, 4, 1.0), (4, 2, 0, 2, 0.3),
    (5, None, 0, 3, -2.0),
])
def test_sequential_greedy_matches_brute_force(seed, blank_id, act, S, bias):
    r = rng(100 + seed)
    D, E, P, H, V, L = 3, 3, 4, 4, 3, 1 + seed % 2
    w = random_weights(r, D, E, P, L, H, V, blank_id=blank_id, act=act, blank_bias=bias, bias_scale=0.3,
                       emb_zero_blank=False)
    nm = NaiveModel(w)
    m = oracle.Model(w)
    T = 6
    enc = r.standard_normal((1, T, D)).astype(np.float32)
    hyp, frames = brute_force_greedy(nm, enc[0], S)
    tok, frm, n, st = oracle.decode_batch(m, enc, np.array([T], np.int32), W=0, S=S)
    assert list(tok[0, : n[0]]) == hyp
    assert list(frm[0, : n[0]]) == frames
    for W in (1, 2, 3, 5, 6, 11):
        tokw, frmw, nw, _ = oracle.decode_batch(m, enc, np.array([T], np.int32), W=W, S=S)
        assert list(tokw[0, : nw[0]]) == hyp, W
        assert list(frmw[0, : nw[0]]) == frames, W


def test_brute_force_table_over_all_reachable_prefixes():
    # tiny enough to enumerate: T=4, V=2, S=2 -> every (t, prefix) reachable under the cap
    r = rng(200)
    D, E, P, H, V, S, T = 2, 2, 3, 3, 2, 2, 4
    w = random_weights(r, D, E, P, 1, H, V, blank_bias=0.2, bias_scale=0.2, emb_zero_blank=False)
    nm, m = NaiveModel(w), oracle.Model(w)
    enc = r.standard_normal((T, D)).astype(np.float32)
    checked = 0
    for n in range(0, 4):
        for prefix in itertools.product(range(V), repeat=n):
            for t0 in range(T):
                lg, *_ = oracle.eval_joint_window(m, enc, T, list(prefix), t0, 1)
                ref = nm.logits(enc[t0], list(prefix))
                assert int(np.argmax(lg[0])) == int(np.argmax(ref))
                assert np.max(np.abs(lg[0] - ref)) < 1e-11
                checked += 1
    assert checked == (1 + 2 + 4 + 8) * T


# ---------------------------------------------------------------------------
# invariants of the decoding loops
# ---------------------------------------------------------------------------
def small_case(seed, B=3, T=40, bias=1.0, S=3, V=12, L=1, act=0, blank_id=None):
    r = rng(300 + seed)
    D, E, P, H = 8, 6, 7, 10
    w = random_weights(r, D, E, P, L, H, V, blank_id=blank_id, act=act, blank_bias=bias, bias_scale=0.1)
    lens = r.integers(0, T + 1, size=B).astype(np.int32)
    lens[0] = T
    enc = r.standard_normal((B, T, D)).astype(np.float32)
    for b in range(B):
        enc[b, lens[b]:] = np.nan  # poison: padded frames must never be decoded
    return w, enc, lens


@pytest.mark.parametrize("seed,bias,S", [(0, 1.0, 3), (1, 0.0, 2), (2, 2.0, 5), (3, -1.0, 1), (4, 1.5, 10), (5, 0.7, 4)])
def test_wind_equals_sequential_for_every_window(seed, bias, S):
    w, enc, lens = small_case(seed, bias=bias, S=S, L=1 + seed % 2, act=seed % 2, blank_id=None if seed % 3 else 0)
    m = oracle.Model(w)
    T = enc.shape[1]
    tok0, frm0, n0, st0 = oracle.decode_batch(m, enc, lens, W=0, S=S)
    assert n0.sum() > 0 or bias > 1.9
    for W in (1, 2, 3, 4, 8, 16, T, T + 5):
        if W > 64:
            continue
        tok, frm, n, st = oracle.decode_batch(m, enc, lens, W=W, S=S)
        assert np.array_equal(n, n0), W
        assert np.array_equal(tok, tok0), W
        assert np.array_equal(frm, frm0), W
        # jumps lie in [0, W]; every frame is consumed exactly once by a jump or a forced advance
        hist = np.array(st["jump_hist"])
        assert hist[W + 1:].sum() == 0
        assert (hist * np.arange(65)).sum() + st["forced"] == lens.sum()
        assert hist.sum() == st["steps"]
        assert st["forced"] == st0["forced"]
        assert st["pred_updates"] == n.sum()
        if W > 1:
            assert st["steps"] <= st0["steps"]


def test_max_symbols_is_honoured():
    for seed, S in [(0, 1), (1, 2), (2, 3)]:
        w, enc, lens = small_case(10 + seed, bias=-3.0, S=S)  # blank strongly disfavoured
        m = oracle.Model(w)
        for W in (0, 1, 4):
            tok, frm, n, st = oracle.decode_batch(m, enc, lens, W=W, S=S)
            for b in range(len(lens)):
                f = frm[b, : n[b]]
                assert np.all(np.diff(f) >= 0)
                if n[b]:
                    assert np.bincount(f).max() <= S
                    assert f.max() < lens[b]
            # with blank this unlikely nearly every frame hits the cap
            assert st["forced"] > 0.5 * lens.sum()
            assert n.sum() >= S * st["forced"]


def test_huge_cap_equals_uncapped_when_loop_terminates():
    w, enc, lens = small_case(20, bias=1.2, S=3)
    m = oracle.Model(w)
    a = oracle.decode_batch(m, enc, lens, W=4, S=50)
    b = oracle.decode_batch(m, enc, lens, W=4, S=1000)
    if a[3]["forced"] == 0:
        assert np.array_equal(a[0][:, :50], b[0][:, :50]) and np.array_equal(a[2], b[2])


def test_all_blank_and_zero_length():
    w, enc, lens = small_case(30, bias=50.0)
    lens[1] = 0
    m = oracle.Model(w)
    for W in (0, 1, 4, 16):
        tok, frm, n, st = oracle.decode_batch(m, enc, lens, W=W, S=3)
        assert n.sum() == 0 and st["pred_updates"] == 0
        if W:
            assert st["steps"] == sum(-(-int(l) // W) for l in lens)


def test_batch_equals_single_and_padding_is_never_read():
    w, enc, lens = small_case(40, B=4, bias=0.8)
    m = oracle.Model(w)
    tok, frm, n, _ = oracle.decode_batch(m, enc, lens, W=4, S=3)
    for b in range(4):
        e1 = np.ascontiguousarray(enc[b : b + 1, : max(1, lens[b])])
        t1, f1, n1, _ = oracle.decode_batch(m, e1, lens[b : b + 1], W=4, S=3, max_out=tok.shape[1])
        assert n1[0] == n[b]
        assert np.array_equal(t1[0, : n1[0]], tok[b, : n[b]])
        assert np.array_equal(f1[0, : n1[0]], frm[b, : n[b]])


def test_output_overflow_reports_full_count():
    w, enc, lens = small_case(50, bias=-3.0, S=3)
    m = oracle.Model(w)
    full = oracle.decode_batch(m, enc, lens, W=4, S=3)
    cut = oracle.decode_batch(m, enc, lens, W=4, S=3, max_out=5)
    assert np.array_equal(full[2], cut[2])
    assert np.array_equal(full[0][:, :5], cut[0])


# ---------------------------------------------------------------------------
# replay check: accepts the oracle's own result, rejects a planted mistake
# ---------------------------------------------------------------------------
def test_replay_accepts_own_output_and_rejects_mistakes():
    w, enc, lens = small_case(60, B=2, bias=0.9, S=3)
    m = oracle.Model(w)
    tok, frm, n, st = oracle.decode_batch(m, enc, lens, W=4, S=3)
    b = 0
    T = int(lens[b])
    tk, fr = tok[b, : n[b]].copy(), frm[b, : n[b]].copy()
    assert n[b] >= 3
    ok = oracle.replay_verify(m, enc[b], T, 3, tk, fr, margin_thr=0.0)
    assert ok["rc"] == 0 and ok["not_argmax"] == 0
    seq = oracle.decode_batch(m, enc[b : b + 1], lens[b : b + 1], W=0, S=3)
    assert ok["decisions"] == seq[3]["decisions"]
    # drop a token: the frame is then implied blank, which the oracle does not agree with
    bad = oracle.replay_verify(m, enc[b], T, 3, np.delete(tk, 1), np.delete(fr, 1), margin_thr=0.0)
    assert bad["rc"] == 1
    # frames out of order
    fr2 = fr.copy()
    fr2[0], fr2[-1] = fr[-1], fr[0]
    if fr[0] != fr[-1]:
        assert oracle.replay_verify(m, enc[b], T, 3, tk, fr2)["rc"] == 2
    # blank as a token
    tk3 = tk.copy()
    tk3[0] = w["blank_id"]
    assert oracle.replay_verify(m, enc[b], T, 3, tk3, fr)["rc"] == 3
    # a wrong token is tolerated only inside the margin
    lg, *_ = oracle.eval_joint_window(m, enc[b], T, [], int(fr[0]), 1)
    order = np.argsort(-lg[0])
    second = int(order[1]) if int(order[1]) != w["blank_id"] else int(order[2])
    gap = lg[0][order[0]] - lg[0][second]
    tk4 = tk.copy()
    tk4[0] = second
    # with a margin below the gap the first decision fails; whatever follows is irrelevant
    assert oracle.replay_verify(m, enc[b], T, 3, tk4[:1], fr[:1], margin_thr=gap * 0.5)["rc"] in (1, 2)
    res = oracle.replay_verify(m, enc[b], T, 3, tk4[:1], fr[:1], margin_thr=gap * 0.5)
    assert res["rc"] == 1 and res["bad_pos"] == fr[0]


def test_low_margin_count_matches_direct_count():
    w, enc, lens = small_case(70, B=1, bias=0.9, S=3)
    m = oracle.Model(w)
    thr = 0.3
    _, _, _, st = oracle.decode_batch(m, enc, lens, W=0, S=3, margin_thr=thr)
    _, _, _, stw = oracle.decode_batch(m, enc, lens, W=4, S=3, margin_thr=thr)
    assert st["low_margin"] == stw["low_margin"] and st["decisions"] == stw["decisions"]
    assert 0 < st["low_margin"] < st["decisions"]


# ---------------------------------------------------------------------------
# Eq. (1): P'(v, t), "v is the first output in the window, at offset t"
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("seed,blank0,W,t0", [(0, False, 4, 0), (1, True, 3, 2), (2, False, 8, 5), (3, True, 1, 1), (4, False, 6, 7)])
def test_first_output_probabilities_match_direct_products(seed, blank0, W, t0):
    # independent evaluator: softmax of the naive model's logits, then the products of Eq. (1) written out
    r = rng(300 + seed)
    T, V = 9, 6
    w = random_weights(r, 5, 4, 6, 2, 7, V, blank_id=0 if blank0 else None, act=seed % 2, blank_bias=0.5, bias_scale=0.2)
    enc = r.standard_normal((T, 5)).astype(np.float32)
    prefix = [int(x) for x in r.integers(1 if blank0 else 0, V if blank0 else V - 1, size=3)]
    prefix = [p for p in prefix if p != w["blank_id"]]
    m = oracle.Model(w)
    logp = oracle.first_output_logprobs(m, enc, T, prefix, t0, W)
    n = min(W, T - t0)
    assert logp.shape == (n, V + 1)
    naive = NaiveModel(w)
    probs = []
    for t in range(n):
        z = naive.logits(enc[t0 + t], prefix)
        e = np.exp(z - z.max())
        probs.append(e / e.sum())
    blank = w["blank_id"]
    expect = np.zeros((n, V + 1))
    for t in range(n):
        before = np.prod([probs[k][blank] for k in range(t)]) if t else 1.0
        for v in range(V + 1):
            if v != blank:
                expect[t, v] = probs[t][v] * before
            else:
                expect[t, v] = before * probs[t][blank] if t == n - 1 else 0.0
    got = np.exp(logp)
    assert np.max(np.abs(got - expect)) < 1e-12
    assert np.all(np.isneginf(logp[: n - 1, blank]))
    # it is a distribution over "what comes first in the window, and where"
    assert abs(got.sum() - 1.0) < 1e-12
    # a window of one frame is the frame's own softmax
    one = np.exp(oracle.first_output_logprobs(m, enc, T, prefix, t0, 1))
    assert np.max(np.abs(one[0] - probs[0])) < 1e-12


def test_first_output_argmax_is_the_greedy_jump_when_blank_dominates_or_not():
    # With a very confident model (logits scaled up) the most probable first output is what Algorithm 2 emits: the
    # first non-blank argmax row and its label, or blank at the last row when every row's argmax is blank.
    r = rng(400)
    T, V, W = 12, 5, 4
    w = random_weights(r, 4, 3, 5, 1, 6, V, blank_bias=0.3)
    w["w_out"] = (w["w_out"] * 40).astype(np.float32)
    w["b_out"] = (w["b_out"] * 40).astype(np.float32)
    enc = r.standard_normal((T, 4)).astype(np.float32)
    m = oracle.Model(w)
    checked = 0
    for t0 in range(T):
        logits, *_ = oracle.eval_joint_window(m, enc, T, [], t0, W)
        labels = logits.argmax(axis=1)
        logp = oracle.first_output_logprobs(m, enc, T, [], t0, W)
        t_best, v_best = np.unravel_index(np.argmax(logp), logp.shape)
        nonblank = [i for i, l in enumerate(labels) if l != w["blank_id"]]
        top2 = np.sort(logits, axis=1)[:, -2:]
        if np.min(top2[:, 1] - top2[:, 0]) < 0.5:
            continue    # not confident enough for the argument to hold
        checked += 1
        if nonblank:
            assert (t_best, v_best) == (nonblank[0], labels[nonblank[0]])
        else:
            assert (t_best, v_best) == (len(labels) - 1, w["blank_id"])
    assert checked >= 4


# ---------------------------------------------------------------------------
# window-based greedy decoding (the best (label, offset) pair of Eq. (1) at every step)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("seed,bias,S", [(0, 1.0, 3), (1, 0.0, 2), (2, -1.0, 1), (3, 1.5, 10)])
def test_window_greedy_with_a_one_frame_window_is_algorithm_1(seed, bias, S):
    # one row: log P'(v, 0) = log softmax, whose argmax is the logits' argmax
    w, enc, lens = small_case(80 + seed, bias=bias, S=S)
    m = oracle.Model(w)
    ref = oracle.decode_batch(m, enc, lens, W=0, S=S)
    got = oracle.decode_window_greedy_batch(m, enc, lens, W=1, S=S)
    assert np.array_equal(ref[2], got[2]) and np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])
    assert got[3]["forced"] == ref[3]["forced"]


def brute_force_window_greedy(nm, enc, W, S):
    """The variant's rules on independently evaluated logits: the whole table log P'(v, j) is built with library
    routines (log_softmax, cumsum) and its first maximum in (row, label) order is taken, the all-blank entry last."""
    T = enc.shape[0]
    hyp, frames, t, count = [], [], 0, 0
    while t < T:
        n = min(W, T - t)
        lg = np.stack([nm.logits(enc[t + j], hyp) for j in range(n)])
        lp = torch.log_softmax(torch.tensor(lg), dim=1).numpy()
        before = np.concatenate([[0.0], np.cumsum(lp[:, nm.blank])])   # blanks on rows < j
        table = lp + before[:n, None]
        table[:, nm.blank] = -np.inf
        flat = int(np.argmax(table))                                   # first maximum, rows ascending then labels
        j, v = divmod(flat, lp.shape[1])
        if before[n] > table[j, v]:                                    # the all-blank candidate wins only strictly
            t += n
            count = 0
            continue
        if j > 0:
            count = 0
        t += j
        hyp.append(v)
        frames.append(t)
        count += 1
        if count == S:
            t += 1
            count = 0
    return hyp, frames


@pytest.mark.parametrize("seed,W,S,bias,blank0,act", [(0, 2, 3, 0.5, False, 0), (1, 4, 2, 1.0, True, 1), (2, 8, 3, 0.0, False, 0),
                                                     (3, 3, 1, -0.5, False, 1), (4, 5, 4, 2.0, True, 0)])
def test_window_greedy_matches_brute_force(seed, W, S, bias, blank0, act):
    r = rng(900 + seed)
    V = 9
    w = random_weights(r, 6, 5, 6, 1 + seed % 2, 8, V, blank_id=0 if blank0 else None, act=act, blank_bias=bias, bias_scale=0.1)
    T = 26
    enc = r.standard_normal((1, T, 6)).astype(np.float32)
    m = oracle.Model(w)
    tok, frm, n, st = oracle.decode_window_greedy_batch(m, enc, np.array([T], np.int32), W=W, S=S)
    hyp, frames = brute_force_window_greedy(NaiveModel(w), enc[0], W, S)
    assert list(tok[0, : n[0]]) == hyp and list(frm[0, : n[0]]) == frames
    hist = np.array(st["jump_hist"])
    assert (hist * np.arange(65)).sum() + st["forced"] == T and hist[W + 1:].sum() == 0
    assert st["pred_updates"] == n[0] and st["steps"] == st["decisions"] == hist.sum()


def table_model(probs):
    """A joiner whose output does not depend on the decoder: frame type k (a one-hot encoder frame) has the label
    distribution probs[k] (labels 0..V-1, blank last)."""
    probs = np.asarray(probs, np.float64)
    K, NV = probs.shape
    V = NV - 1
    z = lambda *s: np.zeros(s, np.float32)
    return dict(D=K, E=2, P=2, L=1, H=K, V=V, blank_id=V, act=0, dtype="f32", emb=z(NV, 2),
                w_ih=[z(8, 2)], w_hh=[z(8, 2)], b_ih=[z(8)], b_hh=[z(8)],
                w_enc=np.eye(K, dtype=np.float32), b_enc=z(K), w_pred=z(K, 2), b_pred=z(K),
                w_out=np.log(probs).T.astype(np.float32), b_out=z(NV))


def test_window_greedy_worked_example_differs_from_algorithm_2():
    # frame types: A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1), C = (x .02, y .03, blank .95)
    # utterance A B C C, W = 2, S = 1 (every emission is followed by a forced advance):
    #   window [A, B]: P'(x,0) = .45, P'(y,0) = .05, P'(x,1) = .5 * .1, P'(y,1) = .5 * .8 = .4, all blank = .05  -> x at frame 0
    #   window [B, C]: P'(y,0) = .8 is the largest                                                               -> y at frame 1
    #   window [C, C]: all blank = .9025                                                                         -> end
    # Algorithms 1 and 2 take the per-frame argmax: A -> blank (.5 > .45), B -> y, C -> blank: only y at frame 1.
    w = table_model([[.45, .05, .5], [.1, .8, .1], [.02, .03, .95]])
    enc = np.eye(3, dtype=np.float32)[[0, 1, 2, 2]][None]
    lens = np.array([4], np.int32)
    m = oracle.Model(w)
    tok, frm, n, st = oracle.decode_window_greedy_batch(m, enc, lens, W=2, S=1)
    assert list(tok[0, : n[0]]) == [0, 1] and list(frm[0, : n[0]]) == [0, 1]
    assert st["steps"] == 3 and st["forced"] == 2 and st["jump_hist"][0] == 2 and st["jump_hist"][2] == 1
    for W in (1, 2, 4):
        tok2, frm2, n2, _ = oracle.decode_batch(m, enc, lens, W=W, S=1)
        assert list(tok2[0, : n2[0]]) == [1] and list(frm2[0, : n2[0]]) == [1]
    tok1, frm1, n1, _ = oracle.decode_window_greedy_batch(m, enc, lens, W=1, S=1)
    assert list(tok1[0, : n1[0]]) == [1] and list(frm1[0, : n1[0]]) == [1]
    # W = 3: window [A, B, C]: .45 for x at 0 still beats .4; then [B, C, C]: y at 1; then [C, C]
    tok3, frm3, n3, _ = oracle.decode_window_greedy_batch(m, enc, lens, W=3, S=1)
    assert list(tok3[0, : n3[0]]) == [0, 1] and list(frm3[0, : n3[0]]) == [0, 1]
    # a later pair can win over an earlier one: A' = (x .3, y .1, blank .6): P'(y,1) = .6 * .8 = .48 > .3 -> jump to frame 1
    w2 = table_model([[.3, .1, .6], [.1, .8, .1], [.02, .03, .95]])
    tok4, frm4, n4, st4 = oracle.decode_window_greedy_batch(oracle.Model(w2), enc, lens, W=2, S=1)
    assert list(tok4[0, : n4[0]]) == [1] and list(frm4[0, : n4[0]]) == [1] and st4["jump_hist"][1] == 1


def test_window_replay_accepts_own_output_and_rejects_mistakes():
    w, enc, lens = small_case(61, B=2, bias=0.9, S=3)
    m = oracle.Model(w)
    W = 4
    tok, frm, n, st = oracle.decode_window_greedy_batch(m, enc, lens, W=W, S=3)
    b, T = 0, int(lens[0])
    tk, fr = tok[b, : n[b]].copy(), frm[b, : n[b]].copy()
    assert n[b] >= 3
    ok = oracle.replay_verify_window(m, enc[b], T, W, 3, tk, fr, margin_thr=0.0)
    assert ok["rc"] == 0 and ok["not_argmax"] == 0
    one = oracle.decode_window_greedy_batch(m, enc[b : b + 1], lens[b : b + 1], W=W, S=3)
    assert ok["decisions"] == one[3]["decisions"]
    # the same sequence is in general not what another window size produces
    assert oracle.replay_verify_window(m, enc[b], T, W, 3, np.delete(tk, 1), np.delete(fr, 1), margin_thr=0.0)["rc"] == 1
    fr2 = fr.copy()
    fr2[0], fr2[-1] = fr[-1], fr[0]
    if fr[0] != fr[-1]:
        assert oracle.replay_verify_window(m, enc[b], T, W, 3, tk, fr2)["rc"] == 2
    tk3 = tk.copy()
    tk3[0] = w["blank_id"]
    assert oracle.replay_verify_window(m, enc[b], T, W, 3, tk3, fr)["rc"] == 3
    # a different label at the first decision passes only with a margin above its gap in log P'
    lp = oracle.first_output_logprobs(m, enc[b], T, [], 0, W)
    j = int(fr[0])
    assert j < W
    other = next(v for v in np.argsort(-lp[j]) if v != tk[0] and v != w["blank_id"])
    gap = lp.max() - lp[j, other]
    tk4 = tk.copy()
    tk4[0] = other
    res = oracle.replay_verify_window(m, enc[b], T, W, 3, tk4[:1], fr[:1], margin_thr=gap * 0.5)
    assert res["rc"] == 1 and res["bad_pos"] == 0 and res["decisions"] == 1
    # with a margin above the gap the first decision passes (whatever happens at the second one)
    res = oracle.replay_verify_window(m, enc[b], T, W, 3, tk4[:1], fr[:1], margin_thr=gap * 1.01)
    assert res["decisions"] >= 2 and res["not_argmax"] >= 1


# ---------------------------------------------------------------------------
# argmax tie rule: lowest index wins (the paper is silent; the reading is fixed here by exact ties)
# ---------------------------------------------------------------------------
TIE_UTTS = [[5, 0, 5, 5, 1, 2, 3, 4, 5, 6, 7, 8, 5], [8, 7, 6, 5, 5, 5, 5, 5, 5, 5, 4, 3, 2, 1, 0], [3], [5, 5, 4],
            [2, 2, 3, 3, 4, 4, 8, 8], []]


@pytest.mark.parametrize("blank_first", [False, True])
@pytest.mark.parametrize("S", [1, 2])
def test_argmax_ties_go_to_the_lowest_index(blank_first, S):
    # Exact ties by construction (dyadic logits, ties only after the bias is added).  Expected winners are written
    # down from the rule, not computed by the oracle: two labels -> the lower label; a label and the blank -> the
    # label when the blank is the last index, the blank when it is index 0; everything equal -> index 0.
    w, target, winners = tie_model(blank_id=0 if blank_first else None)
    blank = w["blank_id"]
    if blank_first:
        assert winners == [3, 3, 70, 0, 0, 0, 298, 10, 0]
    else:
        assert winners == [3, 3, 70, 200, 5, 299, 298, 10, 0]
    enc, lens = tie_utterances(w["D"], TIE_UTTS)
    m = oracle.Model(w)
    # the logits really are the hand-set targets, ties included
    lg, *_ = oracle.eval_joint_window(m, enc[0], int(lens[0]), [], 0, 13)
    for j, k in enumerate(TIE_UTTS[0]):
        assert np.array_equal(lg[j], target[:, k])
    for W in (0, 1, 2, 4, 8, 16):     # 0: Algorithm 1 as written; the others Algorithm 2
        tok, frm, n, st = oracle.decode_batch(m, enc, lens, W=W, S=S)
        for b, types in enumerate(TIE_UTTS):
            want_tok, want_frm = tie_expected(types, winners, blank, S)
            assert list(tok[b, : n[b]]) == want_tok and list(frm[b, : n[b]]) == want_frm, (W, b)
    # the opposite rule (highest index on ties) would give something else on these inputs
    other = [int(np.flatnonzero(target[:, k] == target[:, k].max())[-1]) for k in range(len(winners))]
    assert tie_expected(TIE_UTTS[0], other, blank, S) != tie_expected(TIE_UTTS[0], winners, blank, S)


# ---------------------------------------------------------------------------
# Algorithm 3: WIND beam search
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("seed,W,S,bias", [(0, 4, 3, 1.0), (1, 1, 2, 0.5), (2, 8, 1, 1.5), (3, 3, 10, 2.0)])
def test_beam_search_with_beam_one_is_window_based_greedy(seed, W, S, bias):
    w, enc, lens = small_case(90 + seed, B=1, T=30, bias=bias, S=S)
    m = oracle.Model(w)
    T = int(lens[0])
    hyps, gap, steps = oracle.beam_search(m, enc[0], T, W, 1, S)
    tok, frm, n, st = oracle.decode_window_greedy_batch(m, enc, lens, W=W, S=S)
    assert len(hyps) == 1 and steps == st["steps"]
    assert list(hyps[0][0]) == list(tok[0, : n[0]]) and list(hyps[0][1]) == list(frm[0, : n[0]])


def brute_force_sequence_probabilities(nm, enc, S):
    """Total probability of every token sequence: all alignments walked frame by frame on independently evaluated
    logits (blank advances; a label stays on the frame, the S-th label in a row on a frame advances without a blank)."""
    T = enc.shape[0]
    cache, total = {}, {}

    def logp(t, hyp):
        key = (t, tuple(hyp))
        if key not in cache:
            cache[key] = torch.log_softmax(torch.tensor(nm.logits(enc[t], hyp)), dim=0).numpy()
        return cache[key]

    def walk(t, hyp, count, acc):
        if t == T:
            total[tuple(hyp)] = np.logaddexp(total.get(tuple(hyp), -np.inf), acc)
            return
        lp = logp(t, hyp)
        walk(t + 1, hyp, 0, acc + lp[nm.blank])
        for v in range(len(lp)):
            if v != nm.blank:
                if count + 1 == S:
                    walk(t + 1, hyp + [v], 0, acc + lp[v])
                else:
                    walk(t, hyp + [v], count + 1, acc + lp[v])

    walk(0, [], 0, 0.0)
    return total


@pytest.mark.parametrize("seed,blank0", [(0, False), (1, True)])
def test_beam_search_without_pruning_sums_all_alignments_for_every_window(seed, blank0):
    # a beam wider than the number of hypotheses never prunes: the final score of a token sequence is then the log of
    # its total probability over all alignments, whatever the window
    r = rng(950 + seed)
    V, T, S = 2, 3, 2
    w = random_weights(r, 4, 3, 4, 1, 5, V, blank_id=0 if blank0 else None, act=seed % 2, blank_bias=0.3, bias_scale=0.1)
    enc = r.standard_normal((T, 4)).astype(np.float32)
    want = brute_force_sequence_probabilities(NaiveModel(w), enc, S)
    assert abs(np.logaddexp.reduce(list(want.values()))) < 1e-9            # the sequences' probabilities sum to one
    m = oracle.Model(w)
    for W in (1, 2, 3, 5):
        hyps, gap, steps = oracle.beam_search(m, enc, T, W, 4096, S, max_hyps=4096)
        got = {tuple(int(x) for x in h[0]): h[2] for h in hyps}
        assert set(got) == set(want)
        for k in want:
            assert abs(got[k] - want[k]) < 1e-7, (W, k)
        scores = [h[2] for h in hyps]
        assert scores == sorted(scores, reverse=True)


def test_beam_search_worked_example_beats_greedy():
    # frame types A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1); utterance A B, W = 2, S = 1, K = 2:
    #   t = 0, []: P'(x,0) = .45, P'(y,1) = .5 * .8 = .4 are the two best -> [x] (frame 0, then forced to t = 1) and
    #              [y] (frame 1, forced to t = 2)
    #   t = 1, [x]: window [B]: P'(y,0) = .8, then x and blank tie at .1 (the label comes first) -> [x,y] .36, [x,x] .045
    #   t = 2 = T: [y] .4 > [x,y] .36 > [x,x] .045.   With K = 1 (window-based greedy): [x] then [x,y], .36.
    w = table_model([[.45, .05, .5], [.1, .8, .1]])
    enc = np.eye(2, dtype=np.float32)[[0, 1]]
    m = oracle.Model(w)
    hyps, gap, steps = oracle.beam_search(m, enc, 2, 2, 2, 1)
    assert [list(h[0]) for h in hyps] == [[1], [0, 1], [0, 0]]
    assert [list(h[1]) for h in hyps] == [[1], [0, 1], [0, 1]]
    assert np.allclose([h[2] for h in hyps], np.log([.4, .36, .045]), atol=1e-6) and steps == 2
    one, _, _ = oracle.beam_search(m, enc, 2, 2, 1, 1)
    assert list(one[0][0]) == [0, 1] and abs(one[0][2] - np.log(.36)) < 1e-6
    assert abs(gap - 0.0) < 1e-6      # the x / blank tie is reported as a zero gap


def test_beam_prefix_step_matches_an_independent_evaluation():
    # completing A into B at one frame: P(A) * prod_i P(b_i | frame, decoder after A + b_<i), from the independent
    # evaluator (whole-prefix LSTM re-run, library log-softmax); every proper prefix is removed
    r = rng(970)
    w = random_weights(r, 5, 4, 6, 2, 7, 6, act=1, blank_bias=0.5, bias_scale=0.1)
    nm = NaiveModel(w)
    enc_t = r.standard_normal(5).astype(np.float32)
    hyps = [[1, 2], [1, 2, 3, 0], [1], [4, 4], [1, 2, 5], []]
    scores = [-1.0, -3.5, -0.7, -2.0, -2.5, -4.0]

    def completion(a, b):
        acc = scores[a]
        for i in range(len(hyps[a]), len(hyps[b])):
            lp = torch.log_softmax(torch.tensor(nm.logits(enc_t, hyps[b][:i])), dim=0).numpy()
            acc += lp[hyps[b][i]]
        return acc

    want = list(scores)
    removed = [False] * len(hyps)
    for a in range(len(hyps)):
        for b in range(len(hyps)):
            if a != b and len(hyps[a]) < len(hyps[b]) and hyps[b][: len(hyps[a])] == hyps[a]:
                want[b] = np.logaddexp(want[b], completion(a, b))
                removed[a] = True
    got, gone = oracle.beam_prefix_step(oracle.Model(w), enc_t, hyps, scores)
    assert list(gone) == removed == [True, False, True, False, False, True]
    for b in range(len(hyps)):
        if not removed[b]:
            assert abs(got[b] - want[b]) < 1e-9


def test_beam_search_with_prefix_step_worked_example():
    # frame types A = (x .45, y .05, blank .5), B = (x .1, y .8, blank .1); utterance A B, W = 1, S = 2, K = 2.
    # t = 0, []: x .45 -> [x] stays on frame 0; blank .5 -> [] goes to frame 1.
    # t = 0 again, [x]: x .45 -> [x,x] .2025, second emission on the frame: forced to frame 1; blank .5 -> [x] .225 to frame 1.
    # t = 1, {[] .5, [x,x] .2025, [x] .225}: [] is a prefix of both others, [x] of [x,x].  Completions at frame 1 (type B):
    #     [] -> [x]: .5 * .1 = .05      [] -> [x,x]: .5 * .1 * .1 = .005      [x] -> [x,x]: .225 * .1 = .0225
    #   [x,x] = .2025 + .005 + .0225 = .23; [] and [x] are removed (each is a prefix of something): one hypothesis is left.
    #   [x,x]: y .8 -> [x,x,y] .184 stays; x .1 (label before blank on the tie) -> [x,x,x] .023 stays.
    # t = 1 again: no prefix pair; every second emission is forced to T:
    #   [x,x,y,y] .1472, [x,x,y,x] .0184, [x,x,x,y] .0184, [x,x,x,x] .0023.
    w = table_model([[.45, .05, .5], [.1, .8, .1]])
    enc = np.eye(2, dtype=np.float32)[[0, 1]]
    m = oracle.Model(w)
    pre, _, steps = oracle.beam_search(m, enc, 2, 1, 2, 2, prefix_search=True)
    assert steps == 4
    assert [list(h[0]) for h in pre] == [[0, 0, 1, 1], [0, 0, 1, 0], [0, 0, 0, 1], [0, 0, 0, 0]]
    assert [list(h[1]) for h in pre] == [[0, 0, 1, 1]] * 4
    assert np.allclose(np.exp([h[2] for h in pre]), [.1472, .0184, .0184, .0023], atol=1e-6)
    # without the step the beam at t = 1 is {[] .5, [x] .225}: a different search
    plain, _, _ = oracle.beam_search(m, enc, 2, 1, 2, 2)
    assert abs(np.exp(plain[0][2]) - .1472) > 1e-3
