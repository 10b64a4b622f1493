"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Comparison rule for (token, frame) sequences: bit-exact against the oracle's
sequential result (Algorithm 1), except at decisions whose oracle top-2 logit
margin is below 0.05; there the GPU's choice must still lie within 0.05 of the
oracle's maximum (checked by replaying the GPU's sequence through the oracle),
and the number of such decisions is reported.  Joint logits: 1e-4 abs on the
fp32 path, 2e-2 abs on the bf16-weight path.
"""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import oracle
import wind_synth as ws
from conftest import LOOP_MODES, set_loop_mode
from naive_model import random_weights, tie_expected, tie_model, tie_utterances

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MARGIN = 0.05
TOL = {"f32": 1e-4, "bf16": 2e-2}


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_13765_b200 as p
    p.load_library()
    return p


def check_against_oracle(pkg, weights, enc, lens, W, S, kernels=0, expect_exact=None, sample=None, round_bf16=False,
                         margin=MARGIN):
    """Decode on the GPU, compare with the oracle.  Returns a report dict.  round_bf16: the oracle that rounds enc_proj,
    the hidden state and the joint's activations to bf16 where the bf16 kernels do (a smaller margin can then be asked)."""
    prev = pkg.wind_set_kernels(kernels)
    try:
        model = pkg.WindModel(weights)
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, S)
    finally:
        pkg.wind_set_kernels(prev)
    assert st == 0
    om = oracle.Model(weights, round_bf16=round_bf16)
    B = enc.shape[0]
    idx = list(range(B)) if sample is None else list(sample)
    sub = np.ascontiguousarray(enc[idx])
    otok, ofrm, on, ost = oracle.decode_batch(om, sub, lens[idx], W=0, S=S, max_out=tok.shape[1], margin_thr=margin)

    def replay(k):
        b = idx[k]
        return oracle.replay_verify(om, enc[b], int(lens[b]), S, tok[b, : olen[b]], frm[b, : olen[b]], margin)

    with ThreadPoolExecutor(8) as ex:
        reps = list(ex.map(replay, range(len(idx))))
    exact = 0
    off_argmax = 0
    for k, b in enumerate(idx):
        r = reps[k]
        assert r["rc"] == 0, f"utterance {b}: replay failed {r}"
        off_argmax += r["not_argmax"]
        same = on[k] == olen[b] and np.array_equal(otok[k, : on[k]], tok[b, : olen[b]]) and \
            np.array_equal(ofrm[k, : on[k]], frm[b, : olen[b]])
        exact += bool(same)
        if r["not_argmax"] == 0:
            assert same, f"utterance {b}: every decision is the oracle argmax yet the sequences differ"
        f = frm[b, : olen[b]]
        assert np.all(np.diff(f) >= 0)
        if len(f):
            assert f.max() < lens[b] and np.bincount(f).max() <= S
        assert np.all(tok[b, olen[b]:] == -1)  # untouched beyond out_len
    rep = dict(exact=exact, n=len(idx), off_argmax=off_argmax, low_margin_oracle=ost["low_margin"],
               decisions=ost["decisions"], stats=stats)
    if expect_exact:
        assert exact == len(idx), rep
    if sample is None:
        assert stats["frames"] == int(lens.sum())
        assert stats["tokens"] == int(olen.sum())
        hist = np.array(stats["jump_hist"])
        assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum())
        assert hist[W + 1:].sum() == 0
    print(f"[parity] W={W} S={S} exact {exact}/{len(idx)} utterances, {off_argmax} decisions off the oracle argmax "
          f"(all inside {margin}); oracle low-margin decisions {ost['low_margin']}/{ost['decisions']}")
    return rep, (tok, frm, olen)


def ragged_case(seed, B, T, D, E, P, L, H, V, act=0, blank_id=None, bias=1.0, dtype="f32"):
    r = np.random.default_rng(1000 + seed)
    w = random_weights(r, D, E, P, L, H, V, blank_id=blank_id, act=act, blank_bias=bias, bias_scale=0.1)
    w["dtype"] = dtype
    if dtype == "bf16":
        for k in ("emb", "w_enc", "w_pred", "w_out"):
            w[k] = ws.bf16_round(w[k])
        w["w_ih"] = [ws.bf16_round(a) for a in w["w_ih"]]
        w["w_hh"] = [ws.bf16_round(a) for a in w["w_hh"]]
    lens = r.integers(0, T + 1, size=B).astype(np.int32)
    lens[0] = T
    if B > 2:
        lens[1] = 0
        lens[2] = 1
    enc = r.standard_normal((B, T, D)).astype(np.float32)
    if dtype == "bf16":
        enc = ws.bf16_round(enc)
    for b in range(B):
        enc[b, lens[b]:] = np.nan
    return w, enc, lens


# ---------------------------------------------------------------------------
# fp32 path
# ---------------------------------------------------------------------------
def test_cfg1_tiny_fp32(pkg):
    cfg = ws.CONFIGS["cfg1_tiny"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    rep, out4 = check_against_oracle(pkg, weights, enc, lens, cfg.W, cfg.S)
    rep1, out1 = check_against_oracle(pkg, weights, enc, lens, 1, cfg.S)
    if rep["off_argmax"] == 0 and rep1["off_argmax"] == 0:
        for a, b in zip(out4, out1):
            assert np.array_equal(a, b)
    rate = None
    om = oracle.Model(weights)
    _, _, _, st = oracle.decode_batch(om, enc, lens, W=0, S=cfg.S)
    rate = st["emit_frames"] / lens.sum()
    print(f"[cfg1] oracle non-blank frame rate on the workload sample: {rate:.3f}")


@pytest.mark.parametrize("seed,W,S,act,blank0,L,bias", [
    (0, 1, 3, 0, False, 1, 1.0), (1, 2, 2, 1, True, 2, 0.5), (2, 3, 1, 0, False, 1, 0.0), (3, 4, 5, 1, False, 3, 1.5),
    (4, 8, 10, 0, True, 2, 1.0), (5, 16, 4, 0, False, 1, 2.0), (6, 64, 3, 1, False, 1, 1.0), (7, 5, 2, 0, False, 1, -3.0),
])
def test_fp32_ragged_shapes(pkg, seed, W, S, act, blank0, L, bias):
    # odd sizes on purpose: nothing is a multiple of a tile
    w, enc, lens = ragged_case(seed, B=7, T=53, D=37, E=29, P=41, L=L, H=67, V=45, act=act,
                               blank_id=0 if blank0 else None, bias=bias)
    check_against_oracle(pkg, w, enc, lens, W, S)


def test_fp32_window_invariance_on_gpu(pkg):
    w, enc, lens = ragged_case(20, B=5, T=80, D=32, E=32, P=32, L=1, H=64, V=30, bias=1.0)
    outs = []
    for W in (1, 2, 4, 8, 16, 64):
        rep, out = check_against_oracle(pkg, w, enc, lens, W, 4)
        outs.append((rep, out))
    if all(r["off_argmax"] == 0 for r, _ in outs):
        for _, o in outs[1:]:
            for a, b in zip(o, outs[0][1]):
                assert np.array_equal(a, b)


def test_fp32_joint_logits(pkg):
    w, enc, lens = ragged_case(30, B=6, T=40, D=48, E=24, P=40, L=2, H=72, V=50, act=1, bias=0.7)
    logits_parity(pkg, w, enc, lens, W=4, S=3, tol=TOL["f32"], n_windows=24)


def logits_parity(pkg, weights, enc, lens, W, S, tol, n_windows, kernels=0, seed=0, round_bf16=False):
    """Teacher-forced logits at oracle-chosen prefixes and frames.  round_bf16: against the oracle that rounds enc_proj, the
    hidden state and the joint's activations to bf16 where the bf16 kernels do."""
    om = oracle.Model(weights, round_bf16=round_bf16)
    B, T, _ = enc.shape
    otok, ofrm, on, _ = oracle.decode_batch(om, enc, lens, W=0, S=S)
    r = np.random.default_rng(seed)
    prev = pkg.wind_set_kernels(kernels)
    model = pkg.WindModel(weights)
    worst = 0.0
    rows = 0
    try:
        for rep in range(max(1, n_windows // B)):
            t0 = np.array([r.integers(0, max(1, lens[b])) if lens[b] else 0 for b in range(B)], np.int32)
            if rep == 0:
                t0[0] = max(0, lens[0] - 1)  # a window truncated by the end of the utterance
            plen = np.array([int(np.searchsorted(ofrm[b, : on[b]], t0[b], side="left")) for b in range(B)], np.int32)
            U = max(1, int(plen.max()))
            prefix = np.zeros((B, U), np.int32)
            for b in range(B):
                prefix[b, : plen[b]] = otok[b, : plen[b]]
            d = model.device
            enc_d = pkg.to_device_enc(model, enc)
            logits = torch.full((B, W, model.dims["V"] + 1), float("nan"), dtype=torch.float32, device=d)
            wsb = pkg.alloc_workspace(model, B, T, W)
            pkg.wind_eval_joint_window(model, enc_d, torch.from_numpy(lens).to(d), W, torch.from_numpy(prefix).to(d),
                                       torch.from_numpy(plen).to(d), torch.from_numpy(t0).to(d), logits, wsb)
            got = logits.cpu().numpy()
            for b in range(B):
                ref, *_ = oracle.eval_joint_window(om, enc[b], int(lens[b]), prefix[b, : plen[b]], int(t0[b]), W)
                n = ref.shape[0]
                assert n == max(0, min(W, lens[b] - t0[b]))
                if n:
                    err = np.max(np.abs(got[b, :n].astype(np.float64) - ref))
                    worst = max(worst, float(err))
                    rows += n
                assert np.all(np.isnan(got[b, n:]))  # rows past the window are left untouched
    finally:
        pkg.wind_set_kernels(prev)
    print(f"[logits] {rows} rows, worst abs error {worst:.3e} (tolerance {tol})")
    assert rows > 0 and worst < tol
    return worst


# ---------------------------------------------------------------------------
# bf16-weight path
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("kernels", [1, 0])
def test_bf16_ragged_small(pkg, kernels):
    # odd sizes: always the plain-ALU kernels
    w, enc, lens = ragged_case(40, B=6, T=45, D=40, E=24, P=40, L=2, H=56, V=35, bias=1.0, dtype="bf16")
    check_against_oracle(pkg, w, enc, lens, 4, 3, kernels=kernels)
    logits_parity(pkg, w, enc, lens, W=4, S=3, tol=TOL["bf16"], n_windows=12, kernels=kernels)


@pytest.mark.parametrize("L,act,W", [(2, 0, 4), (1, 1, 8), (3, 0, 1)])
def test_bf16_plain_alu_path_against_the_oracle_in_the_same_precision(pkg, L, act, W):
    # The plain-ALU bf16 kernels round enc_proj, the hidden state and the joint's activations to bf16 and nothing else; the
    # oracle can do the same (Model(round_bf16=True): fp64 sums, the same three roundings).  What is left between the two
    # is fp32 accumulation: logits agree to about 1e-6 unless an fp32 sum falls on the other side of a bf16 rounding
    # boundary than the fp64 sum (one last-place step of one value: about 1e-3 in a logit), against 2e-2 for the fp64
    # oracle.  Transcripts: the margin rule with a margin ten times smaller.
    w, enc, lens = ragged_case(60 + L, B=6, T=45, D=40, E=24, P=40, L=L, H=56, V=35, act=act, bias=1.0, dtype="bf16")
    rep, _ = check_against_oracle(pkg, w, enc, lens, W, 3, kernels=1, round_bf16=True, margin=5e-3)
    assert rep["stats"]["kernels"] == 1 and rep["exact"] >= 5
    worst = logits_parity(pkg, w, enc, lens, W=W, S=3, tol=2e-3, n_windows=24, kernels=1, round_bf16=True)
    print(f"[same precision] L={L} act={act}: worst logit difference {worst:.2e}, {rep['exact']}/6 transcripts equal")


@pytest.mark.parametrize("L", [1, 2, 3])
def test_bf16_streaming_tensor_path_against_the_oracle_in_the_same_precision(pkg, L):
    # The tensor-core loop in its streaming mode rounds in the same three places as the plain-ALU kernels and uses tanhf /
    # expf in the gates, so with a ReLU joint it too is the rounding oracle up to fp32 accumulation (the kernels with
    # resident weights also round pred_proj and use the hardware tanh: they keep the fp64 oracle and its 2e-2).
    set_loop_mode(pkg, "streaming")
    w, enc, lens = ragged_case(80 + L, B=9, T=14, D=64, E=64, P=64, L=L, H=64, V=140, act=0, bias=1.0, dtype="bf16")
    rep, _ = check_against_oracle(pkg, w, enc, lens, 4, 3, kernels=2, round_bf16=True, margin=5e-3)
    assert rep["stats"]["kernels"] == 2 and rep["exact"] >= 8
    worst = logits_parity(pkg, w, enc, lens, W=4, S=3, tol=2e-3, n_windows=36, kernels=2, round_bf16=True)
    print(f"[same precision, streaming] L={L}: worst logit difference {worst:.2e}, {rep['exact']}/9 transcripts equal")


@pytest.mark.parametrize("kernels", [1, 0])
@pytest.mark.parametrize("name,B,lo,hi,W", [
    ("cfg3_large_b128", 5, 1, 150, 8), ("cfg3_large_b128", 3, 100, 300, 1), ("cfg4_xl_r25", 4, 20, 140, 16),
    ("cfg4_xl_r50", 4, 20, 140, 4), ("cfg5_bigvocab", 3, 10, 60, 16),
])
def test_bf16_model_shapes_small_batches(pkg, kernels, name, B, lo, hi, W):
    cfg = ws.small_variant(ws.CONFIGS[name], B, lo, hi)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    rep, _ = check_against_oracle(pkg, weights, enc, lens, W, cfg.S, kernels=kernels)
    assert rep["stats"]["kernels"] == (1 if kernels == 1 else rep["stats"]["kernels"])


@pytest.mark.parametrize("kernels", [1, 0])
@pytest.mark.parametrize("name,W", [("cfg3_large_b128", 8), ("cfg5_bigvocab", 16)])
def test_bf16_joint_logits(pkg, kernels, name, W):
    cfg = ws.small_variant(ws.CONFIGS[name], 8, 30, 90)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    logits_parity(pkg, weights, enc, lens, W=W, S=cfg.S, tol=TOL["bf16"], n_windows=64 if name.startswith("cfg3") else 16,
                  kernels=kernels)


def test_bf16_joint_logits_after_a_long_prefix(pkg):
    # The tensor path rounds the hidden state to bf16 at every update and feeds it back; this checks that the
    # recurrence has not drifted after several hundred updates: windows of the 100 s utterance (large model)
    # evaluated behind oracle prefixes of 500 to 3000 tokens, same tolerance as everywhere else.
    cfg = ws.CONFIGS["cfg2_large_b1"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    om = oracle.Model(weights)
    otok, ofrm, on, _ = oracle.decode_batch(om, enc, lens, W=0, S=cfg.S)
    assert on[0] > 3000
    T = int(lens[0])
    W = 8
    prev = pkg.wind_set_kernels(2)
    try:
        model = pkg.WindModel(weights)
        d = model.device
        enc_d = pkg.to_device_enc(model, enc)
        wsb = pkg.alloc_workspace(model, 1, T, W)
        worst = 0.0
        for want in (500, 1200, 3000):
            t0 = int(ofrm[0, want])                         # a frame reached after about `want` tokens
            plen = int(np.searchsorted(ofrm[0, : on[0]], t0, side="left"))
            assert plen >= want - 10 * cfg.S
            prefix = np.ascontiguousarray(otok[:, :plen])
            logits = torch.full((1, W, cfg.V + 1), float("nan"), dtype=torch.float32, device=d)
            pkg.wind_eval_joint_window(model, enc_d, torch.from_numpy(lens).to(d), W, torch.from_numpy(prefix).to(d),
                                       torch.tensor([plen], dtype=torch.int32, device=d),
                                       torch.tensor([t0], dtype=torch.int32, device=d), logits, wsb)
            ref, *_ = oracle.eval_joint_window(om, enc[0], T, prefix[0], t0, W)
            n = ref.shape[0]
            assert n == min(W, T - t0) and n > 0
            err = float(np.max(np.abs(logits.cpu().numpy()[0, :n].astype(np.float64) - ref)))
            print(f"[long prefix] {plen} tokens fed, window at frame {t0}: worst abs logit error {err:.3e}")
            worst = max(worst, err)
        assert worst < TOL["bf16"]
    finally:
        pkg.wind_set_kernels(prev)


@pytest.mark.parametrize("L,blank0,act,B,W", [(1, True, 1, 9, 4), (1, False, 0, 70, 8), (2, True, 0, 5, 16), (2, False, 1, 33, 2)])
def test_bf16_tensor_path_with_biases_and_other_blank_ids(pkg, L, blank0, act, B, W):
    # tile-sized dimensions, so the tensor-core kernels run (weights resident in shared memory, for one and for two
    # layers), with every bias vector non-zero and the blank either first or last
    w, enc, lens = ragged_case(70 + L + 2 * B, B=B, T=60, D=128, E=192, P=128, L=L, H=192, V=300, act=act,
                               blank_id=0 if blank0 else None, bias=1.0, dtype="bf16")
    rep, _ = check_against_oracle(pkg, w, enc, lens, W, 4, kernels=2)
    assert rep["stats"]["kernels"] == 2
    logits_parity(pkg, w, enc, lens, W=W, S=4, tol=TOL["bf16"], n_windows=2 * B, kernels=2)


@pytest.mark.parametrize("mode", LOOP_MODES)
def test_bf16_tensor_path_more_utterances_than_one_tile(pkg, mode):
    # 150 utterances, one K block per GEMM (H = P = 64): ten utterance groups per weight tile in the resident-weights
    # mode; two 128-row utterance tiles in the streaming mode (forced through wind_set_loop_options)
    set_loop_mode(pkg, mode)
    w, enc, lens = ragged_case(91, B=150, T=24, D=64, E=64, P=64, L=1, H=64, V=140, act=0, bias=1.0, dtype="bf16")
    rep, _ = check_against_oracle(pkg, w, enc, lens, 4, 3, kernels=2)
    assert rep["stats"]["kernels"] == 2
    logits_parity(pkg, w, enc, lens, W=4, S=3, tol=TOL["bf16"], n_windows=150, kernels=2)


@pytest.mark.parametrize("B,W,S,P,H,V,L", [
    (1, 3, 2, 128, 192, 127, 1),       # one utterance; V + 1 = exactly one vocabulary tile
    (17, 20, 3, 192, 64, 300, 2),      # window wider than the control step's 8-row pass; one K block in the joint
    (129, 1, 5, 64, 128, 140, 2),      # W = 1 (Algorithm 1), one utterance beyond a 128 tile
    (200, 8, 3, 128, 128, 257, 1),     # third vocabulary tile holds two entries
    (64, 5, 1, 192, 192, 200, 1),      # S = 1: every emission is followed by a forced advance
    (300, 2, 3, 64, 64, 130, 1),
    (40, 32, 4, 128, 64, 500, 2),
    (148, 4, 3, 256, 256, 1000, 2),
    (129, 2, 2, 256, 128, 152, 2),     # the resident plan takes 128 utterances per projection CTA
    (60, 8, 3, 64, 64, 4099, 1),       # 33 vocabulary tiles: four CTAs per tile, the resident joint runs in two waves
    (100, 8, 2, 128, 128, 2100, 2),    # two layers, 17 vocabulary tiles, two waves
    (90, 16, 3, 64, 128, 3000, 1),     # 24 tiles, six CTAs per tile, three waves of 96-row groups
])
@pytest.mark.parametrize("mode", LOOP_MODES)
def test_bf16_tensor_path_shape_sweep(pkg, mode, B, W, S, P, H, V, L):
    # shapes that send the tile planner of the loop kernel down its different branches, with the resident-weights
    # mode allowed and with wind_set_loop_options forcing the streaming mode
    set_loop_mode(pkg, mode)
    w, enc, lens = ragged_case(300 + B + W, B=B, T=20, D=64, E=64, P=P, L=L, H=H, V=V, act=B % 2, bias=1.5,
                               dtype="bf16")
    rep, _ = check_against_oracle(pkg, w, enc, lens, W, S, kernels=2)
    assert rep["stats"]["kernels"] == 2


def test_bf16_tensor_path_output_overflow(pkg):
    w, enc, lens = ragged_case(92, B=5, T=30, D=64, E=64, P=64, L=1, H=64, V=140, bias=-3.0, dtype="bf16")
    model = pkg.WindModel(w)
    full = pkg.decode(model, enc, lens, 4, 3)
    assert full[4] == 0 and full[3]["kernels"] == 2 and full[2].max() > 5
    tok, frm, olen, stats, st = pkg.decode(model, enc, lens, 4, 3, max_out=5, check=False)
    assert st == pkg.binding.WIND_ERR_OUTPUT_OVERFLOW
    assert olen.max() == 5
    for b in range(5):
        n = min(5, full[2][b])
        assert olen[b] == n and np.array_equal(tok[b, :n], full[0][b, :n]) and np.array_equal(frm[b, :n], full[1][b, :n])


def test_length_aware_batches_give_the_same_transcripts_in_fewer_lock_steps(pkg):
    # an utterance's result does not depend on what shares its batch: planned and arrival-order batches agree bit for bit
    w, enc, lens = ragged_case(95, B=45, T=60, D=64, E=64, P=128, L=1, H=128, V=200, act=1, bias=1.5, dtype="bf16")
    utts = [np.ascontiguousarray(enc[b, : lens[b]]) for b in range(45)]
    model = pkg.WindModel(w)
    t_a, f_a, steps_a = pkg.decode_dataset(model, utts, 4, 3, B=8, plan=False)
    t_p, f_p, steps_p = pkg.decode_dataset(model, utts, 4, 3, B=8, plan=True)
    for b in range(45):
        assert np.array_equal(t_a[b], t_p[b]) and np.array_equal(f_a[b], f_p[b])
    assert steps_p < steps_a
    # and both equal one batch of everything
    tok, frm, olen, _, _ = pkg.decode(model, np.nan_to_num(enc), lens, 4, 3)
    for b in range(45):
        assert np.array_equal(tok[b, : olen[b]], t_p[b]) and np.array_equal(frm[b, : olen[b]], f_p[b])


def test_cfg2_large_b1(pkg):
    cfg = ws.CONFIGS["cfg2_large_b1"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    check_against_oracle(pkg, weights, enc, lens, cfg.W, cfg.S)


def test_cfg3_full_batch_sampled_utterances(pkg):
    # the launch configuration the benchmark times (B = 128, lengths 125..2500, W = 8);
    # the oracle replays a sample of utterances (the shortest few, plus two drawn at random)
    cfg = ws.CONFIGS["cfg3_large_b128"]
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    order = np.argsort(lens)
    sample = sorted(set(order[:6].tolist() + [int(order[40]), int(order[64])]))
    rep, out8 = check_against_oracle(pkg, weights, enc, lens, cfg.W, cfg.S, sample=sample)
    st = rep["stats"]
    assert st["frames"] == int(lens.sum())
    hist = np.array(st["jump_hist"])
    assert (hist * np.arange(65)).sum() + st["forced"] == int(lens.sum())
    # properties that hold at any size
    tok, frm, olen = out8
    for b in range(cfg.B):
        f = frm[b, : olen[b]]
        assert np.all(np.diff(f) >= 0) and (len(f) == 0 or (f.max() < lens[b] and np.bincount(f).max() <= cfg.S))
        assert np.all((tok[b, : olen[b]] >= 0) & (tok[b, : olen[b]] < cfg.V))


def test_bf16_tensor_path_is_window_invariant_on_the_gpu(pkg):
    # A window row's logits come from the same operands in the same order whatever W is, so the tensor-core path
    # must emit the same (token, frame) sequences for every window size, bit for bit (the paper's claim that
    # WIND leaves the result unchanged, here for the GPU path by itself).
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 12, 5, 140)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    model = pkg.WindModel(weights)
    ref = None
    for W in (1, 2, 4, 8, 16, 64):
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, cfg.S)
        assert st == 0 and stats["kernels"] == 2
        if ref is None:
            ref = (tok, frm, olen)
        else:
            assert np.array_equal(olen, ref[2]), W
            assert np.array_equal(tok, ref[0]) and np.array_equal(frm, ref[1]), W


@pytest.mark.parametrize("case", ["large_model_w8", "two_layers_tanh_w3", "many_utterances_w1"])
def test_the_two_resident_kernels_give_the_same_transcripts(pkg, case):
    # The planner picks the resident kernel by batch size; an utterance's transcript must not depend on that choice
    # (nor, therefore, on how many utterances share its batch): same arithmetic in both, bit for bit.
    if case == "large_model_w8":
        cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 12, 5, 140)
        w, (enc, lens), W, S = ws.make_model(cfg), ws.make_enc(cfg, pad="zero"), 8, cfg.S
    elif case == "two_layers_tanh_w3":
        w, enc, lens = ragged_case(501, B=20, T=40, D=64, E=64, P=128, L=2, H=192, V=300, act=1, bias=1.0, dtype="bf16")
        enc, W, S = np.nan_to_num(enc), 3, 4
    else:
        w, enc, lens = ragged_case(502, B=150, T=24, D=64, E=64, P=64, L=1, H=64, V=140, act=0, bias=1.0, dtype="bf16")
        enc, W, S = np.nan_to_num(enc), 1, 3
    model = pkg.WindModel(w)
    outs = {}
    for mode in ("barriers", "counters"):
        set_loop_mode(pkg, mode)
        tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, S)
        assert st == 0 and stats["kernels"] == 2
        outs[mode] = (tok, frm, olen, stats["steps"])
    for a, b in zip(outs["barriers"][:3], outs["counters"][:3]):
        assert np.array_equal(a, b)
    assert outs["barriers"][3] == outs["counters"][3]


TIE_UTTS = [[5, 0, 5, 5, 1, 2, 3, 4, 5, 6, 7, 8, 5], [8, 7, 6, 5, 5, 5, 5, 5, 5, 5, 4, 3, 2, 1, 0], [3], [5, 5, 4],
            [2, 2, 3, 3, 4, 4, 8, 8], [], [0, 1, 2, 3, 4, 5, 6, 7, 8] * 3]


@pytest.mark.parametrize("path", ["f32", "bf16_simt", "bf16_tensor_barriers", "bf16_tensor_counters", "bf16_tensor_streaming"])
@pytest.mark.parametrize("blank_first", [False, True])
def test_argmax_ties_go_to_the_lowest_index_on_the_gpu(pkg, monkeypatch, path, blank_first):
    # Logits with exact ties by construction: two labels in one group of 32 vocabulary entries (one warp of the
    # tensor path's epilogue), in different groups of one 128-entry tile, in different tiles (combined through the
    # 64-bit keys), a label against the blank, and every entry equal.  The expected transcripts are written from the
    # rule (lowest index wins), and the oracle must give the same.
    if path.startswith("bf16_tensor_"):
        set_loop_mode(pkg, path[len("bf16_tensor_"):])
    w, target, winners = tie_model(blank_id=0 if blank_first else None, dtype="f32" if path == "f32" else "bf16")
    blank = w["blank_id"]
    enc, lens = tie_utterances(w["D"], TIE_UTTS)
    kernels = {"f32": 0, "bf16_simt": 1}.get(path, 2)
    prev = pkg.wind_set_kernels(kernels)
    try:
        model = pkg.WindModel(w)
        om = oracle.Model(w)
        for W, S in ((1, 1), (4, 1), (8, 2), (16, 1)):
            tok, frm, olen, stats, st = pkg.decode(model, enc, lens, W, S)
            assert st == 0 and stats["kernels"] == (2 if kernels == 2 else 1)
            otok, ofrm, on, _ = oracle.decode_batch(om, enc, lens, W=0, S=S)
            for b, types in enumerate(TIE_UTTS):
                want_tok, want_frm = tie_expected(types, winners, blank, S)
                assert list(tok[b, : olen[b]]) == want_tok and list(frm[b, : olen[b]]) == want_frm, (W, S, b)
                assert list(otok[b, : on[b]]) == want_tok and list(ofrm[b, : on[b]]) == want_frm
    finally:
        pkg.wind_set_kernels(prev)


@pytest.mark.parametrize("mode", ["barriers", "counters"])
def test_loop_kernel_timeline_can_be_recorded_without_changing_results(pkg, mode):
    set_loop_mode(pkg, mode)
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 8, 30, 80)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights)
    d = model.device
    B, T, _ = enc.shape
    max_out = T * cfg.S
    enc_d = pkg.to_device_enc(model, enc)
    len_d = torch.from_numpy(lens).to(d)
    outs = []
    wsb = pkg.alloc_workspace(model, B, T, cfg.W)
    for first in (-2, 3):
        tok = torch.full((B, max_out), -1, dtype=torch.int32, device=d)
        frm = tok.clone()
        ol = torch.zeros(B, dtype=torch.int32, device=d)
        prev = pkg.wind_set_trace(first)
        try:
            pkg.wind_decode_greedy(model, enc_d, len_d, cfg.W, cfg.S, tok, frm, ol, wsb)
        finally:
            pkg.wind_set_trace(prev)
        outs.append((tok.cpu().numpy(), frm.cpu().numpy(), ol.cpu().numpy()))
        ev = pkg.wind_read_trace(model, B, T, cfg.W, wsb)
        if first < -1:
            assert ev == []
        else:
            roles = [e for e in ev if e["role"] < 8]
            assert roles and {e["step"] for e in roles} <= {3, 4}
            assert {e["phase"] for e in roles} == {0, 1, 2} and all(e["clock"] > 0 for e in ev)
            # marks of every CTA in the first traced step: when it finished its part of the joint (mark 5, phase 0) and
            # of the projection slot (mark 15, phase 2); the CTAs with a decoder tile also when they had written the state
            for mark, ph, least in ((5, 0, 9), (15, 2, 100), (9, 1, 1)):
                ctas = sorted(e["step"] for e in ev if e["role"] == 8 + mark)
                assert len(set(ctas)) == len(ctas) >= least and all(e["phase"] == ph for e in ev if e["role"] == 8 + mark)
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)


# ---------------------------------------------------------------------------
# behaviour of the interface
# ---------------------------------------------------------------------------
def test_determinism_and_workspace_reuse(pkg):
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 6, 10, 120)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    model = pkg.WindModel(weights)
    a = pkg.decode(model, enc, lens, 8, cfg.S)
    b = pkg.decode(model, enc, lens, 8, cfg.S)
    for x, y in zip(a[:3], b[:3]):
        assert np.array_equal(x, y)
    assert a[3] == b[3]


def test_output_overflow_is_reported(pkg):
    w, enc, lens = ragged_case(50, B=4, T=30, D=16, E=16, P=16, L=1, H=32, V=20, bias=-3.0)
    model = pkg.WindModel(w)
    tok, frm, olen, stats, st = pkg.decode(model, enc, lens, 4, 3, max_out=5, check=False)
    assert st == pkg.binding.WIND_ERR_OUTPUT_OVERFLOW
    assert olen.max() == 5
    full = pkg.decode(model, enc, lens, 4, 3)
    for b in range(4):
        n = min(5, full[2][b])
        assert np.array_equal(tok[b, :n], full[0][b, :n])


def test_host_buffer_entry_point_matches_device_entry_point(pkg):
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 4, 10, 90)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights)
    ref = pkg.decode(model, enc, lens, 8, cfg.S)
    B, T, _ = enc.shape
    max_out = T * cfg.S
    enc_h = torch.from_numpy(enc).to(model.torch_dtype).pin_memory()
    len_h = torch.from_numpy(lens).pin_memory()
    tok_h = torch.full((B, max_out), -1, dtype=torch.int32).pin_memory()
    frm_h = torch.full((B, max_out), -1, dtype=torch.int32).pin_memory()
    ol_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    wsb = pkg.alloc_workspace(model, B, T, 8, host_staging_max_out=max_out)
    pkg.wind_decode_greedy_host(model, enc_h, len_h, 8, cfg.S, tok_h, frm_h, ol_h, wsb)
    assert np.array_equal(ol_h.numpy(), ref[2])
    for b in range(B):
        assert np.array_equal(tok_h.numpy()[b, : ref[2][b]], ref[0][b, : ref[2][b]])
        assert np.array_equal(frm_h.numpy()[b, : ref[2][b]], ref[1][b, : ref[2][b]])
    # only the columns up to the longest transcript come back
    longest = int(ref[2].max())
    assert longest < max_out and np.all(tok_h.numpy()[:, longest:] == -1) and np.all(frm_h.numpy()[:, longest:] == -1)
    # only the valid frames go in: poison in the host padding and a zero-length utterance change nothing
    enc2, lens2 = enc.copy(), lens.copy()
    lens2[1] = 0
    for b in range(B):
        enc2[b, lens2[b]:] = np.nan
    ref2 = pkg.decode(model, np.nan_to_num(enc2), lens2, 8, cfg.S)
    enc_h2 = torch.from_numpy(enc2).to(model.torch_dtype).pin_memory()
    len_h2 = torch.from_numpy(lens2).pin_memory()
    pkg.wind_decode_greedy_host(model, enc_h2, len_h2, 8, cfg.S, tok_h, frm_h, ol_h, wsb)
    assert np.array_equal(ol_h.numpy(), ref2[2]) and ol_h.numpy()[1] == 0
    for b in range(B):
        assert np.array_equal(tok_h.numpy()[b, : ref2[2][b]], ref2[0][b, : ref2[2][b]])
    bad = len_h2.clone()
    bad[0] = T + 1
    assert pkg.wind_decode_greedy_host(model, enc_h2, bad, 8, cfg.S, tok_h, frm_h, ol_h, wsb, check=False) == pkg.binding.WIND_ERR_INVALID_ARG


@pytest.mark.parametrize("mode", ["barriers", "counters"])
def test_unfillable_barrier_ends_in_timeout_status_and_the_context_stays_usable(pkg, mode):
    # Failure path of the persistent kernel without hanging anything: every wait in it is bounded, so a grid
    # barrier that can never fill (test hook) makes the CTAs give up after about two seconds and the call return
    # WIND_ERR_TIMEOUT; the next decode on the same context works and gives the usual result.
    set_loop_mode(pkg, mode)
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 4, 10, 40)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights)
    ref = pkg.decode(model, enc, lens, cfg.W, cfg.S)
    assert ref[4] == 0 and ref[3]["kernels"] == 2
    prev = pkg.wind_debug_stall_barrier(1)
    try:
        out = pkg.decode(model, enc, lens, cfg.W, cfg.S, check=False)
    finally:
        pkg.wind_debug_stall_barrier(prev)
    assert out[4] == pkg.binding.WIND_ERR_TIMEOUT
    again = pkg.decode(model, enc, lens, cfg.W, cfg.S)
    assert again[4] == 0
    for a, b in zip(again[:3], ref[:3]):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_device_side_inputs_out_of_range_are_reported_not_read(pkg, dtype):
    # enc_len, prefix tokens and window starts live on the device; the kernels check them there: a length outside
    # [0, T] stops the decode before any frame is read through it, a bad token or window start is replaced by a safe
    # value, and the call returns WIND_ERR_INVALID_ARG.  The next correct call on the same workspace is unaffected.
    dims = dict(D=64, E=64, P=64, L=1, H=64, V=140) if dtype == "bf16" else dict(D=20, E=12, P=24, L=2, H=40, V=30)
    w, enc, lens = ragged_case(96, B=6, T=30, bias=1.0, dtype=dtype, **dims)
    enc = np.nan_to_num(enc)
    model = pkg.WindModel(w)
    INVALID = pkg.binding.WIND_ERR_INVALID_ARG
    ref = pkg.decode(model, enc, lens, 4, 3)
    assert ref[4] == 0 and ref[3]["kernels"] == (2 if dtype == "bf16" else 1)
    for bad_len in (31, -1, 2 ** 30):
        bad = lens.copy()
        bad[5] = bad_len
        out = pkg.decode(model, enc, bad, 4, 3, check=False)
        assert out[4] == INVALID and int(out[2].sum()) == 0
    again = pkg.decode(model, enc, lens, 4, 3)
    assert again[4] == 0
    for a, b in zip(again[:3], ref[:3]):
        assert np.array_equal(a, b)
    # teacher forcing
    d = model.device
    B, T, _ = enc.shape
    enc_d = pkg.to_device_enc(model, enc)
    wsb = pkg.alloc_workspace(model, B, T, 4)
    logits = torch.zeros((B, 4, dims["V"] + 1), dtype=torch.float32, device=d)
    lens_d = torch.from_numpy(lens).to(d)
    prefix = np.ones((B, 2), np.int32)
    plen = np.full(B, 2, np.int32)
    t0 = np.zeros(B, np.int32)

    def call(prefix, t0, lens_t=lens_d):
        pr, pl, tt = (torch.from_numpy(a).to(d) for a in (prefix, plen, t0))
        return pkg.wind_eval_joint_window(model, enc_d, lens_t, 4, pr, pl, tt, logits, wsb, check=False)

    assert call(prefix, t0) == 0
    for tok in (dims["V"] + 1, -7, 2 ** 30):
        bad = prefix.copy()
        bad[3, 1] = tok
        assert call(bad, t0) == INVALID
    for start in (-1, T + 5):
        bad = t0.copy()
        bad[0] = start
        assert call(prefix, bad) == INVALID
    bad_lens = lens.copy()
    bad_lens[2] = T + 1
    assert call(prefix, t0, torch.from_numpy(bad_lens).to(d)) == INVALID
    assert call(prefix, t0) == 0


def test_workspace_too_small_is_rejected(pkg):
    w, enc, lens = ragged_case(60, B=2, T=10, D=8, E=8, P=8, L=1, H=8, V=5)
    model = pkg.WindModel(w)
    d = model.device
    enc_d = pkg.to_device_enc(model, enc)
    tok = torch.zeros((2, 30), dtype=torch.int32, device=d)
    small = torch.empty(1024, dtype=torch.uint8, device=d)
    st = pkg.wind_decode_greedy(model, enc_d, torch.from_numpy(lens).to(d), 4, 3, tok, tok.clone(), tok[:, 0].clone(), small,
                                check=False)
    assert st == pkg.binding.WIND_ERR_WORKSPACE


@pytest.mark.parametrize("V,B,W,resident", [(300, 40, 8, 1), (3000, 90, 16, 1), (3000, 16, 16, 0)])
def test_joint_alone_measurement_runs_and_leaves_the_workspace_usable(pkg, V, B, W, resident):
    # wind_bench_joint: the joint phase of the loop kernel by itself (a measurement aid).  Its figures must be consistent with
    # the tile plan, and a decode in the same workspace right after it must be what a decode in a fresh workspace gives.
    w, enc, lens = ragged_case(95 + B, B=B, T=16, D=64, E=64, P=128, L=1, H=128, V=V, act=0, bias=1.5, dtype="bf16")
    enc = np.nan_to_num(enc)
    model = pkg.WindModel(w)
    if not resident:
        set_loop_mode(pkg, "streaming")
    wsb = pkg.alloc_workspace(model, B, 16, W)
    res = pkg.wind_bench_joint(model, B, W, 20, wsb)
    st, plan = pkg.wind_debug_plan(model.dims, B, W)
    assert st == 0
    assert res["iters"] == 20 and res["ms"] > 0 and res["rows"] == B * W
    assert res["rows_issued"] >= res["rows"] and res["rows_issued"] % 16 == 0
    assert res["labels_issued"] == ((V + 1 + 127) // 128) * 128 and 1 <= res["ctas"] <= plan["grid"]
    assert res["resident"] == resident
    d = model.device
    enc_d = pkg.to_device_enc(model, enc)
    out = []
    for ws_used in (wsb, pkg.alloc_workspace(model, B, 16, W)):
        tok = torch.full((B, 48), -1, dtype=torch.int32, device=d)
        frm = tok.clone()
        ol = torch.zeros(B, dtype=torch.int32, device=d)
        pkg.wind_decode_greedy(model, enc_d, torch.from_numpy(lens).to(d), W, 3, tok, frm, ol, ws_used)
        out.append((tok.cpu().numpy(), frm.cpu().numpy(), ol.cpu().numpy()))
    assert all(np.array_equal(a, b) for a, b in zip(out[0], out[1]))


@pytest.mark.parametrize("kernels,dtype", [(1, "f32"), (2, "bf16")])
def test_profiled_decode_gives_the_same_transcripts_and_consistent_times(pkg, kernels, dtype):
    # wind_profile_decode (the benchmark's per-kernel timing leg): same outputs as the decode entry point; on the plain-ALU
    # path every launch is timed (host-driven loop), on the tensor-core path the loop kernel's time is split by its phase
    # counters, so the parts add up to the loop
    w, enc, lens = ragged_case(97, B=12, T=30, D=64, E=64, P=64, L=2, H=64, V=140, act=0, bias=1.5, dtype=dtype)
    enc = np.nan_to_num(enc)
    model = pkg.WindModel(w)
    prev = pkg.wind_set_kernels(kernels)
    try:
        tok0, frm0, ol0, stats0, st0 = pkg.decode(model, enc, lens, 4, 3)
        d = model.device
        tok = torch.full((12, 90), -1, dtype=torch.int32, device=d)
        frm = tok.clone()
        ol = torch.zeros(12, dtype=torch.int32, device=d)
        wsb = pkg.alloc_workspace(model, 12, 30, 4)
        prof = pkg.wind_profile_decode(model, pkg.to_device_enc(model, enc), torch.from_numpy(lens).to(d), 4, 3, tok, frm, ol, wsb)
    finally:
        pkg.wind_set_kernels(prev)
    assert st0 == 0
    assert np.array_equal(ol.cpu().numpy(), ol0)
    for b in range(12):
        assert np.array_equal(tok.cpu().numpy()[b, : ol0[b]], tok0[b, : ol0[b]]) and np.array_equal(frm.cpu().numpy()[b, : ol0[b]], frm0[b, : ol0[b]])
    assert prof["enc_proj_ms"] > 0 and prof["joint_ms"] > 0 and prof["pred_ms"] > 0
    if kernels == 2:
        assert prof["loop_ms"] > 0 and prof["gate_table_ms"] > 0
        assert abs(prof["joint_ms"] + prof["pred_ms"] - prof["loop_ms"]) < 0.05 * prof["loop_ms"]
        assert abs(prof["lstm_ms"] + prof["proj_ms"] - prof["pred_ms"]) < 1e-6 + 0.01 * prof["pred_ms"]
    else:
        assert prof["joint_launches"] == stats0["steps"] and prof["control_launches"] == stats0["steps"]
