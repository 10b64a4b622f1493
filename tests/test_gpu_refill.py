"""GPU parity of decoding N utterances on B batch rows that are refilled inside the persistent loop.

Algorithm 2 treats the utterances of a batch independently, so what an utterance's row did before it moved in must not
show in its transcript: every utterance's (tokens, frames) from wind_decode_greedy_refill must equal, bit for bit, the
ones wind_decode_greedy gives for it with all N utterances in one batch (same kernel mode forced for both), for every
number of rows -- one row (the utterances one after the other), a few, exactly N, more rows than utterances (the shapes
are such that every row count gets the same kind of tile plan as the batch of N; the randomised sweep in
test_gpu_fuzz.py compares against fixed batches of exactly B rows instead, which holds for any shape).  A sample
is also replayed through the CPU oracle under the margin rule of the parity tests, and the counters are checked
against what the transcripts say.
"""
import numpy as np
import pytest

import oracle
from conftest import set_loop_mode
from test_gpu_parity import MARGIN, ragged_case

torch = pytest.importorskip("torch")
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


CASES = {
    # name: (N, T, P, H, V, L, act, W, S, rows to try)
    "one_layer_w4": (37, 40, 128, 128, 200, 1, 0, 4, 3, [1, 3, 8, 37, 50]),
    "two_layers_w8": (29, 30, 192, 64, 300, 2, 1, 8, 2, [2, 5, 29]),
    "algorithm1_many_rows": (210, 16, 64, 64, 140, 1, 0, 1, 4, [70, 150]),
    "wide_window_two_waves": (40, 48, 64, 128, 3000, 1, 1, 16, 3, [6, 33]),
}


@pytest.mark.parametrize("mode", ["barriers", "streaming"])
@pytest.mark.parametrize("case", list(CASES))
def test_refilled_rows_give_every_utterance_its_single_batch_transcript(pkg, mode, case):
    N, T, P, H, V, L, act, W, S, rows = CASES[case]
    set_loop_mode(pkg, mode)
    w, enc, lens = ragged_case(700 + N, B=N, T=T, D=64, E=64, P=P, L=L, H=H, V=V, act=act, bias=1.5, dtype="bf16")
    lens[N // 2] = 0                       # an empty utterance in the middle of the queue
    lens[-1] = T                           # and a full-length one at its end
    enc = np.nan_to_num(enc)
    for b in range(N):
        enc[b, lens[b]:] = np.nan          # padding is never read
    model = pkg.WindModel(w)
    tok1, frm1, olen1, stats1, st1 = pkg.decode(model, enc, lens, W, S)
    assert st1 == 0 and stats1["kernels"] == 2
    om = oracle.Model(w)
    for B in rows:
        tok, frm, olen, stats, st = pkg.decode_refill(model, enc, lens, B, W, S)
        assert st == 0 and stats["kernels"] == 2, (B, st)
        assert np.array_equal(olen, olen1), f"{case} rows={B}: token counts differ"
        for u in range(N):
            assert np.array_equal(tok[u, : olen[u]], tok1[u, : olen1[u]]), f"{case} rows={B}: tokens of utterance {u}"
            assert np.array_equal(frm[u, : olen[u]], frm1[u, : olen1[u]]), f"{case} rows={B}: frames of utterance {u}"
            assert np.all(tok[u, olen[u]:] == -1)
        assert stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
        hist = np.array(stats["jump_hist"])
        assert (hist * np.arange(65)).sum() + stats["forced"] == int(lens.sum())
        if B >= N:
            assert stats["steps"] == stats1["steps"]      # nothing to refill: the same lock steps as one batch
        else:
            # fewer rows than utterances: more lock steps than one batch of everything, but far fewer than the
            # utterances decoded one after the other
            assert stats["steps"] >= stats1["steps"]
        print(f"[refill] {case} {mode}: {N} utterances on {B} rows, {stats['steps']} lock steps "
              f"(one batch of {N}: {stats1['steps']})")
    # a sample against the oracle (margin rule), on the last row count
    for u in (0, N // 3, N - 1):
        r = oracle.replay_verify(om, enc[u], int(lens[u]), S, tok[u, : olen[u]], frm[u, : olen[u]], MARGIN)
        assert r["rc"] == 0, f"utterance {u}: {r}"


def test_refill_needs_fewer_lock_steps_than_planned_batches(pkg):
    # lengths spread over 10..60 frames: with 8 rows, length-sorted batches still wait for each batch's longest
    # utterance; refilled rows do not
    w, enc, lens = ragged_case(801, B=64, T=60, D=64, E=64, P=128, L=1, H=128, V=200, act=0, bias=1.5, dtype="bf16")
    lens = np.maximum(lens, 10).astype(np.int32)
    enc = np.nan_to_num(enc)
    model = pkg.WindModel(w)
    utts = [np.ascontiguousarray(enc[b, : lens[b]]) for b in range(64)]
    t_p, f_p, steps_planned = pkg.decode_dataset(model, utts, 4, 3, B=8, plan=True)
    tok, frm, olen, stats, st = pkg.decode_refill(model, enc, lens, 8, 4, 3)
    assert st == 0
    for u in range(64):
        assert np.array_equal(tok[u, : olen[u]], t_p[u]) and np.array_equal(frm[u, : olen[u]], f_p[u])
    assert stats["steps"] < steps_planned, (stats["steps"], steps_planned)
    print(f"[refill] 64 utterances on 8 rows: {stats['steps']} lock steps refilled, {steps_planned} in length-sorted batches")
    # the list helper: refilled rows, longest first, results back in the list's order; an fp32 model falls back to batches
    t_r, f_r, steps_r = pkg.decode_dataset(model, utts, 4, 3, B=8, plan=True, refill=True)
    for u in range(64):
        assert np.array_equal(t_r[u], t_p[u]) and np.array_equal(f_r[u], f_p[u])
    assert steps_r < steps_planned
    w32, enc32, lens32 = ragged_case(805, B=10, T=12, D=64, E=64, P=64, L=1, H=64, V=140, dtype="f32")
    m32 = pkg.WindModel(w32)
    u32 = [np.ascontiguousarray(np.nan_to_num(enc32)[b, : lens32[b]]) for b in range(10)]
    a = pkg.decode_dataset(m32, u32, 4, 3, B=4, refill=True)
    b = pkg.decode_dataset(m32, u32, 4, 3, B=4, refill=False)
    assert all(np.array_equal(x, y) for x, y in zip(a[0], b[0])) and a[2] == b[2]


def test_refill_rejects_what_it_does_not_cover(pkg):
    bd = pkg.binding
    w, enc, lens = ragged_case(802, B=6, T=12, D=64, E=64, P=64, L=1, H=64, V=140, dtype="f32")
    model = pkg.WindModel(w)
    enc = np.nan_to_num(enc)
    assert pkg.decode_refill(model, enc, lens, 2, 4, 3, check=False)[4] == bd.WIND_ERR_UNSUPPORTED   # fp32 model
    w, enc, lens = ragged_case(803, B=6, T=12, D=64, E=64, P=64, L=1, H=64, V=140, dtype="bf16")
    model = pkg.WindModel(w)
    enc = np.nan_to_num(enc)
    bad = lens.copy()
    bad[5] = 13                                                                                      # beyond T, in the queue
    assert pkg.decode_refill(model, enc, bad, 2, 4, 3, check=False)[4] == bd.WIND_ERR_INVALID_ARG
    ok = pkg.decode_refill(model, enc, lens, 2, 4, 3)                                                # the context is fine
    assert ok[4] == 0


def test_a_queue_longer_than_the_projection_kernels_prefix_table(pkg):
    # more than 2048 utterances: the encoder projection takes its one-tile-per-CTA form (the persistent kernel keeps the
    # utterances' tile counts in shared memory); short utterances, every one checked against fixed batches of 64 rows
    N, T, B, W, S = 2100, 6, 64, 4, 2
    w, enc, lens = ragged_case(804, B=N, T=T, D=64, E=64, P=64, L=1, H=128, V=140, bias=1.0, dtype="bf16")
    enc = np.nan_to_num(enc)
    model = pkg.WindModel(w)
    tok, frm, olen, stats, st = pkg.decode_refill(model, enc, lens, B, W, S)
    assert st == 0 and stats["frames"] == int(lens.sum()) and stats["tokens"] == int(olen.sum())
    for k in range(0, N, B):
        m = min(B, N - k)
        e = np.zeros((B, T, 64), np.float32); l = np.zeros(B, np.int32)
        e[:m], l[:m] = enc[k: k + m], lens[k: k + m]
        t1, f1, o1, _, st1 = pkg.decode(model, e, l, W, S)
        assert st1 == 0 and np.array_equal(o1[:m], olen[k: k + m])
        for u in range(m):
            assert np.array_equal(t1[u, : o1[u]], tok[k + u, : o1[u]]) and np.array_equal(f1[u, : o1[u]], frm[k + u, : o1[u]])
