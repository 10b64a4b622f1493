"""Stored oracle output (regression pin) and the multi-rank plumbing of the benchmark, on CPU."""
import json
import os
import socket

import numpy as np
import pytest
import torch

import oracle
import wind_synth as ws

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden", "cfg1_tiny_oracle.json")


def test_oracle_reproduces_stored_output_for_every_window():
    g = json.load(open(GOLDEN))
    cfg = ws.CONFIGS[g["config"]]
    assert cfg.seed == g["seed"] and cfg.S == g["S"]
    weights = ws.make_model(cfg)
    assert float(weights["b_out"][cfg.blank_id]) == g["b_out_blank"]
    enc, lens = ws.make_enc(cfg, pad="nan")
    assert [int(x) for x in lens] == g["lens"]
    om = oracle.Model(weights)
    for W in (0, 1, 2, 4, 7, 64):   # 0 = Algorithm 1; the rest Algorithm 2, which must give the same result
        tok, frm, n, _ = oracle.decode_batch(om, enc, lens, W=W, S=cfg.S)
        for b in range(cfg.B):
            assert [int(x) for x in tok[b, : n[b]]] == g["tokens"][b], W
            assert [int(x) for x in frm[b, : n[b]]] == g["frames"][b], W
    # what the stored sequence must satisfy whatever the arithmetic: frames non-decreasing, at most S per frame
    for b in range(cfg.B):
        f = np.array(g["frames"][b])
        assert np.all(np.diff(f) >= 0) and np.bincount(f).max() <= cfg.S and f.max() < g["lens"][b]
        assert all(0 <= t < cfg.V for t in g["tokens"][b])


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    import bench
    r, local, w = bench.dist_setup(world, backend="gloo")
    assert (r, w) == (rank, world)
    bench.barrier(w)
    # every rank decodes its own replica: rank 1 is the slower one, the job's time is the max over ranks
    ms_local = 100.0 if rank == 0 else 250.0
    value, ms_per_step = bench.aggregate_rtfx(audio_seconds_per_rank_step=1000.0, steps=5, ms_local=ms_local, world=w)
    out[rank] = (value, ms_per_step)
    bench.barrier(w)
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_rank_and_sums_the_work():
    import torch.multiprocessing as mp
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        value, ms_per_step = res[rank]
        assert ms_per_step == pytest.approx(50.0)                       # 250 ms over 5 steps: the slower rank
        assert value == pytest.approx(1000.0 * 5 * 2 / 0.250)           # both replicas' audio over that time


def test_schedule_counts_rebuilt_from_transcripts_match_the_oracle_and_a_hand_case():
    # the benchmark's comparison of batched schedules counts passes on transcripts: the rebuilt per-utterance iterations
    # must be the oracle's own (its step counter), and the two schedules' passes those of a case worked by hand
    import bench
    from naive_model import random_weights
    r = np.random.default_rng(5)
    w = random_weights(r, 8, 6, 10, 1, 12, 9, blank_bias=1.0)
    om = oracle.Model(w)
    lens = np.array([30, 17, 0, 25], np.int32)
    enc = r.standard_normal((4, 30, 8)).astype(np.float32)
    for W in (1, 3, 8):
        for S in (1, 3):
            tok, frm, on, st = oracle.decode_batch(om, enc, lens, W=W, S=S)
            kinds = bench.step_kinds(lens, on, frm, W, S)
            per_utt = [oracle.decode_batch(om, enc[b:b + 1], lens[b:b + 1], W=W, S=S)[3]["steps"] for b in range(4)]
            assert [len(k) for k in kinds] == per_utt
            assert [int(k.sum()) for k in kinds] == [int(x) for x in on]
    # utterance A: blank, blank, emit, emit; utterance B: emit, blank, emit
    kinds = [np.array([0, 0, 1, 1], bool), np.array([1, 0, 1], bool)]
    c = bench.schedule_counts(kinds)
    # lock step: 4 passes.  label looping: iteration 1 needs 3 joint passes (A's two blank windows), iteration 2 needs 2
    # (B's blank window), then nothing is left: 5 joint passes, 2 decoder updates
    assert c == {"lock_step_passes": 4, "label_looping_joint_passes": 5, "label_looping_decoder_updates": 2}
