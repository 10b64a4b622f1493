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
