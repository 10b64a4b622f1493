"""GPU parity of Eq. (1), the first-output distribution P'(v, t) of a window, against the CPU oracle.

Tolerance: a logit may be off by the joint's bound (1e-4 fp32 path, 2e-2 bf16-weight path); the log-softmax of a row
moves by at most twice that, and log P'(v, t) adds the blank log-probabilities of the t rows before it, so the bound
on log P'(v, t) is 2 * (t + 1) * bound (+ fp32 rounding of the sums).  The top-K pairs must be the oracle's K best up
to that tolerance: the k-th value returned must equal the oracle's k-th best value within the bound, and each returned
pair's own oracle value must match the value returned for it.
"""
import numpy as np
import pytest

import oracle
import wind_synth as ws
from naive_model import random_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

BOUND = {"f32": 1e-4, "bf16": 2e-2}


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_13765_b200 as p
    p.load_library()
    return p


def run_case(pkg, weights, enc, lens, W, K, seed):
    om = oracle.Model(weights)
    dtype = weights["dtype"]
    B, T, _ = enc.shape
    NV = int(weights["V"]) + 1
    r = np.random.default_rng(seed)
    otok, ofrm, on, _ = oracle.decode_batch(om, enc, lens, W=0, S=3)
    t0 = np.array([r.integers(0, max(1, lens[b])) if lens[b] else 0 for b in range(B)], np.int32)
    t0[0] = max(0, lens[0] - 2)     # a window cut short by the end of the utterance
    plen = np.array([int(np.searchsorted(ofrm[b, : on[b]], t0[b], side="left")) for b in range(B)], np.int32)
    U = max(1, int(plen.max()))
    prefix = np.zeros((B, U), np.int32)
    for b in range(B):
        prefix[b, : plen[b]] = otok[b, : plen[b]]
    model = pkg.WindModel(weights)
    d = model.device
    enc_d = pkg.to_device_enc(model, enc)
    logp = torch.full((B, W, NV), float("nan"), dtype=torch.float32, device=d)
    tl = torch.full((B, K), -7, dtype=torch.int32, device=d)
    tj = torch.full((B, K), -7, dtype=torch.int32, device=d)
    tv = torch.full((B, K), float("nan"), dtype=torch.float32, device=d)
    wsb = pkg.alloc_workspace(model, B, T, W)
    pkg.wind_window_first_output(model, enc_d, torch.from_numpy(lens).to(d), W, torch.from_numpy(prefix).to(d),
                                 torch.from_numpy(plen).to(d), torch.from_numpy(t0).to(d), logp, wsb, K=K, top_label=tl,
                                 top_jump=tj, top_logp=tv)
    got = logp.cpu().numpy().astype(np.float64)
    tl, tj, tv = tl.cpu().numpy(), tj.cpu().numpy(), tv.cpu().numpy().astype(np.float64)
    worst = 0.0
    rows = 0
    for b in range(B):
        ref = oracle.first_output_logprobs(om, enc[b], int(lens[b]), prefix[b, : plen[b]], int(t0[b]), W)
        n = ref.shape[0]
        assert n == max(0, min(W, int(lens[b]) - int(t0[b])))
        assert np.all(np.isnan(got[b, n:]))            # rows past the window are left untouched
        if n == 0:
            assert np.all(tl[b] == -1) and np.all(tj[b] == -1)
            continue
        rows += n
        assert np.array_equal(np.isneginf(got[b, :n]), np.isneginf(ref))   # zeros of Eq. (1): blank before the last row
        for t in range(n):
            tol = 2 * (t + 1) * BOUND[dtype] + 1e-4
            fin = np.isfinite(ref[t])
            err = np.max(np.abs(got[b, t][fin] - ref[t][fin]))
            worst = max(worst, err / tol)
            assert err <= tol, (b, t, err, tol)
        assert abs(np.exp(got[b, :n]).sum() - 1.0) < 5e-3     # still a distribution over the first output
        # the K best pairs
        order = np.sort(ref[np.isfinite(ref)])[::-1]
        kk = min(K, order.size)
        tolk = 2 * n * BOUND[dtype] + 1e-4
        assert np.all(np.diff(tv[b, :kk]) <= 0)
        seen = set()
        for k in range(kk):
            t, v = int(tj[b, k]), int(tl[b, k])
            assert 0 <= t < n and 0 <= v < NV and (t, v) not in seen
            seen.add((t, v))
            assert tv[b, k] == pytest.approx(got[b, t, v], abs=0)         # the value returned is the entry's value
            assert abs(tv[b, k] - order[k]) <= tolk                       # and it is the k-th best up to the bound
            assert abs(ref[t, v] - tv[b, k]) <= tolk
        assert np.all(tl[b, kk:] == -1)
    assert rows > 0
    print(f"[first-output] {rows} rows, worst error / tolerance {worst:.3f}")


def test_first_output_fp32_odd_shapes(pkg):
    r = np.random.default_rng(900)
    w = random_weights(r, 37, 29, 41, 2, 67, 45, blank_id=0, act=1, blank_bias=0.8, bias_scale=0.1)
    B, T = 6, 30
    lens = r.integers(1, T + 1, size=B).astype(np.int32)
    lens[0] = T
    lens[1] = 0
    enc = r.standard_normal((B, T, 37)).astype(np.float32)
    for b in range(B):
        enc[b, lens[b]:] = np.nan
    run_case(pkg, w, enc, lens, W=5, K=4, seed=1)


@pytest.mark.parametrize("name,W,K", [("cfg3_large_b128", 8, 3), ("cfg5_bigvocab", 4, 8), ("cfg3_large_b128", 4, 12)])
def test_first_output_bf16_model_shapes(pkg, name, W, K):
    cfg = ws.small_variant(ws.CONFIGS[name], 6, 20, 70)
    weights = ws.make_model(cfg)
    enc, lens = ws.make_enc(cfg, pad="nan")
    run_case(pkg, weights, enc, lens, W=W, K=K, seed=2)
