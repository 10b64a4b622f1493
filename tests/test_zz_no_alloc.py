"""The entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc (and torch's allocator) must not be called: in a
section that may not synchronise the device, inside a process whose device memory is already
handed out, or in a loop with a hard latency bound.  ``wind_eval_joint_window_static`` serves
them from a scratch array built into the library.  This file checks it, through the C ABI,
against ``wind_eval_joint_window`` (caller-allocated workspace) and against the CPU oracle on the
same inputs, twice in a row with different inputs, so that anything the first call left in the
shared array would show, and checks that the device's free memory is the same after a call as
before it (the first call on a device may load the library's image and is not measured).

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest

import oracle
import wind_synth as ws
from naive_model import random_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

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


def _case(seed, dtype, B, T, D, E, P, L, H, V):
    r = np.random.default_rng(7000 + seed)
    w = random_weights(r, D, E, P, L, H, V, act=seed % 2, blank_bias=1.0, bias_scale=0.1)
    w["dtype"] = dtype
    if dtype == "bf16":
        for k in ("emb", "w_enc", "w_pred", "w_out"):
            w[k] = ws.bf16_round(w[k])
        w["w_ih"] = [ws.bf16_round(a) for a in w["w_ih"]]
        w["w_hh"] = [ws.bf16_round(a) for a in w["w_hh"]]
    lens = r.integers(1, T + 1, size=B).astype(np.int32)
    lens[0] = T
    enc = r.standard_normal((B, T, D)).astype(np.float32)
    if dtype == "bf16":
        enc = ws.bf16_round(enc)
    for b in range(B):
        enc[b, lens[b]:] = np.nan
    U = 4
    prefix = r.integers(0, V, size=(B, U)).astype(np.int32)
    plen = r.integers(0, U + 1, size=B).astype(np.int32)
    t0 = np.array([r.integers(0, lens[b]) for b in range(B)], np.int32)
    t0[0] = T - 1  # a window cut short by the end of the utterance
    return w, enc, lens, prefix, plen, t0


def _both(pkg, case, W):
    w, enc, lens, prefix, plen, t0 = case
    model = pkg.WindModel(w)
    d = model.device
    B, T, _ = enc.shape
    NV = model.dims["V"] + 1
    enc_d = pkg.to_device_enc(model, enc)
    args = [torch.from_numpy(a).to(d) for a in (lens, prefix, plen, t0)]
    ref = torch.full((B, W, NV), float("nan"), dtype=torch.float32, device=d)
    wsb = pkg.alloc_workspace(model, B, T, W)
    pkg.wind_eval_joint_window(model, enc_d, args[0], W, args[1], args[2], args[3], ref, wsb)
    got = torch.full((B, W, NV), float("nan"), dtype=torch.float32, device=d)
    # everything the call needs is allocated by now; the call itself allocates nothing.  One untimed call first:
    # the very first use on a device resolves the array's address (and may load the library's image).
    pkg.wind_eval_joint_window_static(model, enc_d, args[0], W, args[1], args[2], args[3], got)
    torch.cuda.synchronize()
    got.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(d)
    reserved_before = torch.cuda.memory_reserved(d)
    pkg.wind_eval_joint_window_static(model, enc_d, args[0], W, args[1], args[2], args[3], got)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(d)
    assert torch.cuda.memory_reserved(d) == reserved_before      # nothing taken from torch's allocator
    assert free_after >= free_before, (free_before, free_after)   # nothing taken from the device
    # the oracle's logits of the same windows
    om = oracle.Model(w)
    want = []
    for b in range(B):
        o, *_ = oracle.eval_joint_window(om, enc[b], int(lens[b]), prefix[b, : plen[b]], int(t0[b]), W)
        want.append(o)
    return ref.cpu().numpy(), got.cpu().numpy(), lens, t0, want


@pytest.mark.parametrize("dtype,dims", [
    ("f32", dict(B=5, T=40, D=48, E=24, P=40, L=2, H=72, V=50)),
    ("bf16", dict(B=6, T=50, D=128, E=128, P=128, L=1, H=128, V=255)),
])
def test_static_scratch_matches_caller_workspace_twice_in_a_row(pkg, dtype, dims):
    W = 4
    for call, seed in enumerate((1, 2)):  # second call: other weights and inputs, same shared array
        ref, got, lens, t0, want = _both(pkg, _case(seed, dtype, **dims), W)
        rows = 0
        for b in range(ref.shape[0]):
            n = max(0, min(W, int(lens[b]) - int(t0[b])))
            rows += n
            assert want[b].shape[0] == n
            assert np.all(np.isfinite(ref[b, :n]))
            assert np.max(np.abs(got[b, :n] - ref[b, :n])) <= TOL[dtype], (call, b)
            if n:
                assert np.max(np.abs(got[b, :n].astype(np.float64) - want[b])) <= TOL[dtype], (call, b)
            assert np.all(np.isnan(got[b, n:])) and np.all(np.isnan(ref[b, n:]))  # rows past the window untouched
        assert rows > 0


def test_static_scratch_rejects_what_does_not_fit(pkg):
    cfg = ws.small_variant(ws.CONFIGS["cfg3_large_b128"], 64, 500, 500)
    weights = ws.make_model(cfg)
    model = pkg.WindModel(weights)
    need = pkg.wind_workspace_bytes(model, 64, 500, 8)
    assert need > pkg.binding.WIND_STATIC_WORKSPACE_BYTES
    d = model.device
    enc = torch.zeros((64, 500, cfg.D), dtype=model.torch_dtype, device=d)
    z = torch.zeros(64, dtype=torch.int32, device=d)
    lens = torch.full((64,), 500, dtype=torch.int32, device=d)
    logits = torch.zeros((64, 8, cfg.V + 1), dtype=torch.float32, device=d)
    st = pkg.wind_eval_joint_window_static(model, enc, lens, 8, None, z, z, logits, check=False)
    assert st == pkg.binding.WIND_ERR_WORKSPACE
