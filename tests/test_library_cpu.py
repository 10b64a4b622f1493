"""Host-side checks of the CUDA library that need no GPU: it loads, exports every symbol the
header declares, sizes its workspace as documented and rejects bad arguments before any launch."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
import paper_2505_13765_b200 as pkg
from paper_2505_13765_b200 import binding as bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return pkg.load_library()


def large_model(**kw):
    d = dict(D=512, E=640, P=640, L=1, H=640, V=1024, blank_id=1024, act=0, dtype=1)
    d.update(kw)
    return bd.wind_model_t(**d)


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "wind.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(wind_[a-z_]+)\s*\(", text))
    assert declared == set(bd.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    names = [pkg.wind_status_string(i) for i in range(8)]
    assert names[0] == "WIND_OK" and len(set(names)) == 8
    assert pkg.wind_status_string(99) == "WIND_ERR_UNKNOWN"


def test_workspace_grows_with_window_only_by_keys_and_activations(lib):
    # The paper's memory analysis: WIND's only extra state is the window's logits,
    # W x (V+1) floats per utterance (16 x 1025 = 16400 floats for W = 16).  Here the
    # logits stay on chip; per window row the workspace keeps three 8-byte argmax keys (two buffers by step
    # parity, one for the best non-blank label in window-based decoding), the joint's H bf16 activations and, for
    # window-based decoding, the blank logit and four (maximum, sum of exponentials) pairs per vocabulary tile; the
    # resident kernel without grid barriers adds one stamped 8-byte key per vocabulary tile (their number padded to even).
    m = large_model()
    B, T = 128, 2500
    tiles = (m.V + 1 + 127) // 128
    base = pkg.wind_workspace_bytes(m, B, T, 2)   # B * W = 256 rows: no row padding at even W
    for W in (4, 8, 16, 64):
        extra = pkg.wind_workspace_bytes(m, B, T, W) - base
        assert extra == B * (W - 2) * (3 * 8 + 2 * m.H + 4 + 8 * 4 * tiles + 8 * ((tiles + 1) // 2 * 2))
        assert extra <= 4 * B * W * (m.V + 1)  # below the paper's W x (V+1) floats per utterance
    assert 16 * 1025 == 16400
    # dominated by enc_proj [B, T, H] in bf16; the gate table adds (V+1) x 4P floats
    table = 4 * (m.V + 1) * 4 * m.P
    assert base >= 2 * B * T * m.H + table and base < 2 * B * T * m.H * 1.02 + table + (1 << 22)


def test_invalid_arguments_are_rejected_on_the_host(lib):
    m = large_model()
    n = C.c_size_t(0)
    ref = C.byref(m)
    assert lib.wind_workspace_bytes(None, 1, 1, 1, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(ref, 0, 10, 1, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(ref, 1, 10, 0, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(ref, 1, 10, 65, C.byref(n)) == bd.WIND_ERR_UNSUPPORTED
    assert lib.wind_workspace_bytes(ref, 1, 10, 4, None) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(C.byref(large_model(blank_id=1025)), 1, 10, 4, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(C.byref(large_model(L=9)), 1, 10, 4, C.byref(n)) == bd.WIND_ERR_UNSUPPORTED
    assert lib.wind_workspace_bytes(C.byref(large_model(act=2)), 1, 10, 4, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_workspace_bytes(ref, 4096, 4096, 4, C.byref(n)) == bd.WIND_ERR_UNSUPPORTED  # > 2^31 elements
    # null weights / buffers: rejected before any CUDA call (this machine may have no GPU at all)
    args = [ref, None, None, 1, 10, 4, 5, None, None, None, 50, None, 0, None]
    assert lib.wind_decode_greedy(*args) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_decode_window_greedy(*args) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_decode_greedy_host(*args) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_eval_joint_window(ref, None, None, 1, 10, 4, None, 0, None, None, None, None, 0, None) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_read_stats(None, None, None) == bd.WIND_ERR_INVALID_ARG
    fo = [ref, None, None, 1, 10, 4, None, 0, None, None, None, 0, None, None, None, None, 0, None]
    assert lib.wind_window_first_output(*fo) == bd.WIND_ERR_INVALID_ARG
    fo[11] = -1
    assert lib.wind_window_first_output(*fo) == bd.WIND_ERR_INVALID_ARG      # K < 0
    fo[11] = 3
    assert lib.wind_window_first_output(*fo) == bd.WIND_ERR_INVALID_ARG      # K > 0 without output arrays
    # beam search: shape limits and null pointers
    assert lib.wind_beam_workspace_bytes(ref, 100, 8, 0, 3, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_beam_workspace_bytes(ref, 100, 8, 17, 3, C.byref(n)) == bd.WIND_ERR_UNSUPPORTED
    assert lib.wind_beam_workspace_bytes(ref, 100, 65, 4, 3, C.byref(n)) == bd.WIND_ERR_UNSUPPORTED
    assert lib.wind_beam_workspace_bytes(ref, 100, 8, 4, 3, None) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_beam_workspace_bytes(ref, 1500, 8, 4, 10, C.byref(n)) == bd.WIND_OK and 0 < n.value < (1 << 30)
    nh, ns = C.c_int32(0), C.c_int64(0)
    assert lib.wind_beam_search(ref, None, 100, 8, 4, 3, 0, 8, 100, None, None, None, None, C.byref(nh), C.byref(ns), None, 0, None) \
        == bd.WIND_ERR_INVALID_ARG
    n_ev = C.c_int32(0)
    assert lib.wind_read_trace(ref, 1, 10, 4, None, None, None, 0, C.byref(n_ev)) == bd.WIND_ERR_INVALID_ARG


def test_plan_batches_sorts_by_length_and_minimises_the_sum_of_batch_maxima(lib):
    import itertools
    import numpy as np
    r = np.random.default_rng(5)
    for N, B in ((0, 4), (1, 4), (7, 3), (128, 128), (300, 64), (12, 1)):
        lens = r.integers(0, 50, size=N).astype(np.int32)
        order, batch_T = pkg.wind_plan_batches(lens, B)
        assert sorted(order.tolist()) == list(range(N))                      # a permutation
        assert len(batch_T) == (N + B - 1) // B
        sl = lens[order]
        assert np.all(np.diff(sl) <= 0)                                      # longest first
        for a, b in zip(order[:-1], order[1:]):                              # equal lengths keep their order
            if lens[a] == lens[b]:
                assert a < b
        for k, T in enumerate(batch_T):
            assert T == lens[order[k * B: (k + 1) * B]].max()
        arrival = sum(int(lens[k: k + B].max()) for k in range(0, N, B))
        assert int(batch_T.sum()) <= arrival
    # ranks take batches r, r + R, ...: together every utterance exactly once, loads within one (shortest) batch
    lens = r.integers(1, 2500, size=1000).astype(np.int32)
    order, batch_T = pkg.wind_plan_batches(lens, 64)
    shares = [[k for k in range(len(batch_T)) if k % 4 == rank] for rank in range(4)]
    seen = sorted(int(i) for sh in shares for k in sh for i in order[k * 64: (k + 1) * 64])
    assert seen == list(range(1000))
    loads = [int(batch_T[sh].sum()) for sh in shares]
    assert max(loads) - min(loads) <= int(batch_T[0])
    # brute force on a tiny set: no grouping into batches of 2 has a smaller sum of batch maxima
    lens = np.array([9, 2, 7, 7, 1, 4], np.int32)
    order, batch_T = pkg.wind_plan_batches(lens, 2)
    best = min(sum(max(lens[list(perm[k: k + 2])]) for k in range(0, 6, 2)) for perm in itertools.permutations(range(6)))
    assert int(batch_T.sum()) == best
    n = C.c_int32(0)
    buf = (C.c_int32 * 4)()
    assert lib.wind_plan_batches(None, 4, 2, buf, None, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_plan_batches(buf, 4, 0, buf, None, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_plan_batches(buf, -1, 2, buf, None, C.byref(n)) == bd.WIND_ERR_INVALID_ARG
    neg = (C.c_int32 * 2)(3, -1)
    assert lib.wind_plan_batches(neg, 2, 2, buf, None, C.byref(n)) == bd.WIND_ERR_INVALID_ARG


def test_workspace_of_refilled_rows_holds_the_projection_of_the_whole_set(lib):
    # wind_refill_workspace_bytes(N utterances, B rows): everything per row as in wind_workspace_bytes(B), enc_proj for N
    m = large_model()
    T, B, W = 500, 32, 8
    base = pkg.wind_workspace_bytes(m, B, T, W)
    for N in (1, 32, 33, 256):
        n = pkg.wind_refill_workspace_bytes(m, N, T, B, W)
        extra = max(N, B) - B
        assert 0 <= n - base - extra * T * m.H * 2 < 4096, (N, n - base)      # bf16 enc_proj rows, up to alignment
    nb = C.c_size_t(0)
    assert lib.wind_refill_workspace_bytes(C.byref(m), 0, T, B, W, C.byref(nb)) == bd.WIND_ERR_INVALID_ARG
    assert lib.wind_refill_workspace_bytes(C.byref(m), 10 ** 6, 5000, B, W, C.byref(nb)) == bd.WIND_ERR_UNSUPPORTED
    # host staging of the host-buffer entry point: input frames and the three output arrays
    st = pkg.wind_host_staging_bytes(m, B, T, 100)
    assert 0 <= st - (B * T * m.D * 2 + B * 4 + 2 * B * 100 * 4 + B * 4) < 8 * 256
    assert isinstance(lib.wind_last_cuda_error(), bytes)      # empty until a CUDA call fails


def test_debug_hooks_round_trip(lib):
    assert pkg.wind_set_trace(5) == -2 and pkg.wind_set_trace(-9) == 5 and pkg.wind_set_trace(-2) == -2
    assert pkg.wind_debug_stall_barrier(2) == 0 and pkg.wind_debug_stall_barrier(0) == 2


def test_set_kernels_round_trip(lib):
    prev = pkg.wind_set_kernels(bd.WIND_KERNELS_SIMT)
    assert pkg.wind_set_kernels(prev) == bd.WIND_KERNELS_SIMT
    assert pkg.wind_set_kernels(77) == prev  # out of range: unchanged
    assert pkg.wind_set_kernels(prev) == prev


def test_product_path_does_not_touch_the_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2505_13765_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f
