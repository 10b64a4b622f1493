"""The tile planner of the tensor-core loop, checked on the host over many shapes (no GPU needed).

The plan is pure arithmetic on the model dimensions, the batch, the window, the SM count and the opt-in shared memory
per block (``wind_debug_plan``).  A plan that sizes a buffer wrongly shows up on the device as an out-of-range access;
the invariants below are what every kernel relies on, so they are swept here instead: every shared-memory region inside
the launch's dynamic shared memory and inside what the device grants, the regions that must not overlap apart, tensor
memory within its 512 columns, the CTA role sets disjoint and inside the grid, at most four joint waves.
"""
import numpy as np
import pytest

import __graft_entry__ as entry
import paper_2505_13765_b200 as pkg
from paper_2505_13765_b200 import binding as bd

STATIC_SMEM = 4096      # what the planner leaves for the kernels' static shared memory
STREAMING_STATIC_SMEM = 2048   # the streaming-mode kernels declare 1.6 KB
ALIGN_SLACK = 1024      # the kernels align their dynamic shared memory to 1 KB themselves


@pytest.fixture(scope="module", autouse=True)
def lib():
    entry.build()
    pkg.load_library()
    yield
    pkg.wind_set_loop_options()


def up(x, a=1024):
    return (x + a - 1) // a * a


def check_plan(dims, B, W, sms, optin, pl):
    P, H, L, NV = dims["P"], dims["H"], dims["L"], dims["V"] + 1
    G = pl["grid"]
    assert G == sms
    usable = pl["smem_bytes"] - ALIGN_SLACK          # after the kernel's own alignment
    static = STATIC_SMEM if pl["resident"] else STREAMING_STATIC_SMEM
    assert pl["smem_bytes"] <= optin - static, "more dynamic shared memory than the device grants beside the static part"
    assert pl["vt_count"] == (NV + 127) // 128
    rows = B * W
    assert pl["nj"] % 16 == 0 and pl["rg_count"] == (rows + pl["nj"] - 1) // pl["nj"]
    if pl["resident"]:
        assert L <= 2 and pl["l_sets"] == (3 if L == 2 else 1)
        nl, np_, nj = pl["nl"], pl["np"], pl["nj"]
        tile = pl["tile_bytes"]
        assert tile == (P // 64) * 64 * 64 * 2 and pl["buf_off"] == tile
        for off in (pl["buf_off"], pl["z_off"], pl["z_off_p"], pl["stage_off"]):
            assert off % 1024 == 0
        box_l, box_p, zb = nl * P * 2, np_ * P * 2, nj * H * 2
        staging = max(4 * 64 * 16 * 4 + 64 * 4, np_ * 68 * 4, 4 * nj * 8)
        assert pl["stage_off"] + staging <= usable, "epilogue staging runs past the launch's shared memory"
        if pl["dataflow"]:
            # decoder-type CTAs: state box and joint operand share [buf_off, stage_off)
            assert pl["z_off"] == pl["buf_off"] and pl["buf_off"] + max(box_l, zb) <= pl["stage_off"]
            # projection CTAs: box at buf_off, operand at z_off_p (its own region, or shared)
            if pl["z_off_p"] == pl["buf_off"]:
                assert pl["buf_off"] + max(box_p, zb) <= pl["stage_off"]
            else:
                assert pl["z_off_p"] >= pl["buf_off"] + box_p and pl["z_off_p"] + zb <= pl["stage_off"]
            assert nj <= 96                      # the operand build keeps one frame per utterance of a row group
            assert NV <= 1 << 20                 # label field of a key slot
        else:
            stash = min(np_ * W, 256) * 128      # prefetched enc_proj rows behind the projection's state box
            assert pl["buf_off"] + max(zb, box_l, box_p + stash) <= pl["stage_off"], "operand buffer too small"
        # tensor memory: W_out tile, two copies of the joint accumulator, then the decoder / projection accumulator
        assert pl["tm_j"] == H // 2 and pl["tm_l"] >= pl["tm_j"] + 2 * nj and pl["tm_p"] == pl["tm_l"]
        assert pl["tm_l"] + max(nl, 2 * np_) <= 512, "tensor-memory columns"
        # CTA sets
        assert pl["ut_count"] == P // 16 and pl["ht_count"] == H // 64
        assert pl["ql_count"] == (B + nl - 1) // nl and pl["qp_count"] == (B + np_ - 1) // np_
        assert pl["l_items"] == pl["ut_count"] * pl["ql_count"] and pl["p_items"] == pl["ht_count"] * pl["qp_count"]
        decoder_ctas = pl["l_sets"] * pl["l_items"]
        assert decoder_ctas + pl["p_items"] <= G, "decoder and projection CTA sets overlap"
        if pl["w_count"]:
            assert pl["w_first"] == decoder_ctas and pl["w_count"] == (B + 63) // 64
            assert pl["w_first"] + pl["w_count"] <= G - pl["p_items"], "recording CTAs overlap the projection CTAs"
        # joint: one vocabulary tile per CTA, rg_stride CTAs per tile, at most four waves
        assert pl["rg_stride"] >= 1 and pl["vt_count"] * pl["rg_stride"] <= G
        waves = (pl["rg_count"] + pl["rg_stride"] - 1) // pl["rg_stride"]
        assert 1 <= waves <= 4
    else:
        assert pl["stages_lp"] >= 2 and pl["stages_j"] >= 2
        ring = max(pl["stages_lp"] * pl["stage_lp"], pl["stages_j"] * pl["stage_j"])
        assert pl["tile_bytes"] + ring <= usable
        # staging of the projection epilogue behind the ring: pred_proj of a 128-utterance tile
        assert pl["np"] == 16 and pl["stage_off"] == pl["tile_bytes"] + ring
        assert pl["stage_off"] + 128 * pl["np"] * 4 <= usable, "projection staging runs past the launch's shared memory"
        a_bytes = 128 * 64 * 2
        assert pl["stage_lp"] >= a_bytes + max(4 * pl["slots"], pl["np"]) * 64 * 2
        assert pl["stage_j"] >= (a_bytes if pl["j_mode"] == 0 else 0) + pl["nj"] * 64 * 2
        if pl["j_mode"] == 1:
            assert pl["tile_bytes"] == (H // 64) * a_bytes
        assert pl["tm_l"] >= pl["tm_j"] + pl["nj"] and pl["tm_p"] >= pl["tm_l"] + 4 * pl["slots"] and pl["tm_p"] + pl["np"] <= 512
        assert pl["nj"] <= 256 and 4 * pl["slots"] <= 256 and pl["ul"] <= pl["slots"]
        assert pl["mt_count"] == (B + 127) // 128 and pl["ug_count"] * pl["ul"] >= P and pl["hg_count"] * pl["np"] == H


def sweep(n, seed, dataflow):
    r = np.random.default_rng(seed)
    pkg.wind_set_loop_options(dataflow=dataflow)
    seen = {"resident": 0, "streaming": 0, "unsupported": 0}
    for _ in range(n):
        dims = dict(D=64, E=64, P=int(r.choice([64, 128, 192, 256, 320, 512, 640, 1024, 1536])),
                    H=int(r.choice([64, 128, 256, 320, 512, 640, 1024, 1536])), L=int(r.choice([1, 1, 2, 2, 3])),
                    V=int(r.choice([127, 128, 255, 300, 1024, 2000, 4099, 8192, 32000])))
        B = int(r.choice([1, 2, 5, 8, 16, 17, 31, 32, 33, 64, 65, 100, 128, 129, 150, 200, 256, 300, 384, 512]))
        W = int(r.choice([1, 2, 3, 4, 5, 8, 13, 16, 24, 32, 40, 64]))
        sms = int(r.choice([148, 148, 148, 132, 108, 72]))
        optin = int(r.choice([232448, 232448, 166912, 101376]))
        st, pl = pkg.wind_debug_plan(dims, B, W, sms, optin)
        if st == bd.WIND_ERR_UNSUPPORTED:
            seen["unsupported"] += 1
            continue
        assert st == bd.WIND_OK
        try:
            check_plan(dims, B, W, sms, optin, pl)
        except AssertionError as e:
            raise AssertionError(f"{e} -- dims={dims} B={B} W={W} sms={sms} optin={optin} plan={pl}") from None
        seen["resident" if pl["resident"] else "streaming"] += 1
    return seen


@pytest.mark.parametrize("dataflow", [0, 1, -1])
def test_plan_invariants_over_many_shapes(dataflow):
    seen = sweep(4000, 100 + dataflow, dataflow)
    assert seen["resident"] > 500 and seen["streaming"] > 500, seen


def test_the_shapes_that_once_went_wrong_and_the_configured_ones():
    named = [
        # the projection CTA takes 128 utterances: its pred_proj staging must be sized from that number
        (dict(D=64, E=64, P=256, L=2, H=128, V=152), 129, 2),
        # the prefetched enc_proj rows sit behind the projection's state box: part of the buffer's size
        (dict(D=512, E=640, P=640, L=1, H=640, V=1024), 128, 8),
        (dict(D=512, E=640, P=640, L=1, H=640, V=1024), 128, 16),    # resident joint in two waves
        (dict(D=512, E=640, P=640, L=1, H=640, V=1024), 1, 8),
        (dict(D=1024, E=640, P=640, L=2, H=640, V=1024), 64, 8),
        (dict(D=1024, E=640, P=640, L=2, H=640, V=1024), 64, 16),
        (dict(D=1024, E=1024, P=1024, L=1, H=1024, V=8192), 32, 16),
    ]
    for dataflow in (0, 1):
        pkg.wind_set_loop_options(dataflow=dataflow)
        for dims, B, W in named:
            st, pl = pkg.wind_debug_plan(dims, B, W)
            assert st == bd.WIND_OK
            check_plan(dims, B, W, 148, 232448, pl)
            if dims["V"] == 8192:
                assert not pl["resident"]       # 65 vocabulary tiles at 1024 columns: weights are streamed
            else:
                assert pl["resident"] and pl["dataflow"] == dataflow
    # the planner's own choice between the two resident kernels
    pkg.wind_set_loop_options()
    large = dict(D=512, E=640, P=640, L=1, H=640, V=1024)
    assert pkg.wind_debug_plan(large, 1, 8)[1]["dataflow"] == 1 and pkg.wind_debug_plan(large, 64, 8)[1]["dataflow"] == 1
    assert pkg.wind_debug_plan(large, 128, 8)[1]["dataflow"] == 0
    assert pkg.wind_debug_plan(dict(large, L=2), 16, 8)[1]["dataflow"] == 0
    # forcing the streaming mode, and shapes outside the tensor-core path
    pkg.wind_set_loop_options(resident=False)
    assert pkg.wind_debug_plan(large, 128, 8)[1]["resident"] == 0
    pkg.wind_set_loop_options()
    assert pkg.wind_debug_plan(dict(large, P=100), 8, 4)[0] == bd.WIND_ERR_UNSUPPORTED
    assert pkg.wind_debug_plan(dict(large, V=50), 8, 4)[0] == bd.WIND_ERR_UNSUPPORTED
