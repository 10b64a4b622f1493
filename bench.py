#!/usr/bin/env python
"""Benchmark of batched greedy WIND decoding on synthetic data (one JSON line on stdout).

A "step" is one pass of the whole hot path over one batch: a single
``wind_decode_greedy`` call (encoder projection, start-of-sequence decoder update,
device-resident decoding loop) on the B = 128 FastConformer-Large-shaped workload.
Metric: RTFx = audio seconds decoded per second at 80 ms per encoder frame.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME] [--window W]

With N > 1 (under torchrun) every rank decodes its own replica of the batch: the path
has no exchange step, so there is no collective in it; ranks only meet at the barrier
and at the max-over-ranks of the device time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FRAME_SECONDS = 0.08


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str | None):
        self.uuid = uuid
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]
            if self.uuid:
                cmd += ["-i", self.uuid]
            self.proc = subprocess.Popen(cmd, stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------
# rank plumbing (barrier + max over ranks); gloo on CPU in the tests, nccl on GPUs
# ---------------------------------------------------------------------------
def dist_setup(n_gpus: int, backend: str | None = None):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if not dist.is_initialized():
            dist.init_process_group(backend=backend or "nccl", rank=rank, world_size=world)
    return rank, local, world


def barrier(world: int, device=None):
    if world > 1:
        import torch.distributed as dist
        if device is not None and dist.get_backend() == "nccl":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def max_over_ranks(value: float, world: int, device=None) -> float:
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if (device is not None and dist.get_backend() == "nccl") else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rtfx(audio_seconds_per_rank_step: float, steps: int, ms_local: float, world: int, device=None):
    """Whole-job RTFx from per-rank device time: every rank decodes its own replica."""
    ms = max_over_ranks(ms_local, world, device)
    total_audio = audio_seconds_per_rank_step * steps * world
    return total_audio / (ms * 1e-3), ms / steps


# ---------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample of the workload
# ---------------------------------------------------------------------------
def oracle_sample(cfg, lens, W, seconds_target: float, cores: int):
    """The bounded sample both CPU legs time: the first k utterances, each cut to its first F frames.

    The oracle runs one thread per utterance (OpenMP over utterances only), so k = min(cores, B) keeps every core busy
    and the run lasts as long as its costliest utterance: F is chosen so that this is about `seconds_target` at a rough
    0.5e9 fp64 multiply-adds per second and core.  Cost per frame on this generator: about 2.8 tokens (one decoder update
    and one more window each) plus one window, a window being up to min(W, frames left) joint rows.
    """
    k = max(1, min(cores, len(lens)))
    rows_per_frame = (2.8 + 1.0) * min(W, 4)            # jumps are short on this data: windows overlap heavily
    lstm = sum(((cfg.E if l == 0 else cfg.P) + cfg.P) * 4 * cfg.P for l in range(cfg.L)) + cfg.P * cfg.H
    macs_per_frame = cfg.D * cfg.H + rows_per_frame * cfg.H * (cfg.V + 1) + 2.8 * lstm
    frames = int(max(8, seconds_target * 0.5e9 / macs_per_frame))
    return k, frames


def run_cpu_baseline(cfg, weights, enc, lens, W, seconds_target=15.0):
    import oracle
    cores = os.cpu_count() or 1
    k, frames = oracle_sample(cfg, lens, W, seconds_target, cores)
    om = oracle.Model(weights)
    sub_lens = np.minimum(lens[:k], frames).astype(np.int32)
    sub = np.ascontiguousarray(enc[:k, : int(sub_lens.max())])
    t0 = time.perf_counter()
    _, _, on, st = oracle.decode_batch(om, sub, sub_lens, W=W, S=cfg.S)
    dt = time.perf_counter() - t0
    audio = float(sub_lens.sum()) * FRAME_SECONDS
    return dict(value=audio / dt, unit="audio-s/s", cores=min(cores, k), kind="oracle",
                sample=f"first {k} of {cfg.B} utterances, each cut to its first {frames} frames ({int(sub_lens.sum())} frames in all), "
                       f"W={W}, one run, {dt:.1f} s",
                seconds=dt, steps=st["steps"])


def set_loop_mode(pkg, mode):
    if mode == "barriers":
        pkg.wind_set_loop_options(resident=True, dataflow=0)
    elif mode == "counters":
        pkg.wind_set_loop_options(resident=True, dataflow=1)
    elif mode == "streaming":
        pkg.wind_set_loop_options(resident=False)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_large_b128")
    ap.add_argument("--window", type=int, default=0, help="override the workload's window (0 = its default)")
    ap.add_argument("--kernels", type=int, default=0, help="0 auto, 1 plain-ALU kernels, 2 tensor-core kernels")
    ap.add_argument("--batch", type=int, default=0, help="override the number of utterances (profiling captures of a small case)")
    ap.add_argument("--len-lo", type=int, default=0, help="override the shortest utterance length, frames")
    ap.add_argument("--len-hi", type=int, default=0, help="override the longest utterance length, frames")
    ap.add_argument("--loop-mode", default="auto", choices=["auto", "barriers", "counters", "streaming"],
                    help="tensor-core loop: the planner's choice, or resident weights with grid barriers / with arrival counters, or streamed weights")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the W=1 comparison, e2e and per-kernel timing legs")
    ap.add_argument("--op", default="decode", choices=["decode", "first_output", "window_greedy", "dataset", "beam", "joint", "schedule"],
                    help="first_output: time wind_window_first_output (Eq. 1 on one window per utterance) instead of the decode; "
                         "window_greedy: time wind_decode_window_greedy on the whole workload; dataset: 4 x B utterances in "
                         "arrival-order batches against length-aware batches; beam: wind_beam_search on one utterance, beams 2..4")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    import wind_synth as ws
    cfg = ws.CONFIGS[args.workload]
    if args.batch or args.len_lo or args.len_hi:
        cfg = ws.small_variant(cfg, args.batch or cfg.B, args.len_lo or cfg.len_lo, args.len_hi or cfg.len_hi)
    W = args.window or cfg.W

    if args.impl == "reference":
        return reference_arm(args, cfg, W)
    if args.op == "first_output":
        return first_output_op(args, cfg, W)
    if args.op == "window_greedy":
        return window_greedy_op(args, cfg, W)
    if args.op == "dataset":
        return dataset_op(args, cfg, W)
    if args.op == "beam":
        return beam_op(args, cfg, W)
    if args.op == "joint":
        return joint_op(args, cfg, W)
    if args.op == "schedule":
        return schedule_op(args, cfg, W)

    import torch
    import paper_2505_13765_b200 as pkg

    rank, local, world = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    pkg.load_library()
    pkg.wind_set_kernels(args.kernels)
    set_loop_mode(pkg, args.loop_mode)
    peaks = load_peaks()

    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights, device=dev)
    B, T, D = enc_np.shape
    max_out = T * cfg.S
    enc_h = torch.from_numpy(enc_np).to(model.torch_dtype).pin_memory()
    len_h = torch.from_numpy(lens_np).pin_memory()
    enc_d = enc_h.to(dev)
    len_d = len_h.to(dev)
    tok_d = torch.full((B, max_out), -1, dtype=torch.int32, device=dev)
    frm_d = torch.full((B, max_out), -1, dtype=torch.int32, device=dev)
    ol_d = torch.zeros(B, dtype=torch.int32, device=dev)
    wsb = pkg.alloc_workspace(model, B, T, max(W, 1), host_staging_max_out=max_out)
    stream = torch.cuda.current_stream()
    audio_s = float(lens_np.sum()) * FRAME_SECONDS

    def step(window=W):
        pkg.wind_decode_greedy(model, enc_d, len_d, window, cfg.S, tok_d, frm_d, ol_d, wsb, stream=stream)

    def timed(fn, k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(world, dev)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(k):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        barrier(world, dev)
        return e0.elapsed_time(e1)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid)
    sampler.start()
    ms_local = timed(step, args.steps)
    clocks = sampler.stop()
    stats = pkg.wind_read_stats(wsb, stream)
    value, ms_per_step = aggregate_rtfx(audio_s, args.steps, ms_local, world, dev)
    launches = (stats["launches_setup"] + stats["steps"] * stats["launches_per_step"]) * args.steps
    tokens = stats["tokens"]

    out = {
        "metric": "greedy WIND RTFx (audio-s/s at 80 ms/frame)", "value": value, "unit": "audio-s/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "frames": int(lens_np.sum()), "T_max": int(lens_np.max()), "W": W,
                   "max_symbols": cfg.S, "D": cfg.D, "E": cfg.E, "P": cfg.P, "L": cfg.L, "H": cfg.H, "V": cfg.V,
                   "l2": "inputs larger than L2 (enc and enc_proj are each > 126 MB)",
                   "multi_gpu": "replicas only (no exchange step in the path)"},
        "frames_per_s": float(lens_np.sum()) * args.steps * world / (ms_per_step * args.steps * 1e-3),
        "loop_steps": stats["steps"], "us_per_loop_step": ms_per_step * 1e3 / max(1, stats["steps"]),
        "tokens": tokens, "tokens_per_frame": tokens / max(1, stats["frames"]),
        "launches_per_token": (stats["launches_setup"] + stats["steps"] * stats["launches_per_step"]) / max(1, tokens),
        "jump_hist": stats["jump_hist"][: W + 1], "kernels": {1: "simt", 2: "tensor"}.get(stats["kernels"], "?"),
        "gpu_launches": launches, "clocks": clocks,
    }

    if rank == 0 and not args.no_extras:
        # same library at W = 1 (the sequential baseline)
        if W != 1:
            for _ in range(2):
                step(1)
            k1 = max(1, min(args.steps, 3))
            ms1 = timed(lambda: step(1), k1) if world == 1 else None
            if ms1 is not None:
                st1 = pkg.wind_read_stats(wsb, stream)
                out["w1"] = {"value": audio_s * k1 / (ms1 * 1e-3), "ms_per_step": ms1 / k1, "loop_steps": st1["steps"]}
                out["speedup_vs_w1"] = (ms1 / k1) / ms_per_step
        # end to end through the host-buffer entry point: H2D of enc and lengths, D2H of the outputs, every step
        if world == 1:
            tok_h = torch.empty((B, max_out), dtype=torch.int32).pin_memory()
            frm_h = torch.empty((B, max_out), dtype=torch.int32).pin_memory()
            ol_h = torch.empty(B, dtype=torch.int32).pin_memory()

            def step_host():
                pkg.wind_decode_greedy_host(model, enc_h, len_h, W, cfg.S, tok_h, frm_h, ol_h, wsb, stream=stream)

            step_host()
            ke = max(1, min(args.steps, 3))
            ms_e = timed(step_host, ke)
            # bytes that cross the bus: the valid frames and the lengths in, the lengths and the token / frame columns up
            # to the longest transcript out
            longest = int(ol_h.max())
            out["e2e"] = {"value": audio_s * ke / (ms_e * 1e-3), "unit": "audio-s/s",
                          "h2d_bytes_per_step": int(int(lens_np.sum()) * D * enc_h.element_size() + len_h.numel() * 4),
                          "d2h_bytes_per_step": int((2 * B * longest + ol_h.numel()) * 4)}
    elif world > 1:
        # every rank must take part in the same collectives: none are issued in the extras
        pass

    if rank == 0:
        out["roofline"] = roofline(pkg, model, cfg, W, enc_d, len_d, tok_d, frm_d, ol_d, wsb, stream, stats, peaks, lens_np) \
            if (world == 1 and not args.no_extras) else None
        if not args.no_cpu_baseline and world == 1:
            cb = run_cpu_baseline(cfg, weights, enc_np, lens_np, W)
            out["cpu_baseline"] = cb
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def joint_standalone(pkg, model, cfg, W, peaks, iters=1000):
    """The loop kernel's joint phase by itself: `iters` passes back to back inside one launch, on fixed activations of
    all B * W window rows (wind_bench_joint), timed with CUDA events.  Algorithmic flop: 2 H (V+1) per window row;
    issued: what the tiles cover (vocabulary padded to 128, rows to the row-group size)."""
    import torch
    wsb = pkg.alloc_workspace(model, cfg.B, 1, W)
    r = pkg.wind_bench_joint(model, cfg.B, W, iters, wsb, stream=torch.cuda.current_stream())
    s_per_iter = r["ms"] * 1e-3 / r["iters"]
    alg = 2.0 * cfg.H * (cfg.V + 1) * r["rows"] / s_per_iter / 1e12
    issued = 2.0 * cfg.H * r["labels_issued"] * r["rows_issued"] / s_per_iter / 1e12
    peak = peaks["bf16_tflops_sustained"]
    return {"us_per_pass": s_per_iter * 1e6, "passes": r["iters"], "rows": r["rows"], "rows_issued": r["rows_issued"],
            "labels_issued": r["labels_issued"], "ctas": r["ctas"], "kernel": "resident weights" if r["resident"] else "streamed weights",
            "achieved": alg, "issued": issued, "frac": alg / peak, "issued_frac": issued / peak, "unit": "TFLOP/s", "peak": peak,
            "peak_source": peaks["source"] + " sustained bf16"}


def measured_traffic(cfg, W, frames):
    """DRAM bytes of one launch of the loop kernel, from the ncu counters of a small capture of the same shapes
    (the package's measured_traffic.json: bytes that do not grow with the workload, and bytes per encoder frame),
    scaled by the frame count.  None when the shapes have no capture."""
    path = os.path.join(ROOT, "paper_2505_13765_b200", "measured_traffic.json")
    if not os.path.exists(path):
        return None, None
    with open(path) as f:
        table = json.load(f)
    ent = table.get(f"{cfg.name}:W{W}")
    if not ent:
        return None, None
    return ent["fixed_bytes"] + ent["bytes_per_frame"] * frames, ent["source"]


def roofline(pkg, model, cfg, W, enc_d, len_d, tok_d, frm_d, ol_d, wsb, stream, stats, peaks, lens_np):
    """Roofline entry for the dominant kernel.

    Tensor-core path: the whole decoding loop is ONE persistent kernel launch per decode, so it is the
    dominant kernel.  Its algorithmic work per launch is what the method must compute, nothing else:
    2 * H * (V+1) flop per window row evaluated for a decision (rows of finished utterances, rows past an
    utterance's end and tile padding do not count), plus, per decoder update (one start-of-sequence
    update per utterance and one per emitted token), the LSTM stack's sum_l 2 * (in_l + P) * 4P flop and the
    projection's 2 * P * H flop.  The duration is the time between two CUDA events recorded on the stream
    around that launch by the library's timing entry point (one full decode of the workload).  The joint
    phase's share is reported beside it: its duration is the loop duration times the fraction of SM cycles
    the kernel's first CTA spent in that phase (grid-barrier waits included).
    Plain-ALU path: the joint kernel, timed per launch by CUDA events.
    """
    res = pkg.wind_profile_decode(model, enc_d, len_d, W, cfg.S, tok_d, frm_d, ol_d, wsb, stream=stream)
    peak = peaks["bf16_tflops_sustained"]
    joint_flop = 2.0 * cfg.H * (cfg.V + 1) * stats["joint_rows"]
    per_kernel = {k: res[k] for k in res if k.endswith("_ms")}
    frames = float(lens_np.sum())
    enc_flop = 2.0 * cfg.D * cfg.H * frames
    enc_bytes = frames * (cfg.D + cfg.H) * 2.0
    enc = None
    if res["enc_proj_ms"] > 0:
        es = res["enc_proj_ms"] * 1e-3
        enc = {"tflops": enc_flop / es / 1e12, "frac_tensor": enc_flop / es / 1e12 / peaks["bf16_tflops"],
               "gbs": enc_bytes / es / 1e9, "frac_hbm": enc_bytes / es / 1e9 / peaks["hbm_gbs"], "ms": res["enc_proj_ms"]}
    if res["loop_ms"] > 0:
        updates = stats["tokens"] + int((lens_np >= 0).sum())
        lstm_flop = sum(2.0 * ((cfg.E if l == 0 else cfg.P) + cfg.P) * 4 * cfg.P for l in range(cfg.L)) + 2.0 * cfg.P * cfg.H
        flop = joint_flop + updates * lstm_flop
        dur_s = res["loop_ms"] * 1e-3
        achieved = flop / dur_s / 1e12
        js = res["joint_ms"] * 1e-3
        dense = 2.0 * cfg.H * (cfg.V + 1) * cfg.B * W * stats["steps"]
        # DRAM bytes per launch: ncu counters of a small capture of the same shapes, scaled by the frame count (the
        # enc_proj rows, each read once, grow with the workload; weights, gate-table rows and outputs do not)
        traffic, traffic_source = measured_traffic(cfg, W, frames)
        standalone = joint_standalone(pkg, model, cfg, W, peaks)
        return {"kernel": "decoding loop (one persistent launch: joint, decoder-update and projection phases)",
                "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": peaks["source"] + " sustained bf16", "traffic": traffic, "traffic_source": traffic_source,
                "launch_ms": res["loop_ms"], "algorithmic_gflop_per_launch": flop / 1e9,
                "joint_phase": {"us_per_step": js * 1e6 / max(1, stats["steps"]), "achieved": joint_flop / js / 1e12,
                                "frac": joint_flop / js / 1e12 / peak, "dense_issued_frac": dense / js / 1e12 / peak,
                                "rows_per_step": stats["joint_rows"] / max(1, stats["steps"])},
                "joint_standalone": standalone,
                "phase_us_per_step": {"joint": res["joint_ms"] * 1e3 / max(1, stats["steps"]),
                                      "decoder_update": res["lstm_ms"] * 1e3 / max(1, stats["steps"]),
                                      "projection": res["proj_ms"] * 1e3 / max(1, stats["steps"])},
                "enc_proj": enc, "per_kernel_ms": per_kernel}
    rows_per_launch = stats["joint_rows"] / max(1, stats["steps"])
    dur_s = res["joint_ms"] * 1e-3 / max(1, res["joint_launches"])
    achieved = 2.0 * cfg.H * (cfg.V + 1) * rows_per_launch / dur_s / 1e12
    return {"kernel": "windowed joint (plain-ALU kernel)", "bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
            "frac": achieved / peak, "peak_source": peaks["source"] + " sustained bf16", "traffic": None,
            "avg_launch_us": dur_s * 1e6, "rows_per_launch": rows_per_launch, "enc_proj": enc, "per_kernel_ms": per_kernel}


def first_output_op(args, cfg, W):
    """Secondary measurement (one JSON line of its own): Eq. (1) for one window per utterance.

    The call runs the projection, the decoder on an empty prefix and the joint's store epilogue, then the in-place
    Eq. (1) pass with the 4 best (label, offset) pairs.  `value` is windows per second for the whole call; the
    in-place kernel's own share is what `ncu -k regex:first_output` shows for the same command.
    """
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights, device=dev)
    B, T, _ = enc_np.shape
    NV, K = cfg.V + 1, 4
    enc_d = pkg.to_device_enc(model, enc_np)
    len_d = torch.from_numpy(lens_np).to(dev)
    rng = np.random.default_rng(7)
    t0 = torch.from_numpy(np.array([rng.integers(0, max(1, l - W)) for l in lens_np], np.int32)).to(dev)
    plen = torch.zeros(B, dtype=torch.int32, device=dev)
    logp = torch.empty((B, W, NV), dtype=torch.float32, device=dev)
    tl = torch.empty((B, K), dtype=torch.int32, device=dev)
    tj = torch.empty((B, K), dtype=torch.int32, device=dev)
    tv = torch.empty((B, K), dtype=torch.float32, device=dev)
    wsb = pkg.alloc_workspace(model, B, T, W)
    stream = torch.cuda.current_stream()

    def step():
        pkg.wind_window_first_output(model, enc_d, len_d, W, None, plen, t0, logp, wsb, K=K, top_label=tl, top_jump=tj,
                                     top_logp=tv, stream=stream)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    total = float(np.exp(logp.double().cpu().numpy()).sum())
    print(json.dumps({
        "metric": "windows/s, wind_window_first_output (projection + decoder start + joint store + Eq. 1 pass)", "op": "first_output",
        "value": B / (ms * 1e-3), "unit": "windows/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": B, "W": W, "K": K, "V": cfg.V},
        "eq1_pass_algorithmic_bytes": 2 * B * W * NV * 4, "sum_of_probabilities_per_window": total / B,
    }))


def window_greedy_op(args, cfg, W):
    """Secondary measurement (one JSON line of its own): window-based greedy decoding of the whole workload.

    Same inputs, same timing as the main line, through wind_decode_window_greedy; beside it the same library's
    Algorithm 2 decode at the same W (time, lock steps, tokens) and the oracle's window-based decoder on a bounded
    sample of the workload.
    """
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    pkg.wind_set_kernels(args.kernels)
    set_loop_mode(pkg, args.loop_mode)
    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(weights, device=dev)
    B, T, _ = enc_np.shape
    max_out = T * cfg.S
    enc_d = pkg.to_device_enc(model, enc_np)
    len_d = torch.from_numpy(lens_np).to(dev)
    tok_d = torch.full((B, max_out), -1, dtype=torch.int32, device=dev)
    frm_d = torch.full((B, max_out), -1, dtype=torch.int32, device=dev)
    ol_d = torch.zeros(B, dtype=torch.int32, device=dev)
    wsb = pkg.alloc_workspace(model, B, T, W)
    stream = torch.cuda.current_stream()
    audio_s = float(lens_np.sum()) * FRAME_SECONDS

    def run(call, k):
        for _ in range(max(3, args.warmup)):
            call(model, enc_d, len_d, W, cfg.S, tok_d, frm_d, ol_d, wsb, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(k):
            call(model, enc_d, len_d, W, cfg.S, tok_d, frm_d, ol_d, wsb, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / k, pkg.wind_read_stats(wsb, stream)

    ms2, st2 = run(pkg.wind_decode_greedy, max(1, min(args.steps, 3)))
    ms, st = run(pkg.wind_decode_window_greedy, args.steps)
    cb = None
    if not args.no_cpu_baseline:
        import oracle
        cores = os.cpu_count() or 1
        # up to S steps of W rows per frame on a model whose distributions are flat (see the note in the JSON line)
        budget_frames = 15.0 * 0.6e9 * cores / (cfg.H * (cfg.V + 1) * float(cfg.S * W))
        k = max(1, int(np.searchsorted(np.cumsum(lens_np), budget_frames)))
        t0 = time.perf_counter()
        oracle.decode_window_greedy_batch(oracle.Model(weights), np.ascontiguousarray(enc_np[:k]), lens_np[:k], W=W, S=cfg.S)
        dt = time.perf_counter() - t0
        cb = dict(value=float(lens_np[:k].sum()) * FRAME_SECONDS / dt, unit="audio-s/s", cores=cores, kind="oracle",
                  sample=f"first {k} of {cfg.B} utterances ({int(lens_np[:k].sum())} frames), W={W}, one run, {dt:.1f} s")
    print(json.dumps({
        "metric": "window-based greedy RTFx (audio-s/s at 80 ms/frame)", "op": "window_greedy",
        "value": audio_s / (ms * 1e-3), "unit": "audio-s/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": B, "frames": int(lens_np.sum()), "W": W, "max_symbols": cfg.S},
        "loop_steps": st["steps"], "us_per_loop_step": ms * 1e3 / max(1, st["steps"]), "tokens": st["tokens"],
        "jump_hist": st["jump_hist"][: W + 1], "kernels": {1: "simt", 2: "tensor"}.get(st["kernels"], "?"),
        "gpu_launches": (st["launches_setup"] + st["steps"] * st["launches_per_step"]) * args.steps,
        "algorithm2_same_w": {"ms_per_step": ms2, "loop_steps": st2["steps"], "tokens": st2["tokens"],
                              "us_per_loop_step": ms2 * 1e3 / max(1, st2["steps"])},
        "cpu_baseline": cb,
        "note": "random-weight models give flat label distributions, for which the best pair of Eq. (1) is almost always a "
                "label on the window's first row: the variant then emits max_symbols tokens per frame, its worst case for "
                "the number of steps; the per-step cost is what this line measures",
    }))


def dataset_op(args, cfg, W):
    """Secondary measurement (one JSON line of its own): a set of 4 x B utterances decoded batch by batch.

    The same utterances are packed into batches of B twice: in arrival order and by the library's length-aware plan
    (wind_plan_batches).  Both packings are resident on the device before the clock starts; the timed region is the
    decodes of all batches, back to back.  `value` is the planned packing's whole-set RTFx.  `refilled_rows`: the same
    set in ONE call on B batch rows that take the next utterance when theirs is finished (wind_decode_greedy_refill), in
    arrival order and longest first.
    """
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    from dataclasses import replace
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    pkg.wind_set_kernels(args.kernels)
    set_loop_mode(pkg, args.loop_mode)
    B = cfg.B
    big = replace(cfg, B=4 * B)
    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(big, pad="zero")
    model = pkg.WindModel(weights, device=dev)
    N = enc_np.shape[0]
    stream = torch.cuda.current_stream()
    order, batch_T = pkg.wind_plan_batches(lens_np, B)

    def pack(idx_order):
        batches = []
        for k in range(0, N, B):
            idx = idx_order[k: k + B]
            T = int(lens_np[idx].max())
            enc_d = pkg.to_device_enc(model, np.ascontiguousarray(enc_np[idx, :T]))
            len_d = torch.from_numpy(np.ascontiguousarray(lens_np[idx])).to(dev)
            max_out = T * cfg.S
            tok = torch.full((len(idx), max_out), -1, dtype=torch.int32, device=dev)
            batches.append((enc_d, len_d, tok, tok.clone(), torch.zeros(len(idx), dtype=torch.int32, device=dev),
                            pkg.alloc_workspace(model, len(idx), T, W)))
        return batches

    def run(batches, k):
        def once():
            steps = 0
            for enc_d, len_d, tok, frm, ol, wsb in batches:
                pkg.wind_decode_greedy(model, enc_d, len_d, W, cfg.S, tok, frm, ol, wsb, stream=stream)
                steps += pkg.wind_read_stats(wsb, stream)["steps"]
            return steps
        for _ in range(max(3, args.warmup)):
            steps = once()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(k):
            once()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / k, steps

    def run_refill(idx_order, k):
        # all utterances resident at the set's T, decoded on B batch rows that are refilled inside the loop
        T = int(lens_np.max())
        enc_d = pkg.to_device_enc(model, np.ascontiguousarray(enc_np[idx_order, :T]))
        len_d = torch.from_numpy(np.ascontiguousarray(lens_np[idx_order])).to(dev)
        max_out = T * cfg.S
        tok = torch.full((N, max_out), -1, dtype=torch.int32, device=dev)
        frm = tok.clone()
        ol = torch.zeros(N, dtype=torch.int32, device=dev)
        wsb = torch.empty(pkg.wind_refill_workspace_bytes(model, N, T, B, W) + 256, dtype=torch.uint8, device=dev)
        steps = 0
        for _ in range(max(3, args.warmup)):
            pkg.wind_decode_greedy_refill(model, enc_d, len_d, B, W, cfg.S, tok, frm, ol, wsb, stream=stream)
            steps = pkg.wind_read_stats(wsb, stream)["steps"]
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(k):
            pkg.wind_decode_greedy_refill(model, enc_d, len_d, B, W, cfg.S, tok, frm, ol, wsb, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / k, steps

    ms_a, steps_a = run(pack(np.arange(N)), args.steps)
    torch.cuda.empty_cache()
    ms_p, steps_p = run(pack(order), args.steps)
    torch.cuda.empty_cache()
    refill = {}
    try:
        for name, idx_order in (("arrival_order", np.arange(N)), ("longest_first", np.asarray(order))):
            ms_r, steps_r = run_refill(idx_order, args.steps)
            torch.cuda.empty_cache()
            refill[name] = {"ms": ms_r, "lock_steps": steps_r, "value": float(lens_np.sum()) * FRAME_SECONDS / (ms_r * 1e-3)}
    except pkg.WindError as e:      # shapes outside the tensor-core kernel set have no refilled rows
        refill = {"unavailable": str(e)}
    audio_s = float(lens_np.sum()) * FRAME_SECONDS
    print(json.dumps({
        "metric": "greedy WIND RTFx of a set of utterances (audio-s/s at 80 ms/frame)", "op": "dataset",
        "value": audio_s / (ms_p * 1e-3), "unit": "audio-s/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_p, "higher_is_better": True, "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "utterances": N, "B": B, "frames": int(lens_np.sum()), "W": W},
        "length_aware": {"ms": ms_p, "lock_steps": steps_p, "batch_T": [int(t) for t in batch_T]},
        "arrival_order": {"ms": ms_a, "lock_steps": steps_a, "value": audio_s / (ms_a * 1e-3)},
        "speedup_vs_arrival_order": ms_a / ms_p, "refilled_rows": refill,
        "gpu_launches": 4 * len(batch_T) * args.steps,
    }))


def beam_op(args, cfg, W):
    """Secondary measurement (one JSON line per beam width): WIND beam search (Algorithm 3) on the first utterance of
    the workload, beams 2, 3 and 4, through wind_beam_search (encoder frames resident on the device; the call's own
    host-side bookkeeping and its one synchronisation per iteration are inside the timed region, which is wall clock
    around the call: the search is driven from the host).  Beside it the oracle on the utterance's first frames."""
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    b = int(np.argmax(lens_np))
    T = int(lens_np[b])
    enc = np.ascontiguousarray(enc_np[b, :T])
    model = pkg.WindModel(weights, device=dev)
    for K, prefix in ((2, False), (3, False), (4, False), (4, True)):
        for _ in range(2):
            pkg.wind_beam_search(model, enc, W, K, cfg.S, max_hyps=8, prefix_search=prefix)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            hyps, steps, st = pkg.wind_beam_search(model, enc, W, K, cfg.S, max_hyps=8, prefix_search=prefix)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.steps
        cb = None
        if not args.no_cpu_baseline:
            import oracle
            Tc = min(T, 24)
            t1 = time.perf_counter()
            _, _, osteps = oracle.beam_search(oracle.Model(weights), enc[:Tc], Tc, W, K, cfg.S, prefix_search=prefix)
            od = time.perf_counter() - t1
            cb = dict(value=Tc * FRAME_SECONDS / od, unit="audio-s/s", cores=1, kind="oracle",
                      sample=f"first {Tc} frames of the utterance, {osteps} iterations, one run, {od:.1f} s")
        print(json.dumps({
            "metric": "WIND beam search RTFx, one utterance (audio-s/s at 80 ms/frame)", "op": "beam", "value": T * FRAME_SECONDS / dt,
            "unit": "audio-s/s", "n_gpus": 1, "steps": args.steps, "warmup": 2, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "utterance": b, "frames": T, "W": W, "K": K, "max_symbols": cfg.S, "prefix_search": prefix},
            "iterations": steps, "us_per_iteration": dt * 1e6 / max(1, steps), "best_tokens": int(len(hyps[0][0])),
            "best_score": hyps[0][2], "final_hypotheses": len(hyps), "cpu_baseline": cb,
        }))


def joint_op(args, cfg, W):
    """Secondary measurement (one JSON line of its own): the joint phase alone, back to back (see joint_standalone)."""
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    peaks = load_peaks()
    model = pkg.WindModel(ws.make_model(cfg), device=dev)
    res = [joint_standalone(pkg, model, cfg, W, peaks, iters=1000) for _ in range(max(1, args.steps))]
    best = min(res, key=lambda r: r["us_per_pass"])
    print(json.dumps({"metric": "joint phase alone, TFLOP/s of algorithmic work (2 H (V+1) per window row)", "value": best["achieved"],
                      "unit": "TFLOP/s", "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": cfg.name, "B": cfg.B, "W": W, "H": cfg.H, "V": cfg.V}, "joint_standalone": best}))


def step_kinds(lens, tok_len, frames, W, S):
    """Per utterance the kinds of its Algorithm 2 iterations, rebuilt from its transcript: True = the window held a non-blank
    frame (one emission, one decoder update), False = every row blank (t += n)."""
    out = []
    for b in range(len(lens)):
        f, n_tok, length = frames[b], int(tok_len[b]), int(lens[b])
        t, k, cnt, kinds = 0, 0, 0, []
        while t < length:
            n = min(W, length - t)
            if k < n_tok and f[k] < t + n:
                cnt = (cnt if f[k] == t else 0) + 1
                t = int(f[k])
                k += 1
                if cnt == S:
                    t, cnt = t + 1, 0
                kinds.append(True)
            else:
                t, cnt = t + n, 0
                kinds.append(False)
        out.append(np.array(kinds, dtype=bool))
    return out


def schedule_counts(kinds):
    """Passes of the two batched schedules over the same per-utterance iterations.

    Lock step (what the library runs): every pass is one joint evaluation, one masked decoder update and one projection for
    the whole batch; an utterance takes one of its iterations per pass, so the passes are the longest utterance's.
    Label looping proper: an outer iteration repeats the joint (with a fresh window, hence fresh activations) for the
    utterances whose window was all blank until every utterance still decoding holds a non-blank frame, then runs ONE
    decoder update and projection for all of them."""
    lock = max((len(k) for k in kinds), default=0)
    pos = [0] * len(kinds)
    joint_passes = updates = 0
    while True:
        inner, any_emit = 0, False
        for u, k in enumerate(kinds):
            p = pos[u]
            if p >= len(k):
                continue
            nxt = np.flatnonzero(k[p:])
            blanks = int(nxt[0]) if len(nxt) else len(k) - p        # all-blank windows before the next emission
            inner = max(inner, blanks + (1 if len(nxt) else 0))
            any_emit = any_emit or len(nxt) > 0
            pos[u] = p + blanks + (1 if len(nxt) else 0)
        if inner == 0:
            break
        joint_passes += inner
        updates += 1 if any_emit else 0
    return {"lock_step_passes": lock, "label_looping_joint_passes": joint_passes, "label_looping_decoder_updates": updates}


def schedule_op(args, cfg, W):
    """Secondary measurement (one JSON line of its own): how many batched passes the label-looping schedule proper would
    need on this workload against the lock-step schedule the library runs, counted on the transcripts the GPU produced, and
    priced with the per-phase times of the same decode (wind_profile_decode)."""
    import torch
    import wind_synth as ws
    import paper_2505_13765_b200 as pkg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pkg.load_library()
    pkg.wind_set_kernels(args.kernels)
    set_loop_mode(pkg, args.loop_mode)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    model = pkg.WindModel(ws.make_model(cfg), device=dev)
    enc_d = pkg.to_device_enc(model, enc_np)
    len_d = torch.from_numpy(lens_np).to(dev)
    B, T, _ = enc_np.shape
    tok = torch.full((B, T * cfg.S), -1, dtype=torch.int32, device=dev)
    frm, ol = tok.clone(), torch.zeros(B, dtype=torch.int32, device=dev)
    wsb = pkg.alloc_workspace(model, B, T, W)
    stream = torch.cuda.current_stream()
    for _ in range(max(3, args.warmup)):
        pkg.wind_decode_greedy(model, enc_d, len_d, W, cfg.S, tok, frm, ol, wsb, stream=stream)
    stats = pkg.wind_read_stats(wsb, stream)
    prof = pkg.wind_profile_decode(model, enc_d, len_d, W, cfg.S, tok, frm, ol, wsb, stream=stream)
    counts = schedule_counts(step_kinds(lens_np, ol.cpu().numpy(), frm.cpu().numpy(), W, cfg.S))
    assert counts["lock_step_passes"] == stats["steps"], (counts, stats["steps"])
    n = stats["steps"]
    j, l, p = prof["joint_ms"] / n, prof["lstm_ms"] / n, prof["proj_ms"] / n      # ms per pass of each phase
    # label looping proper: every joint pass needs its activations rebuilt (the projection phase's epilogue; priced as a
    # whole projection phase: the phase is bound by its barrier and round trips, not by the GEMM), every update a decoder phase
    est = counts["label_looping_joint_passes"] * (j + p) + counts["label_looping_decoder_updates"] * l
    print(json.dumps({"metric": "batched passes per decode: lock step against label looping proper", "op": "schedule",
                      "value": counts["label_looping_joint_passes"] / max(1, n), "unit": "joint passes relative to lock steps",
                      "higher_is_better": False, "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
                      "config": {"workload": cfg.name, "B": B, "W": W}, **counts,
                      "phase_ms_per_pass": {"joint": j, "decoder_update": l, "projection": p},
                      "lock_step_ms": n * (j + l + p), "label_looping_ms_estimate": est}))


def reference_arm(args, cfg, W):
    """The oracle as it stands, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import wind_synth as ws
    weights = ws.make_model(cfg)
    enc_np, lens_np = ws.make_enc(cfg, pad="zero")
    per_step_target = max(2.0, min(15.0, 120.0 / max(1, args.steps + args.warmup)))   # the whole run within a few minutes
    for _ in range(args.warmup):
        run_cpu_baseline(cfg, weights, enc_np, lens_np, W, per_step_target)
    vals, secs = [], []
    for _ in range(max(1, args.steps)):
        cb = run_cpu_baseline(cfg, weights, enc_np, lens_np, W, per_step_target)
        vals.append(cb["value"]); secs.append(cb["seconds"])
    value = float(np.sum([v * s for v, s in zip(vals, secs)]) / np.sum(secs))
    cb["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": "greedy WIND RTFx (audio-s/s at 80 ms/frame)", "value": value, "unit": "audio-s/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(secs)) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "W": W, "sample": cb["sample"]},
        "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": value, "unit": "audio-s/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    main()
