#!/usr/bin/env python
"""Benchmark of the FFD sparse decode-attention step on B200.

One "step" = the whole hot path on one batch of synthetic input: re-quantize the tail block of every sequence
(cache append), pseudo-max, fused scan -> top-delta select -> exact attention over kept blocks, split combine.
Default workload at one GPU: the 128K mixed-entropy configuration (C3: batch 4, 32 query / 8 KV heads,
head_dim 128, context 131072, delta 6) that the headline metric is quoted on.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference          # the CPU oracle, as it stands, on a bounded sample

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_00097_b200.workloads import CONFIGS, make_workload

METRIC = "sparse_decode_attn_us_per_step"
UNIT = "us/step"
CODE_BYTES_PER_TILE = 2048 + 256          # packed 2-bit codes + fp16 scales of one (block, KV head)
KV_BYTES_PER_TILE = 2 * 64 * 128 * 2      # K tile + V tile of one kept (block, KV head)
# dram__bytes_read + dram__bytes_write of one fused-kernel launch divided by the launch's algorithmic bytes, from
# the ncu capture summarised in profiles/fused_sparse_kernel_C3_ctx32768.md (same kernel, same workload recipe at
# context 32768; traffic grows in proportion to the blocks processed): (308.47 + 5.65) MB / 308.28 MB.
NCU_TRAFFIC_RATIO = 1.018
KERNEL_EVENT_EVERY = 4      # steps between two steps that carry the CUDA-event pair around the fused kernel


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi; every sample is stamped on arrival so that the
    ones taken during the timed region can be told from the rest."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.samples = []      # (arrival time, sm MHz, max MHz, active reasons)

    def start(self, wait_first_sample: float = 5.0):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
            return
        t0 = time.perf_counter()
        while not self.samples and time.perf_counter() - t0 < wait_first_sample:
            time.sleep(0.01)

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm, mx = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            reasons = [n for n, v in zip(self.NAMES, parts[2:6]) if v.lower().startswith("active")]
            self.samples.append((time.perf_counter(), sm, mx, reasons))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [s for s in self.samples if t_begin <= s[0] <= t_end + 0.02]
        window = "timed region"
        if not inside:   # region shorter than the sampling period: fall back to everything seen under load
            inside, window = self.samples, "warm-up + timed region (timed region shorter than one sample)"
        reasons = sorted({r for s in inside for r in s[3]})
        return {"sm_mhz": statistics.median([s[1] for s in inside]) if inside else None,
                "sm_max_mhz": max([s[2] for s in inside]) if inside else None, "samples": len(inside),
                "window": window, "reasons": reasons}


def reduce_max_over_ranks(values, dist, device="cpu"):
    """Max over ranks of a list of floats (the only exchange of a multi-rank run: the path itself shards over
    (sequence, KV head) with no collective)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def union_kept_tiles(kept: np.ndarray, w) -> int:
    """(block, KV head) tiles whose K/V were read: a block is loaded when any query head of the group keeps it."""
    total = 0
    for b in range(w.B):
        nb = w.num_blocks(b)
        k = kept[b, :, :nb].reshape(w.Hkv, w.G, nb)
        total += int(k.any(axis=1).sum())
    return total


def algorithmic_bytes(w, kept_tiles: int, dense: bool = False) -> int:
    tiles = sum(w.num_blocks(b) for b in range(w.B)) * w.Hkv
    if dense:
        return tiles * KV_BYTES_PER_TILE
    return tiles * CODE_BYTES_PER_TILE + kept_tiles * KV_BYTES_PER_TILE


def cpu_baseline(w, delta, threads=None, seconds_target=15.0):
    """Time the oracle, as it stands, on a bounded sample of (sequence, head) rows of the same workload and scale
    to a whole step.  Reported context, not a target."""
    from oracle import ffd_oracle as O
    cores = threads or O.max_threads()
    O.set_threads(cores)
    # sample: one query head per KV-head kind (peaked / flat) per thread, so every core has work
    flat = set(w.flat_heads)
    kinds = {"peaked": [g for g in range(w.Hkv) if g not in flat], "flat": list(flat)}
    units = []
    for kind, gs in kinds.items():
        for i in range(cores):
            if gs:
                g = gs[i % len(gs)]
                units.append((i % w.B, g * w.G + (i // len(gs)) % w.G))
    units = sorted(set(units))
    # the oracle quantizer output is an input of the timed stage (quantization is the append path)
    t0 = time.perf_counter()
    codes, scales = O.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    t_quant = time.perf_counter() - t0
    t0 = time.perf_counter()
    O.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
             w.max_blocks, delta, units=units)
    t = time.perf_counter() - t0
    n_flat = sum(1 for (_, h) in units if (h // w.G) in flat)
    n_peak = len(units) - n_flat
    total_rows = w.B * w.Hq
    # the sample holds the two head kinds in the workload's own proportion, so one factor scales it to a step
    scale = total_rows / len(units)
    step_seconds = t * scale
    return {"value": step_seconds * 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(units)} of {total_rows} (sequence, query head) rows ({n_peak} peaked, {n_flat} flat), "
                      f"scan+select+attend in {t:.2f} s scaled by {scale:.1f}; full-cache quantizer {t_quant:.1f} s "
                      "not included"}


def run_reference(args, rank, world):
    """The reference arm of this build is the CPU oracle (there is no reference implementation to install)."""
    if rank != 0:
        return
    from oracle import ffd_oracle as O
    w = make_workload(args.workload, **workload_overrides(args))
    delta = args.delta if args.delta is not None else w.deltas[0]
    cores = O.max_threads()
    O.set_threads(cores)
    codes, scales = O.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    flat = set(w.flat_heads)
    units = []
    for i in range(cores):
        g = i % w.Hkv
        units.append((i % w.B, g * w.G + (i // w.Hkv) % w.G))
    units = sorted(set(units))
    scale = w.B * w.Hq / len(units)
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        O.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                 w.max_blocks, delta, units=units)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    us = statistics.mean(times) * scale * 1e6
    sample = (f"{len(units)} of {w.B * w.Hq} (sequence, query head) rows per step over all KV-head kinds, "
              f"time scaled by {scale:.1f}")
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, delta, args),
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_overrides(args):
    kw = {}
    if args.context:
        kw["N"] = args.context
    if args.batch:
        kw["B"] = args.batch
    return kw


def workload_config(w, delta, args):
    return {"workload": f"{w.name}: batch {w.B}, {w.Hq} query / {w.Hkv} KV heads, head_dim 128, "
                        f"context {int(w.seq_lens.max())}, 64-token blocks, delta {delta}",
            "seed": w.seed, "delta": delta, "block_tokens": 64, "quant_bits": 2,
            "l2": "L2 flushed before every step (256 MiB written, then 256 MiB of another buffer read so that the "
                  "flush's own write-back drains before the timed region); inputs also larger than L2",
            "step": "tail-block re-quantize + pseudo-max + fused scan/select/attend + combine",
            "kernel_events": f"every {KERNEL_EVENT_EVERY}th timed step carries the CUDA-event pair around the fused kernel "
                             "(roofline.kernel_us is their mean); see step_us_without_kernel_events",
            "aggregate": "value = max-over-ranks step time / n_gpus (each rank decodes its own batch)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=sorted(CONFIGS))
    ap.add_argument("--context", type=int, default=0, help="override the context length (smaller profiling case)")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--delta", type=float, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    from paper_2609_00097_b200 import ffd
    ffd.load_library()                      # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = make_workload(args.workload, **workload_overrides(args))
    delta = args.delta if args.delta is not None else w.deltas[0]
    cfg = ffd.Config(w.Hq, w.Hkv, out_dtype=1)
    dc = ffd.DeviceCache(w, cfg)
    dc.quantize()
    first_token = torch.from_numpy(np.maximum(w.seq_lens - 1, 0)).to("cuda")
    kept = torch.zeros(w.B, w.Hq, w.max_blocks, dtype=torch.uint8, device="cuda")
    dc.decode(delta, kept_mask=kept)
    assert ffd.ffd_read_device_status(dc.workspace) == 0
    kept_np = kept.cpu().numpy()
    kept_tiles = union_kept_tiles(kept_np, w)
    total_tiles = sum(w.num_blocks(b) for b in range(w.B)) * w.Hkv
    head_blocks = sum(w.num_blocks(b) for b in range(w.B)) * w.Hq
    kept_head_blocks = sum(int(kept_np[b, :, : w.num_blocks(b)].sum()) for b in range(w.B))
    sparse_bytes = algorithmic_bytes(w, kept_tiles)
    dense_bytes = algorithmic_bytes(w, 0, dense=True)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    drain = torch.zeros(32 << 20, dtype=torch.int64, device="cuda")      # 256 MiB, only ever read
    stream = torch.cuda.current_stream()
    k_start, k_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k_start.record(), k_stop.record()      # materialise the CUDA events before handing them to the library

    def step():
        dc.quantize(first_token=first_token)
        dc.decode(delta)

    def timed_loop(fn, n, profile_kernel, cold=True):
        """n steps, each bracketed by CUDA events on the launching stream, L2 flushed (untimed) before each."""
        total, kernel = [], []
        for i in range(n):
            if profile_kernel:
                # The event pair around the fused kernel sits between the step's kernels and costs their
                # programmatic-launch overlap (~10 us): it is recorded on every KERNEL_EVENT_EVERY-th step only.
                probe = i % KERNEL_EVENT_EVERY == 0
                ffd.ffd_profile_events(k_start if probe else None, k_stop if probe else None)
            if cold:
                flush.fill_(1)      # evicts every input line from L2 ...
                drain.sum()         # ... and this read sweep pushes the fill's dirty lines out to HBM, so that their
                                    # write-back (an artefact of the flush, not of the workload) ends before the timing starts
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            b.synchronize()
            total.append(a.elapsed_time(b) * 1e3)
            if profile_kernel and probe:
                kernel.append(k_start.elapsed_time(k_stop) * 1e3)
        return total, kernel

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    ffd.ffd_profile_events(k_start, k_stop)
    sampler = ClockSampler(local_rank)
    sampler.start()
    timed_loop(step, args.warmup, False)
    barrier()
    t_begin = time.perf_counter()
    step_us, kernel_us = timed_loop(step, args.steps, True)
    barrier()
    clocks = sampler.stop(t_begin, time.perf_counter())
    # the dense path of the same library, same protocol (context for the speedup figure)
    timed_loop(dc.dense, 3, False)
    dense_us, dense_kernel_us = timed_loop(dc.dense, min(max(5, args.steps // 2), 100), True)
    ffd.ffd_profile_events(None, None)
    # the same step without the event pair around the fused kernel (the records sit between the step's kernels and
    # cost their programmatic-launch overlap): what a caller who does not profile sees
    plain_us, _ = timed_loop(step, min(args.steps, 200), False)
    # the same without the flush (whatever of the previous step is still in L2 stays there) ...
    warm_us, _ = timed_loop(step, min(args.steps, 200), False, cold=False)
    # ... submitted as one CUDA graph (cold L2) ...
    graph_us = None
    try:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            step()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.synchronize()
        graph_us, _ = timed_loop(graph.replay, min(args.steps, 200), False)
    except Exception as exc:   # reported, not fatal: the graph number is an extra
        graph_us = None
        print(f"bench: CUDA graph capture failed: {exc}", file=sys.stderr)
    # ... and a pure-read calibration: a sum over 1 GiB (torch's reduction kernel), cold
    calib = torch.zeros(128 << 20, dtype=torch.int64, device="cuda")
    calib_us, _ = timed_loop(calib.sum, 13, False)
    read_gbs = calib.numel() * 8 / (statistics.median(calib_us[3:]) * 1e-6) / 1e9
    del calib

    # end to end through the public API with HOST buffers: q comes from pinned host memory every step and the
    # output goes back to the host; the KV cache itself is resident (it is a cache), as in a serving loop
    # (q and seq_lens travel as one pinned buffer into the one device allocation they share)
    in_host = dc.step_in.cpu().pin_memory()
    out_host = torch.empty(w.B, w.Hq, 128, dtype=torch.float32).pin_memory()

    def e2e_step():
        dc.step_in.copy_(in_host, non_blocking=True)
        step()
        out_host.copy_(dc.out, non_blocking=True)

    timed_loop(e2e_step, 3, False)
    e2e_us, _ = timed_loop(e2e_step, min(args.steps, 200), False)
    h2d = in_host.numel()
    d2h = out_host.numel() * 4

    # the same step on the 2 + 8 bit key format (kept blocks refined from 8-bit residuals instead of 16-bit keys):
    # tail re-quantize of thumbnails and residuals + pseudo-max + fused kernel + combine, same protocol.  Measured
    # last: it swaps the workspace for the larger one that format needs.
    dc.quantize_residual()

    def residual_step():
        dc.quantize_both(first_token=first_token)
        dc.decode_residual(delta)

    ffd.ffd_profile_events(k_start, k_stop)
    timed_loop(residual_step, 3, False)
    res_us, res_kernel_us = timed_loop(residual_step, min(max(5, args.steps // 2), 100), True)
    ffd.ffd_profile_events(None, None)
    res_bytes = total_tiles * CODE_BYTES_PER_TILE + kept_tiles * (KV_BYTES_PER_TILE // 2 + KV_BYTES_PER_TILE // 4)

    t_step = statistics.mean(step_us)
    t_e2e = statistics.mean(e2e_us)
    t_step, t_e2e = reduce_max_over_ranks([t_step, t_e2e], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    t_kernel = statistics.mean(kernel_us)
    achieved = sparse_bytes / (t_kernel * 1e-6) / 1e9
    t_dense = statistics.mean(dense_us)
    line = {
        "metric": METRIC, "value": t_step / world, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_step / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in / fp32 accumulate (fp16 x fp16 -> fp32 tensor-core scan)",
        "data": "synthetic", "config": workload_config(w, delta, args),
        "clocks": clocks,
        "e2e": {"value": t_e2e / world, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": 4 * args.steps,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (None if NCU_TRAFFIC_RATIO is None else sparse_bytes * NCU_TRAFFIC_RATIO),
                     "peak_source": f"{peak_kind} copy bandwidth (of {peak_kind})", "kernel": "fused_sparse_kernel",
                     "kernel_us": t_kernel, "algorithmic_bytes": sparse_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0},
        "step_us_median": statistics.median(step_us), "step_us_min": min(step_us),
        "step_us_without_kernel_events": statistics.mean(plain_us),
        "step_us_warm_l2": statistics.mean(warm_us),
        "step_us_cuda_graph": None if graph_us is None else statistics.mean(graph_us),
        "read_calibration_gbs": read_gbs,
        "effective_hbm_gbs_step": sparse_bytes / (t_step * 1e-6) / 1e9,
        "sparsity": {"skipped_fraction_per_head": 1.0 - kept_head_blocks / head_blocks,
                     "skipped_fraction_per_loaded_block": 1.0 - kept_tiles / total_tiles,
                     "kept_tiles": kept_tiles, "total_tiles": total_tiles},
        "dense": {"us_per_step": t_dense, "kernel_us": statistics.mean(dense_kernel_us), "bytes": dense_bytes,
                  "effective_hbm_gbs": dense_bytes / (statistics.mean(dense_kernel_us) * 1e-6) / 1e9},
        "speedup_vs_dense": t_dense / t_step,
        "residual_format": {"us_per_step": statistics.mean(res_us), "kernel_us": statistics.mean(res_kernel_us),
                            "algorithmic_bytes": res_bytes,
                            "effective_hbm_gbs": res_bytes / (statistics.mean(res_kernel_us) * 1e-6) / 1e9,
                            "frac": res_bytes / (statistics.mean(res_kernel_us) * 1e-6) / 1e9 / peak,
                            "note": "2-bit thumbnails + 8-bit residual keys: a kept block reads 8 KB + 16 KB "
                                    "instead of 32 KB; same selection, same protocol as the headline step"},
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, delta)
        one = cpu_baseline(w, delta, threads=1, seconds_target=5.0)
        line["cpu_baseline"]["value_1_thread"] = one["value"]
        line["cpu_baseline"]["sample_1_thread"] = one["sample"]
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
