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
# context 32768; traffic grows in proportion to the blocks processed): (308.62 + 6.12) MB / 308.28 MB.
NCU_TRAFFIC_RATIO = 1.021


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


def cpu_baseline(w, delta, threads=None, rows_per_thread=None):
    """Time the oracle, as it stands, on the same workload.  With ``rows_per_thread`` None every (sequence, query
    head) row is computed (the measured time is the step); otherwise a bounded sample with the workload's own mix of
    head kinds, and the measured and the scaled time are reported side by side.  Reported context, not a target."""
    from oracle import ffd_oracle as O
    cores = threads or O.max_threads()
    O.set_threads(cores)
    total_rows = w.B * w.Hq
    units = None
    if rows_per_thread is not None:
        flat = set(w.flat_heads)
        kinds = [[g for g in range(w.Hkv) if g not in flat], sorted(flat)]
        units = []
        for gs in kinds:
            for i in range(cores * rows_per_thread):
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
    n_rows = total_rows if units is None else len(units)
    scale = total_rows / n_rows
    sample = (f"all {total_rows} (sequence, query head) rows, scan+select+attend, nothing scaled" if units is None else
              f"{n_rows} of {total_rows} (sequence, query head) rows in the workload's own mix of head kinds, measured "
              f"time scaled by {scale:.1f}")
    return {"value": t * scale * 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "measured_seconds": t, "scaled_by": scale,
            "sample": sample + f"; full-cache quantizer {t_quant:.1f} s not included"}


def run_reference(args, rank, world):
    """The reference arm of this build is the CPU oracle (there is no reference implementation to install): every
    step computes every (sequence, query head) row of the workload, nothing is scaled."""
    if rank != 0:
        return
    from oracle import ffd_oracle as O
    w = make_workload(args.workload, **workload_overrides(args))
    delta = args.delta if args.delta is not None else w.deltas[0]
    cores = O.max_threads()
    O.set_threads(cores)
    codes, scales = O.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        O.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                 w.max_blocks, delta)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    us = statistics.mean(times) * 1e6
    sample = f"all {w.B * w.Hq} (sequence, query head) rows every step, nothing scaled"
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
            "step": "tail-block re-quantize + the sparse decode call (pseudo-max, fused scan/select/attend and combine kernels; "
                    "one kernel for all of them on geometries with fewer than two 32-block work items per SM)",
            "kernel_events": "roofline.kernel_us comes from a separate loop of the same step in which every step carries "
                             "a CUDA-event pair around the fused kernel; the steps behind `value` carry none",
            "aggregate": "value = max-over-ranks step time / n_gpus (each rank decodes its own batch)"}


def stats(xs):
    return {"mean": statistics.mean(xs), "median": statistics.median(xs), "min": min(xs), "samples": len(xs)}


class Bench:
    """One workload resident on the device and the timing loops over it."""

    def __init__(self, ffd, w, delta, shared=None, bits=2):
        from tests.device_cache import DeviceCache
        self.ffd, self.w, self.delta = ffd, w, delta
        self.dc = DeviceCache(w, ffd.Config(w.Hq, w.Hkv, out_dtype=1, quant_bits=bits))
        self.dc.quantize()
        self.first_token = torch.from_numpy(np.maximum(w.seq_lens - 1, 0)).to("cuda")
        if shared is None:
            shared = {"flush": torch.empty(256 << 20, dtype=torch.uint8, device="cuda"),
                      "drain": torch.zeros(32 << 20, dtype=torch.int64, device="cuda"),      # 256 MiB, only ever read
                      "k_start": torch.cuda.Event(enable_timing=True), "k_stop": torch.cuda.Event(enable_timing=True)}
            shared["k_start"].record(), shared["k_stop"].record()   # materialise the CUDA events for the library
        self.shared = shared
        self.stream = torch.cuda.current_stream()
        kept = torch.zeros(w.B, w.Hq, w.max_blocks, dtype=torch.uint8, device="cuda")
        self.dc.decode(delta, kept_mask=kept)
        assert ffd.ffd_read_device_status(self.dc.workspace) == 0
        kept_np = kept.cpu().numpy()
        self.kept_tiles = union_kept_tiles(kept_np, w)
        self.total_tiles = sum(w.num_blocks(b) for b in range(w.B)) * w.Hkv
        self.head_blocks = sum(w.num_blocks(b) for b in range(w.B)) * w.Hq
        self.kept_head_blocks = sum(int(kept_np[b, :, : w.num_blocks(b)].sum()) for b in range(w.B))
        self.sparse_bytes = algorithmic_bytes(w, self.kept_tiles)
        self.dense_bytes = algorithmic_bytes(w, 0, dense=True)

    def step(self):
        self.dc.quantize(first_token=self.first_token)
        self.dc.decode(self.delta)

    def timed_loop(self, fn, n, profile_kernel=False, cold=True):
        """n steps, each bracketed by CUDA events on the launching stream, L2 flushed (untimed) before each.
        profile_kernel: every step also carries the library's event pair around its fused kernel."""
        sh = self.shared
        self.ffd.ffd_profile_events(sh["k_start"] if profile_kernel else None, sh["k_stop"] if profile_kernel else None)
        total, kernel = [], []
        for _ in range(n):
            if cold:
                sh["flush"].fill_(1)   # evicts every input line from L2 ...
                sh["drain"].sum()      # ... and this read sweep pushes the fill's dirty lines out to HBM, so that their
                                       # write-back (an artefact of the flush, not of the workload) ends before the timing starts
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(self.stream)
            fn()
            b.record(self.stream)
            b.synchronize()
            total.append(a.elapsed_time(b) * 1e3)
            if profile_kernel:
                kernel.append(sh["k_start"].elapsed_time(sh["k_stop"]) * 1e3)
        self.ffd.ffd_profile_events(None, None)
        return total, kernel

    def fidelity(self):
        """Sec. 5 "Retrieval Fidelity Analysis" on the GPU's own two paths: the sparse output against the dense one."""
        dc = self.dc
        dc.decode(self.delta)
        torch.cuda.synchronize()
        o_s, l_s = dc.out.double().clone(), dc.lse.double().clone()
        dc.dense()
        torch.cuda.synchronize()
        o_d, l_d = dc.out.double(), dc.lse.double()
        live = torch.from_numpy(self.w.seq_lens > 0).to("cuda")
        cos = torch.nn.functional.cosine_similarity(o_s, o_d, dim=-1)[live]
        return {"min_cosine_sparse_vs_dense": float(cos.min()), "mean_cosine_sparse_vs_dense": float(cos.mean()),
                "max_abs_lse_error": float((l_s - l_d)[live].abs().max())}

    def brief(self, steps, peak):
        """The figures of a secondary workload: step, fused kernel, bytes and roofline fraction, dense step."""
        self.timed_loop(self.step, 3)
        step_us, _ = self.timed_loop(self.step, steps)
        _, kernel_us = self.timed_loop(self.step, max(steps, 20), profile_kernel=True)
        self.timed_loop(self.dc.dense, 3)
        dense_us, _ = self.timed_loop(self.dc.dense, max(5, steps // 2))
        t_k = statistics.mean(kernel_us)
        gbs = self.sparse_bytes / (t_k * 1e-6) / 1e9
        return {"workload": workload_config(self.w, self.delta, None)["workload"], "us_per_step": statistics.mean(step_us),
                "us_per_step_median": statistics.median(step_us), "kernel_us": stats(kernel_us),
                "algorithmic_bytes": self.sparse_bytes, "achieved_gbs": gbs, "frac": gbs / peak,
                "dense_us_per_step": statistics.mean(dense_us),
                "speedup_vs_dense": statistics.mean(dense_us) / statistics.mean(step_us),
                "skipped_fraction_per_loaded_block": 1.0 - self.kept_tiles / self.total_tiles,
                "fidelity": self.fidelity()}


def depth_table(ffd, peak, steps, batch=4, context=131072):
    """App. "Bandwidth Proportionality of Quantization Depth": the scan at 2, 4 and 8 bits on one scan-only workload
    (sink needle in every head, delta 0: a handful of blocks kept), decode call alone (no tail re-quantize), cold L2.
    kernel_us brackets the scan-select-attend kernel(s) of the call: the fused kernel at 2 bits, the scan kernel plus the
    decode kernel at 4 and 8 bits."""
    rows = []
    w = make_workload("C2", N=context, B=batch)
    tiles = sum(w.num_blocks(b) for b in range(w.B)) * w.Hkv
    for bits in (2, 4, 8):
        b = Bench(ffd, w, 0.0, bits=bits)
        decode = lambda: b.dc.decode(0.0)
        b.timed_loop(decode, 3)
        step_us, _ = b.timed_loop(decode, steps)
        _, kernel_us = b.timed_loop(decode, max(steps, 20), profile_kernel=True)
        scan_bytes = tiles * (1024 * bits + 256)
        t = statistics.mean(kernel_us)
        rows.append({"bits": bits, "bytes_per_block_and_kv_head": 1024 * bits + 256, "scan_bytes": scan_bytes,
                     "kept_tiles": b.kept_tiles, "total_tiles": tiles, "decode_us": statistics.mean(step_us),
                     "kernel_us": stats(kernel_us), "scan_gbs": scan_bytes / (t * 1e-6) / 1e9,
                     "frac": scan_bytes / (t * 1e-6) / 1e9 / peak})
        del b
        torch.cuda.empty_cache()
    base = rows[0]
    for r in rows:
        r["bytes_ratio_vs_2bit"] = r["scan_bytes"] / base["scan_bytes"]
        r["kernel_time_ratio_vs_2bit"] = r["kernel_us"]["mean"] / base["kernel_us"]["mean"]
    return {"workload": f"C2 recipe at batch {batch}, context {context} (32 query / 8 KV heads), delta 0, decode call only",
            "rows": rows}


def selection_table(ffd, w, delta, steps):
    """Sec. 4.4 "Selection-Rule Overhead": the decode call under each selection rule at a matched keep ratio (top-k's k is
    the mean number of blocks a head keeps under top-delta), all through ffd_decode_select's three kernels (scan, select,
    decode), cold L2; the fused ffd_decode call beside them.  What differs between the rows is the select kernel (one
    reduction more for the global max, a prefix scan for the running max, a four-pass radix select for top-k) and the
    blocks each rule keeps."""
    b = Bench(ffd, w, delta)
    dc = b.dc
    kept = torch.zeros(w.B, w.Hq, w.max_blocks, dtype=torch.uint8, device="cuda")
    dc.decode(delta, kept_mask=kept)
    k_match = max(1, round(b.kept_head_blocks / (w.B * w.Hq)))
    rows = []

    def measure(name, fn, mask_fn):
        kept.zero_()
        mask_fn(kept)
        torch.cuda.synchronize()
        frac = sum(int(kept[i, :, : w.num_blocks(i)].sum()) for i in range(w.B)) / b.head_blocks
        loaded = union_kept_tiles(kept.cpu().numpy(), w) / b.total_tiles
        b.timed_loop(fn, 3)
        us, _ = b.timed_loop(fn, steps)
        _, kus = b.timed_loop(fn, max(steps, 20), profile_kernel=True)
        rows.append({"rule": name, "keep_ratio_per_head": frac, "loaded_fraction_of_kv_tiles": loaded,
                     "decode_us": statistics.mean(us),
                     "decode_us_median": statistics.median(us), "kernels_us": statistics.mean(kus)})

    measure("top-delta, fused kernel (ffd_decode)", lambda: dc.decode(delta), lambda m: dc.decode(delta, kept_mask=m))
    for name, rule, k in (("top-delta (pseudo-max)", ffd.RULE_PSEUDO_MAX, 0), ("global max", ffd.RULE_GLOBAL_MAX, 0),
                          ("running max", ffd.RULE_RUNNING_MAX, 0), (f"top-k, k = {k_match}", ffd.RULE_TOP_K, k_match)):
        measure(name, lambda r=rule, kk=k: dc.decode_select(r, kk, delta),
                lambda m, r=rule, kk=k: dc.decode_select(r, kk, delta, kept_mask=m))
    base = rows[1]["decode_us"]
    for r in rows[1:]:
        r["extra_us_vs_top_delta_same_path"] = r["decode_us"] - base
        r["extra_us_per_head"] = (r["decode_us"] - base) / (w.B * w.Hq)
    return {"workload": workload_config(w, delta, None)["workload"], "matched_k": k_match, "rows": rows}


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
    ap.add_argument("--table", default=None, choices=["depth", "selection"],
                    help="print only the quantization-depth table (C2 recipe at --batch / --context, defaults 4 / 131072) or "
                         "the selection-rule table (on --workload) as JSON and exit: small cases of them are what the ncu "
                         "captures of the scan and select kernels run")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the secondary workloads (C4, C5) and the quantization-depth table of the bench line")
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

    if args.table == "depth":
        print(json.dumps(depth_table(ffd, measured_peaks()[0], args.steps, args.batch or 4, args.context or 131072)), flush=True)
        return
    w = make_workload(args.workload, **workload_overrides(args))
    delta = args.delta if args.delta is not None else w.deltas[0]
    if args.table == "selection":
        print(json.dumps(selection_table(ffd, w, delta, args.steps)), flush=True)
        return
    bench = Bench(ffd, w, delta)
    dc, step, timed_loop = bench.dc, bench.step, bench.timed_loop

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    timed_loop(step, args.warmup)
    barrier()
    t_begin = time.perf_counter()
    step_us, _ = timed_loop(step, args.steps)
    barrier()
    clocks = sampler.stop(t_begin, time.perf_counter())
    # the fused kernel alone: the same step, every one with the library's event pair around that kernel (the records sit
    # between the step's kernels and cost their programmatic-launch overlap, so these steps are not the ones behind `value`)
    _, kernel_us = timed_loop(step, max(args.steps, 20), profile_kernel=True)
    # the dense path of the same library, same protocol (context for the speedup figure)
    timed_loop(dc.dense, 3)
    dense_us, _ = timed_loop(dc.dense, min(max(5, args.steps // 2), 100))
    _, dense_kernel_us = timed_loop(dc.dense, 20, profile_kernel=True)
    # the same step without the flush (whatever of the previous step is still in L2 stays there) ...
    warm_us, _ = timed_loop(step, min(args.steps, 200), cold=False)
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
        graph_us, _ = timed_loop(graph.replay, min(args.steps, 200))
    except Exception as exc:   # reported, not fatal: the graph number is an extra
        graph_us = None
        print(f"bench: CUDA graph capture failed: {exc}", file=sys.stderr)
    # ... and a pure-read calibration: a sum over 1 GiB (torch's reduction kernel), cold
    calib = torch.zeros(128 << 20, dtype=torch.int64, device="cuda")
    calib_us, _ = timed_loop(calib.sum, 13)
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

    timed_loop(e2e_step, 3)
    e2e_us, _ = timed_loop(e2e_step, min(args.steps, 200))
    h2d = in_host.numel()
    d2h = out_host.numel() * 4
    fidelity = bench.fidelity()

    # the same step on the 2 + 8 bit key format (kept blocks refined from 8-bit residuals instead of 16-bit keys):
    # tail re-quantize of thumbnails and residuals + pseudo-max + fused kernel + combine, same protocol.  Measured
    # last: it swaps the workspace for the larger one that format needs.
    dc.quantize_residual()

    def residual_step():
        dc.quantize_both(first_token=bench.first_token)
        dc.decode_residual(delta)

    timed_loop(residual_step, 3)
    res_us, _ = timed_loop(residual_step, min(max(5, args.steps // 2), 100))
    _, res_kernel_us = timed_loop(residual_step, 20, profile_kernel=True)
    res_bytes = bench.total_tiles * CODE_BYTES_PER_TILE + bench.kept_tiles * (KV_BYTES_PER_TILE // 2 + KV_BYTES_PER_TILE // 4)

    t_step = statistics.mean(step_us)
    t_e2e = statistics.mean(e2e_us)
    t_step, t_e2e = reduce_max_over_ranks([t_step, t_e2e], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    # kernels of this library per timed step: tail re-quantize + (pseudo-max, fused, combine), or + the single-launch
    # kernel when the geometry has fewer than two 32-block work items per SM (the library's own rule)
    sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
    small = w.B * w.Hkv * ((w.max_blocks + 31) // 32) < 2 * sms
    launches_per_step = 2 if small else 4
    sparse_bytes = bench.sparse_bytes
    t_kernel = statistics.mean(kernel_us)
    achieved = sparse_bytes / (t_kernel * 1e-6) / 1e9
    t_dense = statistics.mean(dense_us)
    t_dense_kernel = statistics.mean(dense_kernel_us)
    t_res_kernel = statistics.mean(res_kernel_us)
    line = {
        "metric": METRIC, "value": t_step / world, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_step / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in / fp32 accumulate (fp16 x fp16 -> fp32 tensor-core scan)",
        "data": "synthetic", "config": workload_config(w, delta, args),
        "clocks": clocks,
        "e2e": {"value": t_e2e / world, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (None if NCU_TRAFFIC_RATIO is None else sparse_bytes * NCU_TRAFFIC_RATIO),
                     "peak_source": f"{peak_kind} copy bandwidth (of {peak_kind})",
                     "kernel": "small_sparse_kernel" if small else "fused_sparse_kernel",
                     "kernel_us": t_kernel, "kernel_us_median": statistics.median(kernel_us),
                     "kernel_us_min": min(kernel_us), "kernel_us_samples": len(kernel_us),
                     "algorithmic_bytes": sparse_bytes, "frac_of_nominal_8TBs": achieved / 8000.0},
        "step_us_median": statistics.median(step_us), "step_us_min": min(step_us),
        "step_us_warm_l2": statistics.mean(warm_us),
        "step_us_cuda_graph": None if graph_us is None else statistics.mean(graph_us),
        "read_calibration_gbs": read_gbs,
        "effective_hbm_gbs_step": sparse_bytes / (t_step * 1e-6) / 1e9,
        "sparsity": {"skipped_fraction_per_head": 1.0 - bench.kept_head_blocks / bench.head_blocks,
                     "skipped_fraction_per_loaded_block": 1.0 - bench.kept_tiles / bench.total_tiles,
                     "kept_tiles": bench.kept_tiles, "total_tiles": bench.total_tiles},
        "fidelity": fidelity,
        "dense": {"us_per_step": t_dense, "kernel_us": t_dense_kernel, "bytes": bench.dense_bytes,
                  "effective_hbm_gbs": bench.dense_bytes / (t_dense_kernel * 1e-6) / 1e9},
        "speedup_vs_dense": t_dense / t_step,
        "residual_format": {"us_per_step": statistics.mean(res_us), "kernel_us": t_res_kernel,
                            "algorithmic_bytes": res_bytes,
                            "effective_hbm_gbs": res_bytes / (t_res_kernel * 1e-6) / 1e9,
                            "frac": res_bytes / (t_res_kernel * 1e-6) / 1e9 / peak,
                            "note": "2-bit thumbnails + 8-bit residual keys: a kept block reads 8 KB + 16 KB "
                                    "instead of 32 KB; same selection, same protocol as the headline step"},
    }
    if not args.no_extras and world == 1:
        # the scan-bound configurations, same protocol, fewer steps: C4 (one 256K sequence) and C5 (paged batch of 16)
        del bench, dc, step, timed_loop, in_host, out_host
        torch.cuda.empty_cache()
        extra = {}
        for name in ("C4", "C5"):
            if name == args.workload:
                continue
            wx = make_workload(name)
            bx = Bench(ffd, wx, wx.deltas[1] if name == "C4" else wx.deltas[0])
            extra[name.lower()] = bx.brief(min(args.steps, 50), peak)
            del bx, wx
            torch.cuda.empty_cache()
        line["extra"] = extra
        line["quantization_depth"] = depth_table(ffd, peak, min(args.steps, 30))
        line["selection_rules"] = selection_table(ffd, w, delta, min(args.steps, 30))
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, delta)
        one = cpu_baseline(w, delta, threads=1, rows_per_thread=8)
        line["cpu_baseline"]["value_1_thread"] = one["value"]
        line["cpu_baseline"]["sample_1_thread"] = one["sample"]
        line["cpu_baseline"]["measured_seconds_1_thread"] = one["measured_seconds"]
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
