#!/usr/bin/env python
"""Benchmark of the multiquery decode-attention hot path on B200.

One step = one whole pass of the path (the split kernel, which also merges the
sequences it cuts; on the FMA path a separate combine kernel) over one batch of
synthetic PaLM-shaped input.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Multi-GPU (torchrun, one rank per GPU): the path shards over whole sequences
(the paper's batch-sharded attention layout, Section 3.3), so every rank runs
the same per-GPU batch with no data-path collective: weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from mqa_workloads import WORKLOADS, make_inputs  # noqa: E402
from paper_2211_05102_b200 import roofline  # noqa: E402

METRIC = "mqa_decode_kv_cache_bandwidth"
UNIT = "GB/s"
DEFAULT_WORKLOAD = "palm540b"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_traffic(workload_name):
    """DRAM bytes per launch of the split kernel from the committed ncu summary, if there is one."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            return json.load(f).get(workload_name)
    except Exception:
        return None


def config_of(w, n_gpus, extra=None):
    cfg = {"workload": f"{w.name}: B={w.B} H={w.H} D={w.D} Lmax={w.Lmax} "
                       f"{'ragged lengths' if w.ragged else 'uniform lengths'} bf16 q/K/V fp32 out",
           "B_per_gpu": w.B, "H": w.H, "D": w.D, "Lmax": w.Lmax, "seed": w.seed,
           "parallelism": f"batch-sharded x{n_gpus}, no collective"}
    if extra:
        cfg.update(extra)
    return cfg


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and active throttle reasons over the samples taken in [t_begin, t_end]
        (time.time() values; all samples if the window holds none)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for line in self.file:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]),
                             [nm for nm, val in zip(names, f[4:8]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        self.file.close()
        os.unlink(self.file.name)
        inside = [r for r in rows if t_begin is not None and t_begin - 0.01 <= r[0] <= t_end + 0.01]
        use = inside or rows
        if use:
            reasons = sorted({nm for r in use for nm in r[4]})
            out.update(sm_mhz=statistics.median(r[1] for r in use), sm_max_mhz=max(r[2] for r in use),
                       power_w=statistics.median(r[3] for r in use), reasons=reasons, samples=len(use),
                       window="timed region" if inside else "whole run (no sample fell inside the timed region)")
        return out


def run_reference(args, w):
    """The fp64 CPU oracle, as it stands, timed on the host cores on a bounded sample
    of the workload (the first `sample_B` sequences)."""
    from oracle import ref
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_B = min(w.B, args.ref_sample_seqs)
    q, k, v, lengths = make_inputs(w)
    q, k, v, lengths = q[:sample_B].contiguous(), k[:sample_B].contiguous(), v[:sample_B].contiguous(), lengths[:sample_B].contiguous()
    rows = int(lengths.clamp(0, w.Lmax).sum())
    nbytes = roofline.ideal_kv_bytes(rows, w.D)
    cores = os.cpu_count() or 1
    for _ in range(args.warmup):
        ref.mqa_decode_ref(q, k, v, lengths, w.scale, num_threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ref.mqa_decode_ref(q, k, v, lengths, w.scale, num_threads=cores)
    dt = (time.perf_counter() - t0) / args.steps
    value = nbytes / dt / 1e9
    sample = f"first {sample_B} of {w.B} sequences of {w.name} ({rows} cache rows) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, args.gpus, {"sample": sample}),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args, w):
    from paper_2211_05102_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    # Every rank owns its own batch of whole sequences (same shapes, rank-specific seed).
    q, k, v, lengths = make_inputs(w, seed=w.seed + rank)
    rows = int(lengths.clamp(0, w.Lmax).sum())
    nbytes = roofline.ideal_kv_bytes(rows, w.D)
    qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), lengths.to(dev)
    out = torch.empty((w.B, w.H, w.D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(w.B, w.H, w.D, w.Lmax, device=dev)
    plan = binding.mqa_decode_plan(w.B, w.H, w.D, w.Lmax)
    stream = torch.cuda.current_stream()

    # L2 hygiene: inputs larger than L2 need nothing; smaller ones get an L2 flush between steps.
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    kv_alloc = 2 * k.numel() * 2
    flush = None
    if kv_alloc < 4 * l2_bytes:
        flush = torch.empty(int(2.5 * l2_bytes), dtype=torch.uint8, device=dev)

    def step():
        if flush is not None:
            flush.fill_(1)
        binding.mqa_decode(qd, kd, vd, ld, out, w.scale, ws, stream=stream, plan=plan)

    sampler = ClockSampler(local_rank)
    if rank == 0 and args.clock_spin_s > 0:
        sampler.start()
        time.sleep(args.clock_spin_s)      # nvidia-smi needs a moment before its first sample
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    launches_per_step = binding.mqa_last_launch_count()

    # ---- timed region: K steps, each bracketed by events so flush time is excluded ----
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, m, b in ev:          # force creation of the event handles
        m.record(stream)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t_begin = time.time()
    wall0 = time.perf_counter()
    for a, m, b in ev:
        if flush is not None:
            flush.fill_(1)
        a.record(stream)
        binding.mqa_decode_profiled(qd, kd, vd, ld, out, w.scale, ws, m, stream=stream, plan=plan)
        b.record(stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop(t_begin, time.time()) if rank == 0 else None
    step_ms = [a.elapsed_time(b) for a, m, b in ev]
    main_ms = [a.elapsed_time(m) for a, m, b in ev]          # split kernel only
    total_ms = sum(step_ms)
    if dist is not None:
        t = torch.tensor([total_ms, sum(main_ms)], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, main_total = float(t[0]), float(t[1])
    else:
        main_total = sum(main_ms)
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    ms_per_step = total_ms / args.steps
    main_ms_avg = main_total / args.steps
    value = world * nbytes / (ms_per_step * 1e-3) / 1e9

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- end to end through the host entry point (pinned host buffers, copies inside the timed region) ----
    e2e = None
    try:
        qh, kh, vh, lh = q.pin_memory(), k.pin_memory(), v.pin_memory(), lengths.pin_memory()
        oh = torch.empty((w.B, w.H, w.D), dtype=torch.float32).pin_memory()
        del flush
        scratch = torch.empty(binding.mqa_decode_host_scratch_bytes(w.B, w.H, w.D, w.Lmax), dtype=torch.uint8, device=dev)
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            binding.mqa_decode_host(qh, kh, vh, lh, oh, w.scale, scratch, stream=stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(e2e_steps):
            binding.mqa_decode_host(qh, kh, vh, lh, oh, w.scale, scratch, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        h2d = q.numel() * 2 + k.numel() * 2 + v.numel() * 2 + lengths.numel() * 4
        e2e = {"value": world * nbytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": oh.numel() * 4, "steps": e2e_steps}
        del scratch
    except Exception as exc:  # report, do not hide
        e2e = {"value": None, "unit": UNIT, "error": repr(exc), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}

    # ---- CPU baseline: the oracle on a bounded sample; doubles as a parity spot check ----
    from oracle import ref
    sample_B = min(w.B, args.ref_sample_seqs)
    cores = os.cpu_count() or 1
    qs, ks, vs, ls = q[:sample_B].contiguous(), k[:sample_B].contiguous(), v[:sample_B].contiguous(), lengths[:sample_B].contiguous()
    t0 = time.perf_counter()
    expect = ref.mqa_decode_ref(qs, ks, vs, ls, w.scale, num_threads=cores)
    cpu_dt = time.perf_counter() - t0
    srows = int(ls.clamp(0, w.Lmax).sum())
    got = out[:sample_B].cpu().double().numpy()
    import numpy as np
    err_ratio = float((np.abs(got - expect) / (2e-3 * (1 + np.abs(expect)))).max())
    cpu = {"value": roofline.ideal_kv_bytes(srows, w.D) / cpu_dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {sample_B} of {w.B} sequences of {w.name} ({srows} cache rows), one repetition, {cpu_dt:.2f} s"}

    peak, peak_kind = measured_peak()
    achieved = nbytes / (main_ms_avg * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "us_per_step": ms_per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in, f32 accumulate",
        "data": "synthetic",
        "config": config_of(w, world, {
            "plan": {"path": {1: "fma", 2: "tcgen05"}[plan.path], "num_ctas": plan.num_ctas, "tile_rows": plan.tile_rows,
                     "adaptive": bool(plan.adaptive),
                     # blocks that took tiles in the last step (workspace header word 3, written by the kernel)
                     "ctas_used": int(ws[:16].view(torch.int32)[3])},
            "l2": "inputs larger than L2" if kv_alloc >= 4 * l2_bytes else "L2 flushed between steps (flush untimed)",
            "ideal_kv_bytes_per_step": nbytes}),
        "pct_of_8000_GBps": 100.0 * value / world / NOMINAL_HBM_GBS,
        "pct_of_measured_copy_peak": 100.0 * value / world / peak,
        "roofline": {"bound": "hbm", "kernel": "split kernel (mqa_fma/mqa_tc)", "achieved": achieved, "peak": peak,
                     "peak_kind": f"{peak_kind} STREAM-style copy", "unit": "GB/s", "frac": achieved / peak,
                     "kernel_us": main_ms_avg * 1e3, "traffic": measured_traffic(w.name)},
        "cpu_baseline": cpu,
        "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        "parity_spot_check_err_over_tol": err_ratio,
        "wall_s_timed_region": wall,
    }
    print(json.dumps(result))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--clock-spin-s", type=float, default=0.3,
                    help="seconds to let the nvidia-smi clock sampler start before the warm-up (0 = no sampling)")
    ap.add_argument("--ref-sample-seqs", type=int, default=512,
                    help="sequences of the workload the CPU oracle is timed on")
    args = ap.parse_args()
    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
