#!/usr/bin/env python
"""Benchmark of the fused synchronisation round on the ResNet-50-shaped workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With --gpus N > 1 and no WORLD_SIZE in the environment the script starts the N ranks itself
(torch.distributed.run on 127.0.0.1); it never reports n_gpus = 1 for a request of more.

One step = one qs_sync_round (form u, select, quantize, memory update, pack, decode, update x,
broadcast) over R = 8 workers of d = 25,557,032 coordinates laid out as ResNet-50's 161 tensors,
Top_k with k = 0.1% d over the flat vector composed with the sign/l1 quantizer; a fresh Laplace
drift is added to the workers' models before every step, outside the timed region.  The reported
value is the minimum bytes a round has to move (16 R d + 8 d + record bytes written and read)
divided by the round time.  Prints one JSON line.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1906_02367_b200 import inputs as I  # noqa: E402

R = 8
METRIC = "sync_round_effective_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
DENSE_PROFILE = os.path.join("profiles", "pass_a_tma_kernel_resnet50_half_size.txt")


def dense_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dense pass on the bench workload, as the
    tracked ncu summary states it (machine-readable lines `bench_traffic_bytes_per_launch:`, `captured:` and
    `kernel:`); the capture is of a half-size case and the figure is scaled by the coordinates (traffic grows
    with d).  None when the summary is missing or does not name the kernel the bench times."""
    path = os.path.join(ROOT, DENSE_PROFILE)
    if not os.path.exists(path):
        return None
    fields = {}
    for line in open(path):
        if ":" in line:
            key, _, val = line.partition(":")
            fields[key.strip()] = val.strip()
    if fields.get("kernel") != "pass_a_tma_kernel" or "bench_traffic_bytes_per_launch" not in fields:
        return None
    return {"bytes": int(fields["bench_traffic_bytes_per_launch"]), "captured": fields.get("captured"),
            "source": DENSE_PROFILE + " (half-size capture scaled by d)"}


def workload(variant, shrink=1):
    sizes = I.scaled_sizes(I.resnet50_tensor_sizes(), shrink)
    off = I.segments_from_sizes(sizes)
    d = int(off[-1])
    if variant == "per_tensor":
        return sizes, off, d, off, I.k_per_tensor_ratio(sizes)
    if variant == "paper_table":                   # the per-tensor rule of the paper's ResNet-50 runs: k_t = min(d_t, 1000)
        return sizes, off, d, off, I.k_per_tensor_capped(sizes, max(1, 1000 // shrink))
    return sizes, off, d, np.array([0, d], np.int64), np.array([I.k_from_ratio(d, 1, 1000)], np.int64)


def min_bytes(d, wire_bytes):
    """Bytes one round cannot avoid: read xw, mem and write mem, xw (16 B per worker coordinate),
    read and write x (8 B per coordinate), records written once and read once."""
    return 16 * R * d + 8 * d + 2 * wire_bytes


def peak_hbm():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 <= t <= t1 and len(r) >= 7] or [r for _, r in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]), "reasons": reasons,
                "power_w_max": max(float(r[2]) for r in rows), "samples": len(rows)}


def max_over_ranks(ms, device):
    """Slowest rank's time: the replicas are independent, the job is as slow as the slowest."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_round, steps, total_ms, world):
    """Whole-job GB/s: every rank moved bytes_per_round per step in total_ms (max over ranks)."""
    return world * bytes_per_round * steps / (total_ms * 1e-3) / 1e9


WORKLOAD_TEXT = ("ResNet-50-shaped round: R=8, d={d} (161 tensors), Top_k k=0.1% ({variant}), "
                 "sign/l1 quantizer, Laplace drift per tensor, memory carried")


def headline_config(variant, d, k_total):
    return {"workload": WORKLOAD_TEXT.format(d=d, variant=variant), "variant": variant, "R": R, "d": d, "k_total": int(k_total),
            "l2_policy": "inputs (3.4 GB per round) larger than L2", "multi_gpu": "independent replicas"}


def time_rounds(torch, ctx, wire, bits, drift, steps, warmup, barrier):
    """warmup untimed rounds, then `steps` rounds timed one by one with CUDA events on the context's stream
    (a fresh drift before each, outside the timed region).  Returns the per-step milliseconds."""
    for _ in range(warmup):
        drift()
        ctx.sync_round(wire, bits_out=bits)
    assert ctx.sync_status() == 0, ctx.last_error()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    for i in range(steps):
        drift()                       # untimed: the local steps that precede a synchronisation
        starts[i].record()
        ctx.sync_round(wire, bits_out=bits)
        ends[i].record()
    barrier()
    assert ctx.sync_status() == 0, ctx.last_error()
    return [s.elapsed_time(e) for s, e in zip(starts, ends)]


def spread(per_step):
    a = np.asarray(per_step, np.float64)
    return {"min": float(a.min()), "median": float(np.median(a)), "max": float(a.max())}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1906_02367_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.selftest_cpu:
        return selftest_cpu(rank, world, args)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_src = peak_hbm()
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    sizes, off, d, _, _ = workload("flat", args.shrink)
    scales = I.tensor_scales(len(sizes), seed=0)
    per_elem = torch.from_numpy(np.repeat(scales, np.diff(off))).to(dev)
    x = torch.from_numpy(I.model_init(d, seed=rank)).to(dev)
    xw = x.expand(R, d).contiguous()
    mem = torch.zeros((R, d), dtype=torch.float32, device=dev)
    e1 = torch.empty((R, d), dtype=torch.float32, device=dev)
    e2 = torch.empty_like(e1)
    bits = torch.zeros(R, dtype=torch.int64, device=dev)

    def drift():
        # Laplace(0, b_t) per tensor as the difference of two exponentials
        e1.exponential_(generator=gen)
        e2.exponential_(generator=gen)
        e1.sub_(e2).mul_(per_elem)
        xw.add_(e1)

    def measure(variant, steps, warmup, sample_clocks):
        """One variant of the headline workload on fresh state; returns (summary dict, context, wire)."""
        _, _, _, seg_off, kseg = workload(variant, args.shrink)
        xw.copy_(x.expand(R, d))
        mem.zero_()
        ctx = B.Context(R, d, int(kseg[0]), 1, B.QS_TOPK, B.QS_SIGN_L1, seed=rank)
        if len(kseg) > 1:
            ctx.set_segments(seg_off, kseg)
        ctx.bind(x, xw, mem)
        wire = ctx.new_wire()
        ctx.enable_phase_timing(True)
        sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid)) if sample_clocks else None
        st0 = None

        def timed_barrier():
            nonlocal st0
            barrier()
            if st0 is None:                       # first call: the warm-up is over
                st0 = ctx.stats()
                ctx.phase_timing()
        t0 = time.time()
        per_step = time_rounds(torch, ctx, wire, bits, drift, steps, warmup, timed_barrier)
        t1 = time.time()
        clocks = sampler.stop(t0, t1) if sampler else None
        phases = ctx.phase_timing()
        ctx.enable_phase_timing(False)
        st1 = ctx.stats()
        wire_bytes = int(bits.sum().item() + 7) // 8
        # the last round's records once more in the gap-coded form (outside the timed region): what
        # would travel with the indices sent as gaps, and what the two conversions cost
        packed = torch.zeros((R, ctx.gap_words()), dtype=torch.int32, device=dev)
        gap_bits = torch.zeros(R, dtype=torch.int64, device=dev)
        back = torch.zeros_like(wire)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for _ in range(2):
            ev[0].record()
            ctx.recode_gaps(wire, packed, None, gap_bits)
            ev[1].record()
            ctx.decode_gaps(packed, back)
            ev[2].record()
        torch.cuda.synchronize()
        assert ctx.sync_status() == 0 and torch.equal(back, wire), "gap-coded records do not decode to the plain ones"
        gap = {"wire_bytes_per_round": int(gap_bits.sum().item() + 7) // 8, "recode_ms": ev[0].elapsed_time(ev[1]),
               "decode_ms": ev[1].elapsed_time(ev[2])}
        del packed, back
        total_ms = max_over_ranks(float(sum(per_step)), dev)
        bmin = min_bytes(d, wire_bytes)
        value = aggregate_value(bmin, steps, total_ms, world)
        out = {"value": value, "ms_per_step": total_ms / steps, "ms_per_step_spread": spread(per_step),
               "pct_of_nominal_8TBps": 100.0 * value / world / NOMINAL_HBM_GBS, "pct_of_measured_copy": 100.0 * value / world / peak,
               "min_bytes_per_round": bmin, "wire_bytes_per_round": wire_bytes, "gap_coded": gap, "k_total": int(kseg.sum()),
               "gpu_launches": st1["launches"] - st0["launches"],
               "fallback_worker_rounds": st1["fallback_worker_rounds"] - st0["fallback_worker_rounds"],
               "phases_ms_per_round": {k: v / max(1, phases["rounds"]) for k, v in phases.items() if k != "rounds"},
               "clocks": clocks, "seg_off": seg_off, "kseg": kseg}
        return out, ctx, wire

    m, ctx, wire = measure(args.variant, args.steps, args.warmup, rank == 0)
    seg_off, kseg = m.pop("seg_off"), m.pop("kseg")
    result = {
        "metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": headline_config(args.variant, d, m["k_total"]),
        "worker_elements_per_s": world * R * d / (m["ms_per_step"] * 1e-3),
        "pct_of_nominal_8TBps": m["pct_of_nominal_8TBps"], "pct_of_measured_copy": m["pct_of_measured_copy"],
        "min_bytes_per_round": m["min_bytes_per_round"], "wire_bytes_per_round": m["wire_bytes_per_round"],
        "gap_coded": m["gap_coded"],
        "ms_per_step_median": m["ms_per_step_spread"]["median"], "ms_per_step_spread": m["ms_per_step_spread"],
        "gpu_launches": m["gpu_launches"], "fallback_worker_rounds": m["fallback_worker_rounds"],
        "phases_ms_per_round": m["phases_ms_per_round"], "kernels_per_round": m["gpu_launches"] / max(1, args.steps),
        "clocks": m["clocks"],
    }
    # roofline of the dominant kernel (the dense pass: reads xw, mem, writes mem, reads x once):
    # 12 B per worker coordinate + 4 B per coordinate
    dense_ms = m["phases_ms_per_round"]["dense_pass"]
    dense_bytes = 12 * R * d + 4 * d
    achieved = dense_bytes / (dense_ms * 1e-3) / 1e9 if dense_ms > 0 else 0.0
    traffic = dense_traffic() if args.shrink == 1 else None
    result["roofline"] = {"kernel": "pass_a_tma_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                          "frac": achieved / peak, "peak_source": peak_src,
                          "traffic": traffic["bytes"] if traffic else None,
                          "traffic_source": traffic["source"] if traffic else None, "traffic_captured": traffic["captured"] if traffic else None,
                          "achieved_from_traffic": traffic["bytes"] / (dense_ms * 1e-3) / 1e9 if traffic and dense_ms > 0 else None,
                          "algorithmic_bytes_per_launch": dense_bytes, "ms_per_launch": dense_ms,
                          "note": "the event-timed launch includes launch latency; above 1.0 means the pass is as fast as the copy the peak was measured with"}

    if rank == 0 and world == 1 and not args.no_e2e:
        result["e2e"] = run_e2e(torch, ctx, x, xw, mem, wire, bits, drift, d)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        drift()
        torch.cuda.synchronize()
        result["cpu_baseline"] = cpu_round(x.cpu().numpy(), xw.cpu().numpy(), mem.cpu().numpy(), seg_off, kseg, d)
    ctx.destroy()
    del wire
    if rank == 0 and world == 1 and args.variant == "flat" and args.shrink == 1 and not args.headline_only:
        # the other workloads named with the headline one, each timed the same way on a shorter run
        other, ctx2, wire2 = measure("per_tensor", max(20, args.steps // 2), max(12, args.warmup // 2), False)
        ctx2.destroy()
        del wire2
        table, ctx3, wire3 = measure("paper_table", max(20, args.steps // 4), max(12, args.warmup // 2), False)
        ctx3.destroy()
        del wire3
        for k in ("seg_off", "kseg", "clocks"):
            other.pop(k)
            table.pop(k)
        del e1, e2, xw, mem, per_elem
        torch.cuda.empty_cache()
        result["other_workloads"] = {"config2_per_tensor": other, "config2_paper_table_k_min_dt_1000": table,
                                     "config3_randk": time_config3(torch, B, dev, peak),
                                     "config5_sweep": time_config5(torch, B, dev, peak)}
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


def time_large(torch, B, dev, peak, R_, d, k, s, sparsifier, drift_rows, x, xw, mem, seed, steps=5, warmup=4):
    """One large single-segment QSGD workload on preallocated state: median round time and the derived figures."""
    mem.zero_()
    xw.copy_(x.expand(R_, d))
    ctx = B.Context(R_, d, k, s, sparsifier, B.QS_QSGD, seed=seed)
    ctx.bind(x, xw, mem)
    wire = ctx.new_wire()
    bits = torch.zeros(R_, dtype=torch.int64, device=dev)
    per_step = time_rounds(torch, ctx, wire, bits, drift_rows, steps, warmup, torch.cuda.synchronize)
    st = ctx.stats()
    ms = float(np.median(per_step))
    bmin = 16 * R_ * d + 8 * d + 2 * (int(bits.sum().item() + 7) // 8)
    gbs = bmin / (ms * 1e-3) / 1e9
    ctx.destroy()
    del wire
    torch.cuda.empty_cache()
    return {"k": k, "s": s, "ms_per_round": ms, "GBps": gbs, "pct_of_nominal_8TBps": 100 * gbs / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100 * gbs / peak, "worker_elements_per_s": R_ * d / (ms * 1e-3),
            "fallback_worker_rounds": st["fallback_worker_rounds"], "steps": steps, "warmup": warmup}


def time_config3(torch, B, dev, peak, shrink=1, steps=5, warmup=4):
    """R = 16, d = 2^26 (divided by shrink), Gaussian drift N(0, 1e-3), Rand_k k = 1% by keyed-hash rank, QSGD s = 4."""
    R3, d = 16, (1 << 26) // shrink
    gen = torch.Generator(device=dev)
    gen.manual_seed(3)
    x = torch.from_numpy(I.model_init(d, seed=1)).to(dev)
    xw = x.expand(R3, d).contiguous()
    mem = torch.zeros((R3, d), dtype=torch.float32, device=dev)
    e1 = torch.empty(d, dtype=torch.float32, device=dev)

    def drift():
        for r in range(R3):
            e1.normal_(0.0, 1e-3, generator=gen)
            xw[r].add_(e1)
    out = time_large(torch, B, dev, peak, R3, d, I.k_from_ratio(d, 1, 100), 4, B.QS_RANDK, drift, x, xw, mem, seed=3,
                     steps=steps, warmup=warmup)
    out["workload"] = "Rand_k round: R=16, d=%d, drift N(0,1e-3), Rand_k k=1%% by keyed-hash rank, QSGD s=4" % d
    del x, xw, mem, e1
    torch.cuda.empty_cache()
    return out


def time_config5(torch, B, dev, peak, steps=4, warmup=20):
    """R = 4, d = 2^28, drift N(0, 1e-3) with 0.1% outliers x100, Top_k ratio in {1e-4, 1e-3, 1e-2, 1e-1} x QSGD
    s in {2, 16, 256}: the twelve points."""
    R5, d = 4, 1 << 28
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    x = torch.from_numpy(I.model_init(d, seed=1)).to(dev)
    xw = x.expand(R5, d).contiguous()
    mem = torch.zeros((R5, d), dtype=torch.float32, device=dev)
    e1 = torch.empty(d, dtype=torch.float32, device=dev)
    hit = torch.empty(d, dtype=torch.float32, device=dev)

    def drift():
        for r in range(R5):
            e1.normal_(0.0, 1e-3, generator=gen)
            hit.uniform_(generator=gen)
            e1.mul_(torch.where(hit < 1e-3, 100.0, 1.0))
            xw[r].add_(e1)
    points = []
    for den in (10000, 1000, 100, 10):
        for s in (2, 16, 256):
            p = time_large(torch, B, dev, peak, R5, d, I.k_from_ratio(d, 1, den), s, B.QS_TOPK, drift, x, xw, mem,
                           seed=den + s, steps=steps, warmup=warmup)
            p["ratio"] = 1.0 / den
            points.append(p)
    del x, xw, mem, e1, hit
    torch.cuda.empty_cache()
    return {"workload": "large-d sweep: R=4, d=2^28, drift N(0,1e-3) + 0.1% outliers x100, Top_k x QSGD", "points": points}


def selftest_cpu(rank, world, args):
    """The launch path without a GPU (used by the CPU tests): the ranks that the launcher started meet
    over gloo, every rank reports a made-up time, rank 0 prints the line the real run would print,
    with the slowest rank's time.  No kernel runs and the line says so."""
    import torch
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks(1.0 + rank, torch.device("cpu"))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"selftest": "launch path only: no kernel ran", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms, "value": aggregate_value(1e9, 1, ms, world), "unit": UNIT}))


def launch_ranks(args):
    """--gpus N without a launcher around us: start the N ranks (one process per GPU) the way a launcher
    would, and hand their exit status on.  Refuses when the machine has fewer GPUs than asked for."""
    import socket
    if not args.selftest_cpu:
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} asked for, {have} CUDA device(s) visible\n")
            return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_e2e(torch, ctx, x, xw, mem, wire, bits, drift, d, steps=3):
    """Same round with the state living in pinned host memory: every step copies x, xw, mem to the
    device, runs qs_sync_round and copies x, xw, mem and the records back."""
    hx = torch.empty(x.shape, dtype=x.dtype, pin_memory=True)
    hxw = torch.empty(xw.shape, dtype=xw.dtype, pin_memory=True)
    hmem = torch.empty(mem.shape, dtype=mem.dtype, pin_memory=True)
    hwire = torch.empty(wire.shape, dtype=wire.dtype, pin_memory=True)
    times = []
    for i in range(steps + 1):
        drift()
        hx.copy_(x); hxw.copy_(xw); hmem.copy_(mem)
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        x.copy_(hx, non_blocking=True); xw.copy_(hxw, non_blocking=True); mem.copy_(hmem, non_blocking=True)
        ctx.sync_round(wire, bits_out=bits)
        hx.copy_(x, non_blocking=True); hxw.copy_(xw, non_blocking=True); hmem.copy_(mem, non_blocking=True)
        hwire.copy_(wire, non_blocking=True)
        e.record()
        torch.cuda.synchronize()
        if i:
            times.append(s.elapsed_time(e))
    wire_bytes = int(bits.sum().item() + 7) // 8
    state = 4 * (d + 2 * R * d)
    ms = float(np.mean(times))
    return {"value": min_bytes(d, wire_bytes) / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": state, "d2h_bytes_per_step": state + wire.numel() * 4, "steps": steps}


def cpu_round(x, xw, mem, seg_off, kseg, d):
    """The oracle, as it stands, on the host cores: one round over the given state."""
    from oracle import oracle as O
    cores = os.cpu_count() or 1
    plan = O.Plan(R, d, s=1, sparsifier=O.TOPK, quantizer=O.SIGN_L1, seed=0, offsets=seg_off, kseg=kseg)
    threads = min(cores, R)
    t0 = time.perf_counter()
    out = O.sync_round(plan, 0, x, xw, mem, mode=O.NTH, nthreads=threads)
    dt = time.perf_counter() - t0
    assert out["rc"] == 0
    wire_bytes = int(out["bits"].sum() + 7) // 8
    return {"value": min_bytes(d, wire_bytes) / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "seconds": dt, "sample": f"one round, R={R}, d={d}, nth_element selection, workers spread over {threads} threads"}


def run_reference(args):
    """The CPU oracle as the reference arm, on the bench's own configuration: every step is one full
    round (R = 8, all 25,557,032 coordinates, nth_element selection, workers over the host threads).
    One Laplace drift is drawn once and added before every step (drawing 2 x 10^8 fresh samples per
    step on the host would take longer than the round)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sizes, off, d, seg_off, kseg = workload("flat")
    rng = np.random.default_rng(0)
    x = I.model_init(d, seed=0)
    xw = np.broadcast_to(x, (R, d)).copy()
    mem = np.zeros((R, d), np.float32)
    scales = np.repeat(I.tensor_scales(len(sizes), seed=0), np.diff(off))
    drift = np.empty((R, d), np.float32)
    for r in range(R):
        drift[r] = rng.laplace(0.0, 1.0, d).astype(np.float32) * scales
    times, last = [], None
    for i in range(args.steps + args.warmup):
        xw += drift
        last = cpu_round(x, xw, mem, seg_off, kseg, d)
        if i >= args.warmup:
            times.append(last["seconds"])
    ms = 1e3 * float(np.mean(times))
    value = min_bytes(d, 0) / (ms * 1e-3) / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": headline_config("flat", d, int(kseg.sum())),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"] + "; the same drift added before every step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_config3(args):
    """The Rand_k round of config 3 alone (R = 16, d = 2^26 / --shrink): one JSON line."""
    import torch
    from paper_1906_02367_b200 import binding as B
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peak, peak_src = peak_hbm()
    out = time_config3(torch, B, dev, peak, shrink=args.shrink, steps=max(2, min(args.steps, 20)), warmup=max(3, min(args.warmup, 6)))
    out["peak_source"] = peak_src
    print(json.dumps({"metric": "config3_randk_round", "unit": "ms", **out}))


def run_sweep5(args):
    """Large-d sweep: R = 4, d = 2^28, Gaussian drift N(0, 1e-3) with 0.1% outliers x100, Top_k ratio in
    {1e-4, 1e-3, 1e-2, 1e-1} x QSGD s in {2, 16, 256}.  One JSON line with the twelve points."""
    import torch
    from paper_1906_02367_b200 import binding as B
    R5, d = 4, 1 << 28
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    x = torch.from_numpy(I.model_init(d, seed=1)).to(dev)
    xw = x.expand(R5, d).contiguous()
    mem = torch.zeros((R5, d), dtype=torch.float32, device=dev)
    e1 = torch.empty(d, dtype=torch.float32, device=dev)
    hit = torch.empty(d, dtype=torch.float32, device=dev)

    def drift():
        for r in range(R5):
            e1.normal_(0.0, 1e-3, generator=gen)
            hit.uniform_(generator=gen)
            e1.mul_(torch.where(hit < 1e-3, 100.0, 1.0))
            xw[r].add_(e1)

    peak, peak_src = peak_hbm()
    points = []
    for den in (10000, 1000, 100, 10):
        for s in (2, 16, 256):
            k = I.k_from_ratio(d, 1, den)
            mem.zero_()
            xw.copy_(x.expand(R5, d))
            ctx = B.Context(R5, d, k, s, B.QS_TOPK, B.QS_QSGD, seed=den + s)
            ctx.bind(x, xw, mem)
            wire = ctx.new_wire()
            bits = torch.zeros(R5, dtype=torch.int64, device=dev)
            for _ in range(max(3, args.warmup // 4)):
                drift()
                ctx.sync_round(wire, bits_out=bits)
            st0 = ctx.stats()
            times = []
            for _ in range(max(3, args.steps // 20)):
                drift()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                ctx.sync_round(wire, bits_out=bits)
                b.record()
                torch.cuda.synchronize()
                times.append(a.elapsed_time(b))
            assert ctx.sync_status() == 0, ctx.last_error()
            st1 = ctx.stats()
            ms = float(np.median(times))
            bmin = 16 * R5 * d + 8 * d + 2 * (int(bits.sum().item() + 7) // 8)
            gbs = bmin / (ms * 1e-3) / 1e9
            points.append({"ratio": 1.0 / den, "k": k, "s": s, "ms_per_round": ms, "GBps": gbs,
                           "pct_of_nominal_8TBps": 100 * gbs / NOMINAL_HBM_GBS, "pct_of_measured_copy": 100 * gbs / peak,
                           "worker_elements_per_s": R5 * d / (ms * 1e-3),
                           "fallback_worker_rounds": st1["fallback_worker_rounds"] - st0["fallback_worker_rounds"]})
            ctx.destroy()
            del wire
            torch.cuda.empty_cache()
    print(json.dumps({"metric": METRIC, "unit": UNIT, "config": {"workload": "large-d sweep: R=4, d=2^28, Top_k x QSGD"},
                      "peak_source": peak_src, "points": points}))


def run_async(args):
    """Algorithm 2 on the headline workload: every worker takes local steps all the time, and at each
    step only the workers whose turn it is (gaps drawn uniformly from 1..H, H = 4) synchronise against
    their own anchors.  Not the headline line: one JSON line with the bytes an asynchronous round has
    to move (24 B per active worker coordinate: read xw, mem, anchor, write mem, xw, anchor; 4 B per
    coordinate to read x; records written and read) over the time of the rounds."""
    import torch
    from paper_1906_02367_b200 import binding as B
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    sizes, off, d, seg_off, kseg = workload("flat", args.shrink)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4321)
    per_elem = torch.from_numpy(np.repeat(I.tensor_scales(len(sizes), seed=0), np.diff(off))).to(dev)
    x = torch.from_numpy(I.model_init(d, seed=0)).to(dev)
    xw = x.expand(R, d).contiguous()
    anchors = xw.clone()
    mem = torch.zeros((R, d), dtype=torch.float32, device=dev)
    e1 = torch.empty((R, d), dtype=torch.float32, device=dev)
    e2 = torch.empty_like(e1)

    def drift():
        e1.exponential_(generator=gen)
        e2.exponential_(generator=gen)
        e1.sub_(e2).mul_(per_elem)
        xw.add_(e1)

    T = args.warmup + args.steps
    sched = I.async_schedule(R, T + 1, 4, seed=3)[:T]
    ctx = B.Context(R, d, int(kseg[0]), 1, B.QS_TOPK, B.QS_SIGN_L1, seed=0)
    ctx.bind(x, xw, mem, anchors)
    wire = ctx.new_wire()
    bits = torch.zeros(R, dtype=torch.int64, device=dev)
    peak, peak_src = peak_hbm()
    total_ms, total_bytes, rounds, active = 0.0, 0, 0, 0
    dense_bytes = 0
    for t in range(T):
        drift()
        mask = sched[t]
        n_act = int(mask.sum())
        if n_act == 0:
            continue
        if t == args.warmup:
            ctx.enable_phase_timing(True)
            ctx.phase_timing()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.sync_round(wire, mask=mask, bits_out=bits)
        b.record()
        torch.cuda.synchronize()
        if t >= args.warmup:
            wire_bytes = int((bits.cpu().numpy() * mask).sum() + 7) // 8
            total_ms += a.elapsed_time(b)
            total_bytes += 24 * n_act * d + 4 * d + 2 * wire_bytes
            dense_bytes += 16 * n_act * d
            rounds += 1
            active += n_act
    assert ctx.sync_status() == 0, ctx.last_error()
    phases = ctx.phase_timing()
    st = ctx.stats()
    gbs = total_bytes / (total_ms * 1e-3) / 1e9
    dense_gbs = dense_bytes / (phases["dense_pass"] * 1e-3) / 1e9 if phases["dense_pass"] > 0 else 0.0
    print(json.dumps({
        "metric": "async_round_effective_bandwidth", "value": gbs, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_round": total_ms / max(1, rounds), "rounds_timed": rounds,
        "mean_active_workers": active / max(1, rounds), "higher_is_better": True, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"ResNet-50-shaped asynchronous rounds (Algorithm 2): R=8, d={d}, gaps uniform on 1..4, "
                               "Top_k k=0.1% flat, sign/l1 quantizer, Laplace drift per tensor, memory and anchors carried",
                   "l2_policy": "inputs larger than L2"},
        "pct_of_nominal_8TBps": 100.0 * gbs / NOMINAL_HBM_GBS, "pct_of_measured_copy": 100.0 * gbs / peak,
        "dense_pass": {"achieved": dense_gbs, "peak": peak, "frac": dense_gbs / peak, "peak_source": peak_src,
                       "bytes": "16 B per active worker coordinate"},
        "fallback_worker_rounds": st["fallback_worker_rounds"],
    }))
    ctx.destroy()


def run_step(args):
    """The round with the preceding local step taken inside it (qs_sync_round_step) against the two
    calls it replaces, plain and with momentum, on the headline workload.  Not the headline line.
    Bytes the fused form has to move: the round's 16 R d + 8 d plus the gradient read (4 R d), plus
    the velocity read and written (8 R d) with momentum."""
    import torch
    from paper_1906_02367_b200 import binding as B
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    sizes, off, d, seg_off, kseg = workload("flat", args.shrink)
    gen = torch.Generator(device=dev)
    gen.manual_seed(99)
    per_elem = torch.from_numpy(np.repeat(I.tensor_scales(len(sizes), seed=0), np.diff(off))).to(dev)
    x = torch.from_numpy(I.model_init(d, seed=0)).to(dev)
    xw = x.expand(R, d).contiguous()
    mem = torch.zeros((R, d), dtype=torch.float32, device=dev)
    vel = torch.zeros((R, d), dtype=torch.float32, device=dev)
    grad = torch.empty((R, d), dtype=torch.float32, device=dev)
    e2 = torch.empty_like(grad)
    ctx = B.Context(R, d, int(kseg[0]), 1, B.QS_TOPK, B.QS_SIGN_L1, seed=0)
    ctx.bind(x, xw, mem)
    wire = ctx.new_wire()
    bits = torch.zeros(R, dtype=torch.int64, device=dev)
    peak, peak_src = peak_hbm()

    def new_grad():                    # Laplace(0, b_t) per tensor; eta = 1 makes the step the headline drift
        grad.exponential_(generator=gen)
        e2.exponential_(generator=gen)
        grad.sub_(e2).mul_(per_elem)

    def timed(fn):
        times = []
        for i in range(args.warmup + args.steps):
            new_grad()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                times.append(a.elapsed_time(b))
        assert ctx.sync_status() == 0, ctx.last_error()
        return float(np.mean(times))

    out = {}
    for name, v, mu, extra in (("plain", None, 0.0, 4), ("momentum", vel, 0.5, 12)):
        def separate():
            if v is None:
                ctx.local_step(grad, 1.0)
            else:
                ctx.local_step_momentum(grad, v, 1.0, mu)
            ctx.sync_round(wire, bits_out=bits)
        ms_sep = timed(separate)
        vel.zero_()
        ms_fused = timed(lambda: ctx.sync_round_step(wire, grad, 1.0, vel=v, mu=mu, bits_out=bits))
        vel.zero_()
        bmin = (16 + extra) * R * d + 8 * d + 2 * (int(bits.sum().item() + 7) // 8)
        gbs = bmin / (ms_fused * 1e-3) / 1e9
        out[name] = {"ms_two_calls": ms_sep, "ms_fused": ms_fused, "min_bytes_fused": bmin, "GBps_fused": gbs,
                     "pct_of_nominal_8TBps": 100 * gbs / NOMINAL_HBM_GBS, "pct_of_measured_copy": 100 * gbs / peak}
    print(json.dumps({"metric": "sync_round_with_local_step", "unit": "ms", "steps": args.steps, "warmup": args.warmup,
                      "config": {"workload": f"ResNet-50-shaped round with its local step: R=8, d={d}, Top_k 0.1% flat, sign/l1"},
                      "peak_source": peak_src, "variants": out}))
    ctx.destroy()


def run_sharded(args):
    """The headline job (R = 8 workers) spread over the ranks: each rank holds R / N workers and a
    replica of x, the packed records are all-gathered (NCCL), every rank decodes all of them.  Total
    work is fixed, so this line reports strong scaling; the default line stays N independent replicas."""
    import torch
    import torch.distributed as dist
    from paper_1906_02367_b200 import binding as B, sharded
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sizes, off, d, seg_off, kseg = workload("flat", args.shrink)
    base, count = sharded.partition(R, world)[rank]
    gen = torch.Generator(device=dev)
    gen.manual_seed(777 + rank)
    per_elem = torch.from_numpy(np.repeat(I.tensor_scales(len(sizes), seed=0), np.diff(off))).to(dev)
    x = torch.from_numpy(I.model_init(d, seed=0)).to(dev)
    xw = x.expand(count, d).contiguous()
    mem = torch.zeros((count, d), dtype=torch.float32, device=dev)
    e1 = torch.empty((count, d), dtype=torch.float32, device=dev)
    e2 = torch.empty_like(e1)
    ctx = B.Context(count, d, int(kseg[0]), 1, B.QS_TOPK, B.QS_SIGN_L1, seed=0)
    ctx.bind(x, xw, mem)
    wire = ctx.new_wire()
    gap = {}
    if args.gap_coded:                    # the records cross the all-gather in their gap-coded form
        gap = dict(packed_local=torch.zeros((count, ctx.gap_words()), dtype=torch.int32, device=dev),
                   records=torch.zeros((R, ctx.wire_words()), dtype=torch.int32, device=dev))
    job = sharded.ShardedRound(R, ctx, wire, rank=rank, world=world, **gap)

    def drift():
        e1.exponential_(generator=gen)
        e2.exponential_(generator=gen)
        e1.sub_(e2).mul_(per_elem)
        xw.add_(e1)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        drift()
        job.round(t)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        drift()
        if world > 1:
            dist.barrier()                # the ranks enter the round together, as after a local step
        starts[i].record()
        job.round(args.warmup + i)
        ends[i].record()
    barrier()
    assert ctx.sync_status() == 0, ctx.last_error()
    total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in zip(starts, ends))), dev)
    bmin = 16 * R * d + 8 * d * world                  # every rank updates its own replica of x
    if rank == 0:
        print(json.dumps({
            "metric": "sharded_round_effective_bandwidth", "value": bmin * args.steps / (total_ms * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "strong", "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"ResNet-50-shaped round, R=8 workers over {world} GPU(s), d={d}, Top_k 0.1% flat, sign/l1; "
                                   "separate calls with one all-gather of the records", "workers_per_gpu": count,
                       "exchange": "gap-coded records" if args.gap_coded else "plain records",
                       "words_exchanged_per_record": int(job.exchanged_words)}}))
    ctx.destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="flat", choices=["flat", "per_tensor", "paper_table", "async", "step", "sharded", "config3"])
    ap.add_argument("--shrink", type=int, default=1, help="divide every tensor size (profiling on a small case)")
    ap.add_argument("--sweep5", action="store_true", help="run the d = 2^28 ratio x s sweep instead of the headline workload")
    ap.add_argument("--gap-coded", action="store_true", help="--variant sharded: exchange the records in their gap-coded form")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the other workloads (per tensor, config 3, config 5 sweep)")
    ap.add_argument("--selftest-cpu", action="store_true", help="launch-path self-test without a GPU (gloo, no kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_ranks(args))
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus and args.impl == "ours":
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started {os.environ['WORLD_SIZE']} rank(s)\n")
        sys.exit(2)
    if args.sweep5:
        run_sweep5(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.variant == "async":
        run_async(args)
    elif args.variant == "step":
        run_step(args)
    elif args.variant == "sharded":
        run_sharded(args)
    elif args.variant == "config3":
        run_config3(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
