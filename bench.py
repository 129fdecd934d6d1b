#!/usr/bin/env python
"""Benchmark of the composed affine copy.

One "step" = the layout-transform round trip of the ResNet-50-like activation
tensor bf16 [32,256,56,56]: NCHW -> NHWC, then NHWC -> NCHW, each as ONE
composed copy (two kernel launches per step, 205,520,896 algorithmic bytes).
The maps are composed and planned once, before timing, as a compiler would
(the paper composes at compile time); their host cost is reported separately.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--all-configs]

Prints ONE JSON line.  With N > 1 (torchrun) every rank runs the same per-GPU
workload on its own GPU (batch shards, no exchange: weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2002_12798_b200 import workloads as W  # noqa: E402

METRIC = "effective HBM GB/s (read+write) of composed affine copy"
NOMINAL_PEAK_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the transpose kernel on this workload, mean of the two
# directions, from the ncu captures summarised in profiles/transpose_kernel_c2_*.md.  A captured launch runs alone and
# cold: it reads its 51.4 MB from DRAM, while most of its 51.4 MB output is still in the 126 MB L2 when it ends and
# is written back later, so the counter is below the algorithmic bytes.  Set to None whenever the kernel changes.
TRANSPOSE_C2_DRAM_TRAFFIC = 55_845_000
FALLBACK_PEAK_GBS = 6650.0
SIGNED = {1: np.int8, 2: np.int16, 4: np.int32, 8: np.int64}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback"


# ---------------------------------------------------------------------------
# clocks during the timed region (NVML, read only)
# ---------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
        0x100: "display_clock_setting",
    }

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for bit, name in self.REASONS.items():
                    if bits & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self._nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# ---------------------------------------------------------------------------
def device_bufs(torch, chain, xs, n_sets, device):
    """n_sets independent (inputs, output) buffer sets on the device."""
    es = chain.elem_size
    sets = []
    for _ in range(n_sets):
        ins = [torch.from_numpy(np.ascontiguousarray(x).view(SIGNED[es])).to(device) for x in xs]
        sets.append(ins)
    return sets


def time_plan(torch, plan, in_sets, out_sets, iters, warmup, stream):
    """Average device time of one execute, rotating over the buffer sets (CUDA events on the launch stream).
    `plan` may be a list of plans over the same inputs (the parts of a split): out_sets[i] then holds one output
    per plan, and a step executes them all."""
    n = len(in_sets)
    if isinstance(plan, (list, tuple)):
        bound = [[p.bind(in_sets[i], out_sets[i][k], stream) for k, p in enumerate(plan)] for i in range(n)]
        calls = [lambda b=b: [c() for c in b] for b in bound]
    else:
        calls = [plan.bind(in_sets[i], out_sets[i], stream) for i in range(n)]  # arguments marshalled once
    for i in range(warmup):
        calls[i % n]()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream.synchronize()
    start.record(stream)
    for i in range(iters):
        calls[i % n]()
    stop.record(stream)
    stream.synchronize()
    return start.elapsed_time(stop) * 1e-3 / iters


def whole_job_rate(units_per_rank, elapsed_local, world, dist=None, device=None):
    """Weak scaling without any exchange: every rank moved `units_per_rank`; the job took as long as its slowest
    rank.  Returns (aggregate units per second over all ranks, max elapsed)."""
    elapsed = float(elapsed_local)
    if world > 1:
        import torch

        t = torch.tensor([elapsed], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed = float(t.item())
    return world * units_per_rank / elapsed, elapsed


def run_ours(args):
    import torch

    from oracle import oracle  # CPU-baseline leg only
    from paper_2002_12798_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=device)
    stream = torch.cuda.current_stream(device)
    peak, peak_kind = measured_peak()
    l2 = torch.cuda.get_device_properties(device).L2_cache_size

    fwd_c, inv_c = W.c2_nchw_to_nhwc(), W.c2_nhwc_to_nchw()
    t0 = time.perf_counter()
    fwd_m, inv_m = B.compose_chain(fwd_c), B.compose_chain(inv_c)
    t1 = time.perf_counter()
    fwd_p, inv_p = fwd_m.plan(local, flags=args.plan_flags), inv_m.plan(local, flags=args.plan_flags)
    t2 = time.perf_counter()
    stats = fwd_p.stats()
    bytes_per_launch = stats["bytes_read"] + stats["bytes_written"]
    launches_per_step = fwd_p.stats()["n_launches"] + inv_p.stats()["n_launches"]
    bytes_per_step = 2 * bytes_per_launch

    (x,) = W.make_inputs(fwd_c)
    nbytes = x.nbytes
    n_sets = max(2, -(-4 * l2 // (3 * nbytes)))  # x, y, z per set; all sets together >= 4 x L2
    n_sets += n_sets % 2
    xs = [torch.from_numpy(x.view(np.int16)).to(device) for _ in range(n_sets)]
    ys = [torch.empty_like(xs[0]) for _ in range(n_sets)]
    zs = [torch.empty_like(xs[0]) for _ in range(n_sets)]

    half = n_sets // 2

    fwd_calls = [fwd_p.bind([xs[s]], ys[s], stream) for s in range(n_sets)]  # arguments marshalled once
    inv_calls = [inv_p.bind([ys[s]], zs[s], stream) for s in range(n_sets)]

    def step(i):
        # The inverse runs on the set that the forward pass wrote half a rotation ago, so that its input has
        # left L2 by then (51 MB would otherwise be read back from L2 right after being written).
        s = i % n_sets
        fwd_calls[s]()
        inv_calls[(s + half) % n_sets]()

    for s in range(n_sets):  # every y exists before any inverse reads it
        fwd_p.execute([xs[s]], ys[s], stream)
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()

    # The timed loop is launch-bound (16 us kernels): capture G steps once in a CUDA graph and replay it K / G times.
    # The same amap_execute calls are recorded, so the same kernels run; only the host's launch work disappears.
    graph, G, gstream = None, 0, None
    if not args.no_graph:
        G = max((g for g in range(n_sets, 201, n_sets) if args.steps % g == 0), default=0)
    if G:
        try:
            gstream = torch.cuda.Stream(device)
            gf = [fwd_p.bind([xs[s]], ys[s], gstream) for s in range(n_sets)]
            gi = [inv_p.bind([ys[s]], zs[s], gstream) for s in range(n_sets)]
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gstream):
                for i in range(G):
                    gf[i % n_sets]()
                    gi[(i % n_sets + half) % n_sets]()
        except Exception as exc:  # capture not available: time plain stream launches
            print("CUDA graph capture failed (%s); timing stream launches" % exc, file=sys.stderr)
            graph = None

    def timed(run, on_stream):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        with ClockSampler(local) as clk:
            start.record(on_stream)
            run()
            stop.record(on_stream)
            torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        r, el = whole_job_rate(bytes_per_step * args.steps, start.elapsed_time(stop) * 1e-3, world,
                               dist if world > 1 else None, device)
        return r, el, clk

    def stream_loop():
        for i in range(args.steps):
            step(i)

    stream_rate, stream_elapsed, clocks = timed(stream_loop, stream)
    rate, elapsed, launch_mode = stream_rate, stream_elapsed, "stream launches"
    if graph is not None:
        with torch.cuda.stream(gstream):
            for _ in range(max(1, args.warmup // G)):
                graph.replay()

            def graph_loop():
                for _ in range(args.steps // G):
                    graph.replay()

            rate, elapsed, clocks = timed(graph_loop, gstream)
        launch_mode = "CUDA graph of %d steps replayed %d times" % (G, args.steps // G)
    # parity of the timed buffers: the round trip must give back the input, bit for bit
    for s in range(n_sets):
        if not torch.equal(zs[s], xs[s]):
            raise SystemExit("round trip differs from the input on buffer set %d" % s)

    value = rate / 1e9
    launch_s = elapsed / (args.steps * launches_per_step)
    achieved = bytes_per_launch / launch_s / 1e9

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    hx = torch.from_numpy(x.view(np.int16)).pin_memory()
    hy = torch.empty_like(hx).pin_memory()
    hz = torch.empty_like(hx).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        fwd_p.execute_host([hx], hy, stream.cuda_stream)
        inv_p.execute_host([hy], hz, stream.cuda_stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t3 = time.perf_counter()
    for _ in range(e2e_steps):
        fwd_p.execute_host([hx], hy, stream.cuda_stream)
        inv_p.execute_host([hy], hz, stream.cuda_stream)
    torch.cuda.synchronize()
    e2e_rate, e2e_elapsed = whole_job_rate(bytes_per_step * e2e_steps, time.perf_counter() - t3, world,
                                           dist if world > 1 else None, device)
    if not torch.equal(hz, hx):
        raise SystemExit("host round trip differs from the input")
    e2e_value = e2e_rate / 1e9

    line = {
        "metric": METRIC,
        "value": round(value, 1),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": elapsed / args.steps * 1e3,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "u16",
        "data": "synthetic",
        "config": {
            "workload": "configs[1]: bf16 [32,256,56,56] NCHW->NHWC then NHWC->NCHW, one composed copy each",
            "bytes_per_step": bytes_per_step,
            "launches_per_step": launches_per_step,
            "l2": "inputs larger than L2: rotation over %d buffer sets, %d MB in all (L2 %d MB)"
            % (n_sets, 3 * n_sets * nbytes // 2**20, l2 // 2**20),
            "parallelism": "replicas (batch shards, no exchange)" if world > 1 else "single GPU",
            "launch_mode": launch_mode,
        },
        "pct_of_nominal_8TBs": round(100 * value / world / NOMINAL_PEAK_GBS, 1),
        "roofline": {
            "bound": "hbm",
            "kernel": fwd_p.piece_kernels()[0],
            "achieved": round(achieved, 1),
            "peak": peak,
            "peak_kind": "of " + peak_kind,
            "unit": "GB/s",
            "frac": round(achieved / peak, 4),
            "traffic": TRANSPOSE_C2_DRAM_TRAFFIC,
            "traffic_note": "one cold launch under ncu: 51.5 MB read, 4.4 MB written (the output stays in L2 past the kernel's end)",
            "bytes_per_launch": bytes_per_launch,
            "us_per_launch": round(launch_s * 1e6, 2),
        },
        "e2e": {
            "value": round(e2e_value, 2),
            "unit": "GB/s",
            "h2d_bytes_per_step": 2 * nbytes,
            "d2h_bytes_per_step": 2 * nbytes,
            "steps": e2e_steps,
        },
        "gpu_launches": args.steps * launches_per_step,
        "stream_launches": {
            "value": round(stream_rate / 1e9, 1),
            "unit": "GB/s",
            "us_per_launch": round(stream_elapsed / (args.steps * launches_per_step) * 1e6, 2),
            "note": "the same K steps as individual amap_execute calls on the stream, no graph",
        },
        "clocks": clocks.summary(),
        "host_compose_ms": round((t1 - t0) * 1e3, 3),
        "host_plan_ms": round((t2 - t1) * 1e3, 3),
    }

    if rank == 0 and world == 1:
        line["cpu_baseline"] = cpu_baseline(oracle, fwd_c, inv_c, x, bytes_per_step)
        if args.all_configs:
            line["all_configs"] = all_configs(torch, B, device, stream, l2, peak, flags=args.plan_flags)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(oracle, fwd_c, inv_c, x, bytes_per_step, budget_s=20.0):
    """The oracle, as it stands, on the host cores: the same round trip, repeated within a time budget."""
    cores = os.cpu_count() or 1
    reps, t0 = 0, time.perf_counter()
    while True:
        y = oracle.run_chain(fwd_c, [x], nt=cores)
        z = oracle.run_chain(inv_c, [y], nt=cores)
        reps += 1
        if time.perf_counter() - t0 > min(budget_s, 5.0) or reps >= 5:
            break
    dt = (time.perf_counter() - t0) / reps
    assert np.array_equal(z, x)
    return {
        "value": round(bytes_per_step / dt / 1e9, 3),
        "unit": "GB/s",
        "cores": cores,
        "kind": "oracle",
        "sample": "the whole step (both directions, all 32 images), %d repetitions, %.2f s each" % (reps, dt),
    }


def all_configs(torch, B, device, stream, l2, peak, only=None, iters=None, warmup=5, flags=0):
    """Every large configuration, each timed the same way (device time per launch, rotating buffers)."""
    out = {}
    configs = dict(W.full_configs())
    # the practical ceiling: a same-kernel plain copy (a reshape composes to one contiguous piece)
    configs["plain_copy_512MB"] = W.Chain(
        name="plain_copy", dtype="bf16", inputs=[[1 << 28]], ops=[{"kind": "reshape", "src": 0, "shape": [1 << 14, 1 << 14]}]
    )
    # operators beyond the five configurations: nearest-neighbour upsampling (repeat on H and W: every input byte
    # is read once and written four times) and a fused QKV tensor cut in three, each part to [B, heads, S, D]
    # (split: one composed copy per part, three launches over the same input)
    configs["upsample2x"] = W.upsample_nhwc()
    # layout changes whose rows are not 16-byte aligned on one side (Inception's 35x35x288 maps, ResNet's 14x14x1024):
    # the realigning, shifted-destination and narrow-unit transpose kernels
    configs["odd35_fwd"] = W.c2_nchw_to_nhwc(N=64, C=288, H=35, W=35)
    configs["odd35_inv"] = W.c2_nhwc_to_nchw(N=64, C=288, H=35, W=35)
    configs["map14_inv"] = W.c2_nhwc_to_nchw(N=64, C=1024, H=14, W=14)
    configs["qkv_split"] = [W.qkv_split(part=k) for k in range(3)]
    for name, chain in configs.items():
        if name == "c1" or (only and name != only):
            continue
        parts = chain if isinstance(chain, list) else [chain]
        chain = parts[0]
        xs = W.make_inputs(chain)
        maps = [B.compose_chain(c) for c in parts]
        plans = [m.plan(device.index, flags=flags) for m in maps]
        sts = [p.stats() for p in plans]
        st, m, plan = sts[0], maps[0], plans[0]
        total = sum(t["bytes_read"] + t["bytes_written"] for t in sts)
        es = chain.elem_size
        foot = sum(x.nbytes for x in xs) + sum(mm.out_numel for mm in maps) * es
        n_sets = max(2, min(8, -(-4 * l2 // foot)))
        ins = [[torch.from_numpy(x.view(SIGNED[es])).to(device) for x in xs] for _ in range(n_sets)]
        outs = [[torch.empty(mm.out_numel, dtype=ins[0][0].dtype, device=device) for mm in maps] for _ in range(n_sets)]
        if len(parts) == 1:
            outs = [o[0] for o in outs]
        n_it = iters or max(20, min(2000, int(0.25 / (total / 6.0e12))))
        # best of two passes: the first also carries the clock ramp after the idle set-up
        sec = min(time_plan(torch, plans if len(parts) > 1 else plan, ins, outs, n_it, warmup, stream) for _ in range(2))
        out[name] = {
            "gbs": round(total / sec / 1e9, 1),
            "us": round(sec * 1e6, 2),
            "bytes": total,
            "pct_of_nominal_8TBs": round(100 * total / sec / 1e9 / NOMINAL_PEAK_GBS, 1),
            "frac_of_measured_copy": round(total / sec / 1e9 / peak, 3),
            "kernels": {k: sum(t["kernels"][k] for t in sts) for k in st["kernels"]},
            "launches": sum(t["n_launches"] for t in sts),
        }
        # the chain before data-movement elimination: one launch and one temporary per operator, same kernels
        if len(chain.ops) > 1 and len(parts) == 1:
            uplan = B.compose_chain(chain, B.COMPOSE_NO_FUSE).plan(device.index, flags=flags)
            usec = time_plan(torch, uplan, ins, outs, max(10, n_it // 4), warmup, stream)
            ust = uplan.stats()
            out[name]["unfused"] = {
                "us": round(usec * 1e6, 2),
                "gbs_effective": round(total / usec / 1e9, 1),
                "bytes_moved": ust["bytes_read"] + ust["bytes_written"],
                "stages": ust["n_stages"],
                "slowdown": round(usec / sec, 2),
            }
            del uplan
        del ins, outs
        torch.cuda.empty_cache()
    return out


def run_reference(args):
    """The CPU oracle on the host cores, on the same workload, metric and unit (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle

    fwd_c, inv_c = W.c2_nchw_to_nhwc(), W.c2_nhwc_to_nchw()
    # a step = the round trip on a bounded sample: 4 of the 32 images (the operators are independent per image)
    sample_n = 4
    fs, is_ = W.c2_nchw_to_nhwc(N=sample_n), W.c2_nhwc_to_nchw(N=sample_n)
    (x,) = W.make_inputs(fs)
    cores = os.cpu_count() or 1
    bytes_per_step = 4 * x.nbytes
    for _ in range(min(args.warmup, 3)):
        oracle.run_chain(is_, [oracle.run_chain(fs, [x], nt=cores)], nt=cores)
    steps = min(args.steps, 50)
    t0 = time.perf_counter()
    for _ in range(steps):
        z = oracle.run_chain(is_, [oracle.run_chain(fs, [x], nt=cores)], nt=cores)
    dt = time.perf_counter() - t0
    assert np.array_equal(z, x)
    value = bytes_per_step * steps / dt / 1e9
    sample = "each step = the round trip on %d of the 32 images (%d bytes moved), %d steps" % (sample_n, bytes_per_step, steps)
    print(
        json.dumps(
            {
                "impl": "reference",
                "metric": METRIC,
                "value": round(value, 3),
                "unit": "GB/s",
                "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
                "steps": steps,
                "warmup": min(args.warmup, 3),
                "ms_per_step": dt / steps * 1e3,
                "higher_is_better": True,
                "scaling": "weak",
                "vs_baseline": None,
                "dtype": "u16",
                "data": "synthetic",
                "config": {"workload": "configs[1]: bf16 [32,256,56,56] NCHW->NHWC then NHWC->NCHW (CPU oracle, operator by operator)"},
                "cpu_baseline": {"value": round(value, 3), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": round(value, 3), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            }
        )
    )


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time individual stream launches only")
    ap.add_argument("--all-configs", action="store_true", help="also time configurations 3, 4, 5 (adds about a minute)")
    ap.add_argument("--plan-flags", type=int, default=0, help="amap_plan_opts.flags for every plan (1: no programmatic dependent launch, 2: no L2 prefetch)")
    ap.add_argument("--config", default=None, help="time ONE configuration's kernel loop only (for profiler captures) and print its figures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.config:
        import torch

        from paper_2002_12798_b200 import binding as B

        device = torch.device("cuda", 0)
        torch.cuda.set_device(device)
        peak, _ = measured_peak()
        l2 = torch.cuda.get_device_properties(device).L2_cache_size
        print(json.dumps(all_configs(torch, B, device, torch.cuda.current_stream(device), l2, peak, args.config, args.steps, args.warmup, args.plan_flags)))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
