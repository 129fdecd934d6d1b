#!/usr/bin/env python
"""Benchmark of the composed affine copy.

One "step" = the layout-transform round trip of the ResNet-50-like activation
tensor bf16 [32,256,56,56]: NCHW -> NHWC, then NHWC -> NCHW, each as ONE
composed copy (two kernel launches per step, 205,520,896 algorithmic bytes).
The maps are composed and planned once, before timing, as a compiler would
(the paper composes at compile time); their host cost is reported separately.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--all-configs]

The K-step region is timed R >= 10 times back to back (one CUDA-event pair per
repetition, no host synchronisation in between, so that the GPU reaches the
clocks it holds under sustained load); `ms_per_step` and `value` are the MEDIAN
repetition, best and worst are reported beside it.  The same line carries a
table with every large configuration (each timed the same way, with a same-size
plain copy and the view-aware torch chain beside it).

Prints ONE JSON line.  With N > 1 (torchrun) every rank runs the same per-GPU
workload on its own GPU (batch shards, no exchange: weak scaling).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
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
FALLBACK_PEAK_GBS = 6650.0
SIGNED = {1: np.int8, 2: np.int16, 4: np.int32, 8: np.int64}

# DRAM traffic of the dominant kernel in steady state: dram__bytes_read.sum + dram__bytes_write.sum per launch, the
# mean over consecutive launches of the timed loop on its rotating buffers (ncu, counters only, caches left as the
# previous launch leaves them).  Valid only for the kernel source it was taken on: the digest below is that of the
# kernel sources at capture time, and the line reports traffic = null when they have changed since.
STEADY_STATE_TRAFFIC = {
    "bytes_per_launch": 101_929_856,
    "kernel_digest": "0c8db0a62d0ee835",
    "note": "ncu counters over 16 consecutive launches of the timed loop, caches as the previous launch leaves them: "
            "51.55 MB read + 50.38 MB written per launch, 0.992 of the algorithmic bytes",
}
KERNEL_SOURCES = ("kernels.cuh", "device_table.hpp", "plan_execute.cu")


def kernel_digest():
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2002_12798_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


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
    REJECT = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.power, self.reasons, self.max_mhz = [], [], set(), None
        self.period = period_s
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
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
                bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for bit, name in self.REASONS.items():
                    if bits & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

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
        s = self.samples
        return {
            "sm_mhz": statistics.median(s) if s else None,
            "sm_mhz_min": min(s) if s else None,
            "sm_max_mhz": self.max_mhz,
            "power_w": round(statistics.median(self.power), 1) if self.power else None,
            "reasons": sorted(self.reasons),
            "samples": len(s),
            "rejected": any(r in self.reasons for r in self.REJECT),
        }


# ---------------------------------------------------------------------------
# timing
# ---------------------------------------------------------------------------
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


def rep_stats(rep_seconds, per_rep_units=1):
    """Median / best / worst of the repetitions, per unit (a step or a launch)."""
    v = sorted(s / per_rep_units for s in rep_seconds)
    med = statistics.median(v)
    return {"n": len(v), "median": med, "best": v[0], "worst": v[-1], "spread_pct": round(100 * (v[-1] - v[0]) / med, 2)}


def time_repetitions(torch, run_rep, reps, stream, world=1, dist=None, device=None, sampler=None):
    """Runs `run_rep()` (which enqueues one repetition on `stream`) `reps` times back to back with a CUDA event
    between repetitions and no host synchronisation inside; barrier + synchronize on both sides.  Returns the
    per-repetition device times in seconds (max over ranks)."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ctx = sampler if sampler is not None else _Null()
    with ctx:
        ev[0].record(stream)
        for r in range(reps):
            run_rep()
            ev[r + 1].record(stream)
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    secs = [ev[r].elapsed_time(ev[r + 1]) * 1e-3 for r in range(reps)]
    if world > 1:
        t = torch.tensor(secs, dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        secs = [float(x) for x in t.tolist()]
    return secs


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def measure_calls(torch, calls, stream, bytes_per_call, device_index, reps=10, rep_seconds=0.02, warmup=5, max_launches=4000):
    """Median-of-`reps` device time of one call, rotating over `calls` (one per buffer set), with the clocks seen."""
    n = len(calls)
    for i in range(max(warmup, n)):
        calls[i % n]()
    torch.cuda.synchronize()
    est = bytes_per_call / 6.0e12
    per_rep = max(20, min(max_launches, int(rep_seconds / est)))
    per_rep += (-per_rep) % n  # whole rotations
    state = {"i": 0}

    def run_rep():
        i0 = state["i"]
        for i in range(per_rep):
            calls[(i0 + i) % n]()
        state["i"] = i0 + per_rep

    run_rep()  # one untimed repetition: clocks ramp up after the idle set-up
    sampler = ClockSampler(device_index)
    secs = time_repetitions(torch, run_rep, reps, stream, sampler=sampler)
    st = rep_stats(secs, per_rep)
    clk = sampler.summary()
    return {
        "us": round(st["median"] * 1e6, 2),
        "us_best": round(st["best"] * 1e6, 2),
        "us_worst": round(st["worst"] * 1e6, 2),
        "gbs": round(bytes_per_call / st["median"] / 1e9, 1),
        "reps": reps,
        "launches_per_rep": per_rep,
        "sm_mhz": clk["sm_mhz"],
        "reasons": clk["reasons"],
    }


def rate_fields(row, peak):
    row["pct_of_nominal_8TBs"] = round(100 * row["gbs"] / NOMINAL_PEAK_GBS, 1)
    row["frac_of_measured_copy"] = round(row["gbs"] / peak, 3)
    return row


# ---------------------------------------------------------------------------
# the configurations beside the headline workload
# ---------------------------------------------------------------------------
TABLE_CONFIGS = ("c2_fwd", "c2_inv", "c3", "c3_merge", "c4", "c5", "odd35_fwd", "odd35_inv", "map14_inv", "map7_inv",
                 "map71_fwd", "map71_inv", "map14_c1020_inv")


def bench_configs():
    configs = dict(W.full_configs())
    # the practical ceiling: a same-kernel plain copy (a reshape composes to one contiguous piece)
    configs["plain_copy_512MB"] = plain_copy_chain(1 << 28)
    # operators beyond the five configurations: nearest-neighbour upsampling (repeat on H and W: every input byte
    # is read once and written four times) and a fused QKV tensor cut in three, each part to [B, heads, S, D]
    configs["upsample2x"] = W.upsample_nhwc()
    # layout changes whose rows are not 16-byte aligned on one side.  Rows short enough for a panel (Inception's
    # 35x35x288 maps, ResNet's 14x14x1024 and 7x7x2048): the flat-source and flat-destination transposes
    configs["odd35_fwd"] = W.c2_nchw_to_nhwc(N=64, C=288, H=35, W=35)
    configs["odd35_inv"] = W.c2_nhwc_to_nchw(N=64, C=288, H=35, W=35)
    configs["map14_inv"] = W.c2_nhwc_to_nchw(N=64, C=1024, H=14, W=14)
    configs["map7_inv"] = W.c2_nhwc_to_nchw(N=128, C=2048, H=7, W=7)
    # longer rows (71x71x192 maps): the realigning and shifted-destination kernels; a channel count that is no
    # multiple of 16 bytes (14x14x1020): 8-byte units
    configs["map71_fwd"] = W.c2_nchw_to_nhwc(N=32, C=192, H=71, W=71)
    configs["map71_inv"] = W.c2_nhwc_to_nchw(N=32, C=192, H=71, W=71)
    configs["map14_c1020_inv"] = W.c2_nhwc_to_nchw(N=64, C=1020, H=14, W=14)
    configs["qkv_split"] = [W.qkv_split(part=k) for k in range(3)]   # three maps, three launches
    configs["qkv_split_one_launch"] = W.qkv_split_all()               # one map with three outputs, one launch
    return configs


def plain_copy_chain(numel, dtype="bf16"):
    n = int(numel)
    f = 1
    for c in (1 << 14, 1 << 10, 256, 16, 2):
        if n % c == 0:
            f = c
            break
    return W.Chain(name="plain_copy", dtype=dtype, inputs=[[n]], ops=[{"kind": "reshape", "src": 0, "shape": [n // f, f]}])


def torch_view_chain(torch, name, chain):
    """The same result with torch's own operators, views kept as views (reshape / slice / permute cost nothing until
    a copy is forced): the strong library baseline on the same GPU.  Returns fn(list of typed tensors) -> tensor."""
    F = torch.nn.functional
    if name in ("c2_fwd", "odd35_fwd", "map71_fwd"):
        return lambda xs: xs[0].permute(0, 2, 3, 1).contiguous()
    if name in ("c2_inv", "odd35_inv", "map14_inv", "map7_inv", "map71_inv", "map14_c1020_inv"):
        return lambda xs: xs[0].permute(0, 3, 1, 2).contiguous()
    if name == "c3":
        B_, S, HD = chain.inputs[0]
        keep = chain.ops[2]["stop"][2]
        heads = chain.ops[0]["shape"][2]
        return lambda xs: torch.cat([x.view(B_, S, heads, HD // heads).transpose(1, 2)[:, :, :keep] for x in xs], 2)
    if name == "c3_merge":
        B_, heads, S, D = chain.inputs[0]
        return lambda xs: xs[0].transpose(1, 2).reshape(B_, S, heads * D)
    if name == "c4":
        return lambda xs: torch.cat([F.pad(x, (1, 1, 1, 1)) for x in xs], 1).permute(0, 2, 3, 1).contiguous()
    if name == "c5":
        N, H, Wd, C = chain.inputs[0]
        op = chain.ops[0]
        k, s, p = op["kh"], op["stride"], op["pad"]
        Ho, Wo = (H + 2 * p - k) // s + 1, (Wd + 2 * p - k) // s + 1

        def f(xs):
            cols = F.unfold(xs[0].permute(0, 3, 1, 2), kernel_size=k, padding=p, stride=s)  # [N, C*k*k, Ho*Wo], (c, r, s)
            return cols.view(N, C, k * k, Ho * Wo).permute(0, 3, 2, 1).reshape(N * Ho * Wo, k * k * C)

        return f
    if name == "upsample2x":
        return lambda xs: xs[0].repeat_interleave(2, dim=1).repeat_interleave(2, dim=2)
    return None


def typed(torch, t, dtype_name):
    return t.view({"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}.get(dtype_name, t.dtype))


class Case:
    """One configuration set up on the device: composed maps, plans, rotating buffer sets and the bound calls."""

    def __init__(self, torch, B, chain, device, stream, l2, flags=0):
        self.parts = chain if isinstance(chain, list) else [chain]
        self.chain = self.parts[0]
        es = self.es = self.chain.elem_size
        self.xs = W.make_inputs(self.chain)
        self.maps = [B.compose_chain(c, outputs=c.meta.get("outputs")) for c in self.parts]
        self.plans = [m.plan(device.index, flags=flags) for m in self.maps]
        self.stats = [p.stats() for p in self.plans]
        self.total = sum(t["bytes_read"] + t["bytes_written"] for t in self.stats)
        foot = sum(x.nbytes for x in self.xs) + sum(sum(m.out_numels) for m in self.maps) * es
        self.n_sets = n_sets = max(2, min(8, -(-4 * l2 // foot)))
        self.ins = [[torch.from_numpy(x.view(SIGNED[es])).to(device) for x in self.xs] for _ in range(n_sets)]
        dt = self.ins[0][0].dtype
        # per buffer set and per map: one tensor, or a list of them when the map has several outputs
        self.outs = [[[torch.empty(n, dtype=dt, device=device) for n in m.out_numels] if len(m.out_numels) > 1
                      else torch.empty(m.out_numel, dtype=dt, device=device) for m in self.maps] for _ in range(n_sets)]
        bound = [[p.bind(self.ins[i], self.outs[i][k], stream) for k, p in enumerate(self.plans)] for i in range(n_sets)]
        self.calls = [(lambda b=b: [c() for c in b]) if len(b) > 1 else b[0] for b in bound]
        self.launches = sum(t["n_launches"] for t in self.stats)
        self.single = len(self.parts) == 1 and len(self.maps[0].out_numels) == 1


def config_rows(torch, B, device, stream, l2, peak, names, flags=0, extras=False, oracle=None, reps=10):
    """One row per configuration: the composed copy (median of `reps` repetitions), a plain copy of the same number
    of bytes with the library's own copy kernel, and the view-aware torch chain.  With `extras`: the unfused
    operator-by-operator chain on the GPU and the CPU oracle (single thread and all cores), whose output the GPU
    result is compared with."""
    out = {}
    configs = bench_configs()
    for name in names:
        case = Case(torch, B, configs[name], device, stream, l2, flags)
        chain, es, xs, total, ins, outs, n_sets = case.chain, case.es, case.xs, case.total, case.ins, case.outs, case.n_sets
        sts = case.stats
        row = rate_fields(measure_calls(torch, case.calls, stream, total, device.index, reps=reps), peak)
        row["bytes"] = total
        row["launches"] = case.launches
        row["kernels"] = {k: sum(t["kernels"][k] for t in sts) for k in sts[0]["kernels"]}
        row["launch_kernels"] = [l["kernel"] for p in case.plans for l in p.launches()]
        row["buffer_sets"] = n_sets
        ours = outs[0][0].clone() if case.single else None

        # the library's own plain copy of the same number of bytes (practical ceiling at this size)
        if name != "plain_copy_512MB":
            cchain = plain_copy_chain(total // (2 * es), chain.dtype)
            cplan = B.compose_chain(cchain).plan(device.index, flags=flags)
            cn = total // (2 * es)
            csets = max(2, min(8, -(-4 * l2 // total)))
            cin = [torch.empty(cn, dtype=ins[0][0].dtype, device=device) for _ in range(csets)]
            cout = [torch.empty(cn, dtype=ins[0][0].dtype, device=device) for _ in range(csets)]
            ccalls = [cplan.bind([cin[i]], cout[i], stream) for i in range(csets)]
            c = measure_calls(torch, ccalls, stream, total, device.index, reps=reps)
            row["plain_copy_same_bytes"] = {"us": c["us"], "gbs": c["gbs"], "ratio": round(row["us"] / c["us"], 3)}
            del cin, cout, ccalls, cplan

        # torch's own operators on the same GPU, views kept as views
        fn = torch_view_chain(torch, name, chain) if case.single else None
        if fn is not None:
            tin = [[typed(torch, t.view(list(shape)), chain.dtype) for t, shape in zip(s, chain.inputs)] for s in ins]
            got = fn(tin[0])
            same = bool(torch.equal(got.contiguous().view(ins[0][0].dtype).reshape(-1), ours))
            del got
            tcalls = [lambda s=s: fn(s) for s in tin]
            with torch.cuda.stream(stream):
                t = measure_calls(torch, tcalls, stream, total, device.index, reps=reps, max_launches=400)
            row["torch_view_chain"] = {"us": t["us"], "gbs_effective": t["gbs"], "slowdown": round(t["us"] / row["us"], 2),
                                       "same_bits": same}
            del tin, tcalls

        if extras and len(chain.ops) > 1 and case.single:
            # the chain before data-movement elimination: one launch and one temporary per operator, same kernels
            uplan = B.compose_chain(chain, B.COMPOSE_NO_FUSE).plan(device.index, flags=flags)
            ucalls = [uplan.bind(ins[i], outs[i][0], stream) for i in range(n_sets)]
            u = measure_calls(torch, ucalls, stream, total, device.index, reps=reps, max_launches=400)
            ust = uplan.stats()
            row["unfused"] = {"us": u["us"], "gbs_effective": u["gbs"], "bytes_moved": ust["bytes_read"] + ust["bytes_written"],
                              "stages": ust["n_stages"], "slowdown": round(u["us"] / row["us"], 2)}
            del uplan, ucalls
        if extras and oracle is not None and case.single:
            row["cpu_oracle"] = oracle_row(oracle, chain, xs, total, ours.cpu().numpy())
        out[name] = row
        del ins, outs, case, ours
        torch.cuda.empty_cache()
    return out


def consumer_rows(torch, B, device, stream, l2, names=("c5", "c3"), flags=0, reps=10):
    """The composed map handed to the CONSUMER instead of being run as a copy: a row-sum kernel that reads the
    inputs through the map, against the same kernel reading a materialised result (copy first, then reduce)."""
    out = {}
    configs = bench_configs()
    for name in names:
        case = Case(torch, B, configs[name], device, stream, l2, flags)
        m, es, n_sets = case.maps[0], case.es, case.n_sets
        rows = {"c5": m.out_numel // (9 * 128), "c3": m.out_numel // 128}.get(name, m.out_numel // 128)
        cols = m.out_numel // rows
        sums = [torch.empty(rows, dtype=torch.int32, device=device) for _ in range(n_sets)]
        fused = [m.bind_consume_row_sums(case.ins[i], rows, cols, sums[i], stream) for i in range(n_sets)]
        ident = B.compose_chain(plain_copy_chain(m.out_numel, case.chain.dtype))
        reduce_ = [ident.bind_consume_row_sums([case.outs[i][0]], rows, cols, sums[i], stream) for i in range(n_sets)]
        copy_then = [lambda i=i: (case.calls[i](), reduce_[i]()) for i in range(n_sets)]
        st = case.stats[0]
        fused_bytes = st["bytes_read"] + 4 * rows
        unfused_bytes = st["bytes_read"] + 2 * st["bytes_written"] + 4 * rows
        f = measure_calls(torch, fused, stream, fused_bytes, device.index, reps=reps, max_launches=1000)
        ref = sums[0].clone()
        u = measure_calls(torch, copy_then, stream, unfused_bytes, device.index, reps=reps, max_launches=1000)
        out[name] = {
            "what": "uint32 row sums of the chain's result [%d, %d]" % (rows, cols),
            "through_the_map": {"us": f["us"], "bytes_moved": fused_bytes},
            "copy_then_reduce": {"us": u["us"], "bytes_moved": unfused_bytes},
            "speedup": round(u["us"] / f["us"], 2),
            "same_sums": bool(torch.equal(ref, sums[0])),
        }
        del case, sums, fused, reduce_, copy_then
        torch.cuda.empty_cache()
    return out


def oracle_row(oracle, chain, xs, total_bytes, gpu_out):
    """The oracle on one configuration: single thread and all cores, its output compared with the GPU's."""
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    want = oracle.run_chain(chain, xs, nt=cores)
    t1 = time.perf_counter()
    same = bool(np.array_equal(want.reshape(-1).view(gpu_out.dtype), gpu_out))
    row = {"cores": cores, "s_all_cores": round(t1 - t0, 3), "gbs_all_cores": round(total_bytes / (t1 - t0) / 1e9, 3),
           "gpu_matches_oracle": same}
    t0 = time.perf_counter()
    oracle.run_chain(chain, xs, nt=1)
    t1 = time.perf_counter()
    row["s_single_thread"] = round(t1 - t0, 3)
    row["gbs_single_thread"] = round(total_bytes / (t1 - t0) / 1e9, 3)
    return row


# ---------------------------------------------------------------------------
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
    dist = None
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
    K = args.steps

    # The timed loop is launch-bound (16 us kernels): capture G steps once in a CUDA graph and replay it K / G times
    # per repetition.  The same amap_execute calls are recorded, so the same kernels run; only the host's launch work
    # disappears.
    graph, G, gstream = None, 0, None
    if not args.no_graph:
        G = max((g for g in range(n_sets, 201, n_sets) if K % g == 0), default=0)
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

    # How many repetitions of the K-step region: at least 10, and enough of them that the timed region lasts
    # --min-seconds, so that the clock sampler sees the state the GPU settles in under load.
    est_step = bytes_per_step / 6.0e12
    reps = max(args.reps, min(5000, int(math.ceil(args.min_seconds / (K * est_step)))))

    def stream_rep():
        for i in range(K):
            step(i)

    # individual stream launches (no graph): the figure a caller sees who enqueues every copy himself
    s_reps = max(10, min(reps, int(math.ceil(0.3 / (K * est_step)))))
    stream_secs = time_repetitions(torch, stream_rep, s_reps, stream, world, dist, device)
    stream_st = rep_stats(stream_secs, K)
    if graph is not None:
        with torch.cuda.stream(gstream):
            def graph_rep():
                for _ in range(K // G):
                    graph.replay()

            # untimed: the warm-up steps again as graph replays, then a heat-up stretch of the same length as the
            # timed region's first third
            for _ in range(max(1, args.warmup // G) + max(1, reps // 3) * (K // G)):
                graph.replay()
            sampler = ClockSampler(local)
            secs = time_repetitions(torch, graph_rep, reps, gstream, world, dist, device, sampler)
        launch_mode = "CUDA graph of %d steps replayed %d times per repetition" % (G, K // G)
    else:
        sampler = ClockSampler(local)
        secs = time_repetitions(torch, stream_rep, reps, stream, world, dist, device, sampler)
        launch_mode = "stream launches"
    st = rep_stats(secs, K)
    clocks = sampler.summary()
    # parity of the timed buffers: the round trip must give back the input, bit for bit (the forward result is
    # compared with the oracle's in the CPU-baseline leg below)
    for s in range(n_sets):
        if not torch.equal(zs[s], xs[s]):
            raise SystemExit("round trip differs from the input on buffer set %d" % s)

    sec_per_step = st["median"]
    value = world * bytes_per_step / sec_per_step / 1e9
    launch_s = sec_per_step / launches_per_step
    achieved = bytes_per_launch / launch_s / 1e9

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    hx = torch.from_numpy(x.view(np.int16)).pin_memory()
    hy = torch.empty_like(hx).pin_memory()
    hz = torch.empty_like(hx).pin_memory()
    e2e_steps = max(3, min(K, 10))
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
    e2e_rate, e2e_elapsed = whole_job_rate(bytes_per_step * e2e_steps, time.perf_counter() - t3, world, dist, device)
    if not torch.equal(hz, hx):
        raise SystemExit("host round trip differs from the input")
    e2e_value = e2e_rate / 1e9

    digest = kernel_digest()
    traffic_valid = STEADY_STATE_TRAFFIC["kernel_digest"] == digest and STEADY_STATE_TRAFFIC["bytes_per_launch"]
    line = {
        "metric": METRIC,
        "value": round(value, 1),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": K,
        "warmup": args.warmup,
        "ms_per_step": sec_per_step * 1e3,
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
        "repetitions": {
            "n": st["n"],
            "what": "the K-step region, back to back, one CUDA-event pair each; ms_per_step and value are the median",
            "ms_per_step_median": st["median"] * 1e3,
            "ms_per_step_best": st["best"] * 1e3,
            "ms_per_step_worst": st["worst"] * 1e3,
            "spread_pct": st["spread_pct"],
            "value_best": round(world * bytes_per_step / st["best"] / 1e9, 1),
            "value_worst": round(world * bytes_per_step / st["worst"] / 1e9, 1),
            "timed_region_s": round(sum(secs), 3),
        },
        "pct_of_nominal_8TBs": round(100 * value / world / NOMINAL_PEAK_GBS, 1),
        "roofline": {
            "bound": "hbm",
            "kernel": "amap_transpose_one<2, unsigned int> (%s)" % fwd_p.piece_kernels()[0],
            "achieved": round(achieved, 1),
            "peak": peak,
            "peak_kind": "of " + peak_kind,
            "unit": "GB/s",
            "frac": round(achieved / peak, 4),
            "traffic": STEADY_STATE_TRAFFIC["bytes_per_launch"] if traffic_valid else None,
            "traffic_note": STEADY_STATE_TRAFFIC["note"] if traffic_valid else "null: the kernel sources changed since the counters were taken (digest %s)" % digest,
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
        "gpu_launches": reps * K * launches_per_step,
        "stream_launches": {
            "value": round(world * bytes_per_step / stream_st["median"] / 1e9, 1),
            "unit": "GB/s",
            "us_per_launch": round(stream_st["median"] / launches_per_step * 1e6, 2),
            "repetitions": stream_st["n"],
            "note": "the same K steps as individual amap_execute calls on the stream, no graph; median repetition",
        },
        "clocks": clocks,
        "host_compose_ms": round((t1 - t0) * 1e3, 3),
        "host_plan_ms": round((t2 - t1) * 1e3, 3),
    }

    if rank == 0 and world == 1:
        line["cpu_baseline"] = cpu_baseline(oracle, fwd_c, inv_c, x, bytes_per_step, ys[0].cpu().numpy().view(np.uint16))
        del xs, ys, zs, fwd_calls, inv_calls, graph
        torch.cuda.empty_cache()
        names = list(TABLE_CONFIGS)
        if args.all_configs:
            names += ["upsample2x", "qkv_split", "qkv_split_one_launch", "plain_copy_512MB"]
        if not args.no_table:
            line["configs"] = config_rows(torch, B, device, stream, l2, peak, names, flags=args.plan_flags,
                                          extras=args.all_configs, oracle=oracle, reps=max(10, args.reps))
            line["consumer"] = consumer_rows(torch, B, device, stream, l2, flags=args.plan_flags, reps=max(10, args.reps))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(oracle, fwd_c, inv_c, x, bytes_per_step, gpu_forward=None, budget_s=20.0):
    """The oracle, as it stands, on the host cores: the same round trip, repeated within a time budget.  Its
    forward result is also what the GPU's timed forward buffer is compared with."""
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
    out = {
        "value": round(bytes_per_step / dt / 1e9, 3),
        "unit": "GB/s",
        "cores": cores,
        "kind": "oracle",
        "sample": "the whole step (both directions, all 32 images), %d repetitions, %.2f s each" % (reps, dt),
    }
    if gpu_forward is not None:
        if not np.array_equal(y.reshape(-1), gpu_forward.reshape(-1)):
            raise SystemExit("the timed forward buffer differs from the oracle's result")
        out["gpu_matches_oracle"] = True
    return out


def run_reference(args):
    """The CPU oracle on the host cores, on the same workload, metric and unit (rank 0 only): every step is the
    whole round trip on all 32 images."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle

    fwd_c, inv_c = W.c2_nchw_to_nhwc(), W.c2_nhwc_to_nchw()
    (x,) = W.make_inputs(fwd_c)
    cores = os.cpu_count() or 1
    bytes_per_step = 4 * x.nbytes

    def step():
        return oracle.run_chain(inv_c, [oracle.run_chain(fwd_c, [x], nt=cores)], nt=cores)

    t0 = time.perf_counter()
    step()
    first = time.perf_counter() - t0
    # the steps and warm-up asked for, unless they would not end within about two minutes
    steps = max(1, min(args.steps, int(100.0 / first)))
    warmup = max(0, min(args.warmup, int(20.0 / first)) - 1)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        z = step()
    dt = time.perf_counter() - t0
    assert np.array_equal(z, x)
    value = bytes_per_step * steps / dt / 1e9
    sample = "each step = the whole round trip on all 32 images (%d bytes moved), %d steps" % (bytes_per_step, steps)
    print(
        json.dumps(
            {
                "impl": "reference",
                "metric": METRIC,
                "value": round(value, 3),
                "unit": "GB/s",
                "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
                "steps": steps,
                "warmup": warmup + 1,
                "ms_per_step": dt / steps * 1e3,
                "higher_is_better": True,
                "scaling": "weak",
                "vs_baseline": None,
                "dtype": "u16",
                "data": "synthetic",
                "config": {
                    "workload": "configs[1]: bf16 [32,256,56,56] NCHW->NHWC then NHWC->NCHW, one composed copy each",
                    "bytes_per_step": bytes_per_step,
                    "how": "CPU oracle, operator by operator, OpenMP over the outermost loop",
                },
                "cpu_baseline": {"value": round(value, 3), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": round(value, 3), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            }
        )
    )


def run_one_config(args):
    """Runs ONE configuration's launches and nothing else (for profiler captures): W warm-up launches, then K."""
    import torch

    from paper_2002_12798_b200 import binding as B

    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    stream = torch.cuda.current_stream(device)
    l2 = torch.cuda.get_device_properties(device).L2_cache_size
    if args.config == "c2_round_trip":
        # the headline loop itself: forward and inverse alternating over the rotating buffer sets, the inverse
        # reading what the forward pass wrote half a rotation earlier
        fwd_c, inv_c = W.c2_nchw_to_nhwc(), W.c2_nhwc_to_nchw()
        fwd_p = B.compose_chain(fwd_c).plan(0, flags=args.plan_flags)
        inv_p = B.compose_chain(inv_c).plan(0, flags=args.plan_flags)
        (x,) = W.make_inputs(fwd_c)
        n_sets = max(2, -(-4 * l2 // (3 * x.nbytes)))
        n_sets += n_sets % 2
        xs = [torch.from_numpy(x.view(np.int16)).to(device) for _ in range(n_sets)]
        ys = [torch.empty_like(xs[0]) for _ in range(n_sets)]
        zs = [torch.empty_like(xs[0]) for _ in range(n_sets)]
        for s_ in range(n_sets):
            fwd_p.execute([xs[s_]], ys[s_], stream)
        fc = [fwd_p.bind([xs[s_]], ys[s_], stream) for s_ in range(n_sets)]
        ic = [inv_p.bind([ys[s_]], zs[s_], stream) for s_ in range(n_sets)]
        calls = [lambda s_=s_: (fc[s_](), ic[(s_ + n_sets // 2) % n_sets]()) for s_ in range(n_sets)]
        st = fwd_p.stats()
        total = 2 * (st["bytes_read"] + st["bytes_written"])

        class _C:
            launches = 2

        case = _C()
    elif args.config in ("consumer_c5", "consumer_c3"):
        # the row-sum consumer reading through the map (nothing is copied)
        name = args.config.split("_")[1]
        case = Case(torch, B, bench_configs()[name], device, stream, l2, args.plan_flags)
        m, n_sets = case.maps[0], case.n_sets
        cols = {"c5": 9 * 128, "c3": 128}[name]
        rows = m.out_numel // cols
        sums = [torch.empty(rows, dtype=torch.int32, device=device) for _ in range(n_sets)]
        calls = [m.bind_consume_row_sums(case.ins[i], rows, cols, sums[i], stream) for i in range(n_sets)]
        total = case.stats[0]["bytes_read"] + 4 * rows
        case.launches = 1
    else:
        case = Case(torch, B, bench_configs()[args.config], device, stream, l2, args.plan_flags)
        calls, n_sets, total = case.calls, case.n_sets, case.total
    for i in range(args.warmup):
        calls[i % n_sets]()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream.synchronize()
    start.record(stream)
    for i in range(args.steps):
        calls[i % n_sets]()
    stop.record(stream)
    stream.synchronize()
    sec = start.elapsed_time(stop) * 1e-3 / args.steps
    print(json.dumps({args.config: {"us": round(sec * 1e6, 2), "gbs": round(total / sec / 1e9, 1), "bytes": total,
                                    "buffer_sets": n_sets, "launches": case.launches}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--reps", type=int, default=10, help="least number of repetitions of the K-step region (median reported)")
    ap.add_argument("--min-seconds", type=float, default=1.5, help="repeat the K-step region until the timed region lasts this long")
    ap.add_argument("--no-graph", action="store_true", help="time individual stream launches only")
    ap.add_argument("--no-table", action="store_true", help="leave the per-configuration table out")
    ap.add_argument("--all-configs", action="store_true",
                    help="more rows (upsampling, QKV split, 512 MB plain copy) and, per row, the unfused chain and the CPU oracle")
    ap.add_argument("--plan-flags", type=int, default=0, help="amap_plan_opts.flags for every plan (1: no programmatic dependent launch, 2: no L2 prefetch)")
    ap.add_argument("--config", default=None, help="run ONE configuration's launches only (for profiler captures) and print its figures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.reps = max(args.reps, 10)
    if args.config:
        run_one_config(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
