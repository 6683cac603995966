#!/usr/bin/env python
"""Benchmark of the NOVAK per-parameter optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

One "step" = one novak_step (one fused kernel launch) over a whole synthetic
parameter set.  Prints ONE JSON line (rank 0).  Default workload: the
ResNet-50-shaped set (161 tensors, 25,557,032 fp32 parameters), the
configuration the headline metric is quoted on.

  value     parameter updates/s with everything resident in HBM (CUDA events
            around exactly K steps, max over ranks).
  roofline  algorithmic bytes per launch / average launch duration against the
            measured HBM copy rate of this machine (MEASURED_PEAKS.json).
  e2e       the same metric through novak_step_host: gradients start in pinned
            host memory, updated parameters are copied back, inside the timed
            region.
  cpu_baseline  the CPU oracle, as it stands, on the host cores (reported
            baseline, not a target).

With N > 1 (torchrun) every rank steps its own replica of the workload on its
own GPU: the step has no cross-element term, hence no collective on the data
path; only the barrier and the MAX of the timings use the process group.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "parameter updates/sec per novak_step"
UNIT = "param-updates/s"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the step kernel, by the
# lookahead action of the launch, from the ncu captures summarised under profiles/
# (novak_step_kernel_traffic.md): LAST: a step without / with a synchronisation;
# TRAJ_MEAN: first step of a window, a middle step, the synchronisation step.  A capture
# stops counting (traffic = null) as soon as the kernel sources differ from what was
# profiled (hashes below).
NCU_SOURCES = {"novak_step_kernel.cuh": "49bfe18d1bf9b988", "novak_step_types.h": "42992d0d45a7d8b6",
               "novak_launch.cu": "944348f3a890e975"}
NCU_TRAFFIC = {
    ("resnet50", "last"): {"plain": 657.53e6, "sync": 861.93e6},
    ("resnet50", "traj_mean"): {"first": 759.31e6, "middle": 860.55e6, "sync": 965.08e6},
    ("vgg16", "last"): {"plain": 3815.81e6, "sync": 4921.99e6},
    ("vgg16", "traj_mean"): {"first": 4372.67e6, "middle": 4921.70e6, "sync": 5480.16e6},
    ("vit-b16", "last"): {"plain": 2190.63e6, "sync": 2882.72e6},
    ("vit-b16", "traj_mean"): {"first": 2537.26e6, "middle": 2884.15e6, "sync": 3233.24e6},
}


def ncu_traffic(workload: str, mode: str, k: int, t_first: int, n_steps: int):
    """Per-launch DRAM traffic from the committed ncu captures, averaged over the lookahead
    schedule of the timed steps [t_first, t_first + n_steps), or None when no capture
    matches the workload or the built kernel."""
    import hashlib
    rec = NCU_TRAFFIC.get((workload, mode))
    if rec is None or k <= 1 or t_first <= 1:
        return None
    for name, want in NCU_SOURCES.items():
        path = os.path.join(ROOT, "paper_2601_07876_b200", "csrc", name)
        try:
            with open(path, "rb") as f:
                if hashlib.sha256(f.read()).hexdigest()[:16] != want:
                    return None
        except OSError:
            return None
    total = 0.0
    for t in range(t_first, t_first + n_steps):
        if t % k == 0:
            total += rec["sync"]
        elif mode == "last":
            total += rec["plain"]
        else:
            total += rec["first"] if (t - 1) % k == 0 else rec["middle"]
    return total / n_steps


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="workload index 0..4")
    ap.add_argument("--lookahead-mode", default="last", choices=["last", "traj_mean"])
    ap.add_argument("--clip", type=float, default=0.0,
                    help="c_clip of the global-norm clipping (0: off, the headline path)")
    ap.add_argument("--centralize", action="store_true",
                    help="gradient centralization on tensors with more than one dimension")
    ap.add_argument("--centralize-in-step", type=int, default=None, choices=[0, 1],
                    help="0: centralization always through the statistics pass (default 1: "
                         "inside the step kernel when nothing else needs the whole gradient)")
    ap.add_argument("--layer-adaptation", action="store_true",
                    help="layer-wise trust ratios (Eq. 19): theta, g, m, v are read once more")
    ap.add_argument("--layer-adaptation-in-step", type=int, default=None, choices=[0, 1],
                    help="0: two statistics kernels, then the step (default 1: layer adaptation and "
                         "update as one kernel whose updates find theta and the direction in L2)")
    ap.add_argument("--layer-adaptation-lead", type=int, default=None,
                    help="elements by which that kernel's updates trail its statistics beyond what "
                         "the longest tensor needs")
    ap.add_argument("--layer-adaptation-group", type=int, default=None,
                    help="chunk-table entries per CTA of that kernel (1..8)")
    ap.add_argument("--adaptive-beta", action="store_true", help="Eq. 3-4 (host scalars only)")
    ap.add_argument("--zero1", action="store_true",
                    help="one group sharded over the ranks (reduce-scatter, step on the owned "
                         "range, all-gather) instead of one replica per rank: strong scaling")
    ap.add_argument("--auto-lr", action="store_true",
                    help="Eq. 20-22: statistics pass plus one more read of the parameters")
    ap.add_argument("--bf16-copy", action="store_true",
                    help="the step also writes a bf16 copy of the parameters (+2 B per element)")
    ap.add_argument("--true-nesterov", action="store_true",
                    help="every step is a true-Nesterov step (Eq. 10-12): look-ahead kernel, then "
                         "the step, which reads theta_{t-1} from the save buffer; the closure "
                         "between the two is the caller's and not part of the step (+16 B per "
                         "element)")
    ap.add_argument("--restore-pass", action="store_true",
                    help="with --true-nesterov: a separate restore kernel between look-ahead "
                         "and step (+8 B per element more)")
    ap.add_argument("--moment-dtype", default="f32", choices=["f32", "bf16"],
                    help="storage type of m and v (bf16: 20 B per element instead of 28)")
    ap.add_argument("--graph", type=int, default=0, metavar="G",
                    help="graph-capturable step: G consecutive steps are captured into one CUDA "
                         "graph (stream capture) and the timed region replays it; steps is "
                         "rounded down to a multiple of G")
    ap.add_argument("--pool", type=int, default=4, help="gradient sets rotated through")
    ap.add_argument("--grad-offset", type=int, default=0, metavar="E",
                    help="start every gradient buffer E elements off the parameters' 16-byte "
                         "phase (E = 1..3: the gradient alone is then fetched element by element)")
    ap.add_argument("--chunk-elems", type=int, default=None)
    ap.add_argument("--ctas-per-sm", type=int, default=None)
    ap.add_argument("--serpentine", type=int, default=None)
    ap.add_argument("--dependent-launch", type=int, default=None)
    ap.add_argument("--lib", default=None, help="alternative libnovak.so (tuning builds)")
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--host-segment-elems", type=int, default=None,
                    help="run length of novak_step_host's pipeline (0: no pipelining)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--min-timed-seconds", type=float, default=0.5,
                    help="the K-step timed region is repeated until the repeats total at least "
                         "this long; ms_per_step is the median over the repeats")
    ap.add_argument("--max-repeats", type=int, default=2000)
    ap.add_argument("--per-step-steps", type=int, default=300,
                    help="steps of the separate pass that times every step on its own (0: skip)")
    ap.add_argument("--no-per-feature", action="store_true",
                    help="skip the paths around the plain step on the headline workload (key per_feature)")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the other workloads / lookahead modes (key per_workload)")
    return ap.parse_args()


def algorithmic_bytes_per_elem(grad_bytes: int, k: int, mode: str, t: int,
                               phase2: bool = False, trust: float = 0.0,
                               copy16: bool = False, auto: bool = False,
                               true_nesterov: bool = False, moment_bytes: int = 4) -> int:
    """Bytes the method itself has to move for one element on step t: theta, g, m, v
    read, theta, m, v written (Section 5.5: 4 reads + 3 writes), plus the lookahead
    arrays on the steps that touch them, plus one more read of g (`phase2`) when the
    global norm is needed before the first update (clipping, automatic learning-rate
    scaling).  Centralization alone adds nothing: a row mean is a statistic of one row,
    which fits on chip, so every byte still has to move only once."""
    mb = moment_bytes
    b = 4 + 2 * mb + grad_bytes + 4 + 2 * mb + (grad_bytes if phase2 else 0)
    if trust:
        # theta, g, m, v are needed twice (the norms of Eq. 19, then the update).  A tensor
        # that fits in L2 has to come from DRAM only once; `trust` is the share of the
        # group's elements in tensors too large for that (1.0: every tensor read twice).
        b += float(trust) * (4 + 2 * mb + grad_bytes)
    if copy16:
        b += 2
    if auto:
        b += 4                           # ||theta_t|| of Eq. 21
    if true_nesterov:
        b += 12 + mb                     # Eq. 10: theta, m read, save, theta written
    if true_nesterov == "restore":
        b += 8                           # the separate restore pass: save read, theta written
    if k <= 0:
        return b
    sync = t % k == 0
    if mode == "last" or k == 1:
        if t == 1:
            b += 4                       # slow <- theta_0
        if sync:
            b += 4 if t == 1 else 8      # slow read (not at t=1) + written
        return b
    first = (t - 1) % k == 0
    if t == 1:
        b += 4
    if not first:
        b += 4                           # running sum read
    if sync:
        b += 8                           # slow read + written
    else:
        b += 4                           # running sum written
    return b


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception as exc:  # pragma: no cover
            self.error = str(exc)

    _NAMES = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
        0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
        0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self._NAMES.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [],
                    "note": "no NVML samples"}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def run_reference(args, rank):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    import torch
    from oracle import novak_oracle as O
    from paper_2601_07876_b200 import workloads as W

    wl = W.get_workload(args.config)
    hyper = dict(wl.hyper, lookahead_mode=args.lookahead_mode)
    cores = len(os.sched_getaffinity(0))
    rng = np.random.default_rng(W.MASTER_SEED)

    def make(n):
        o = O.Oracle(O.Config.from_hyper(hyper), [rng.normal(0, 0.05, n)])
        g = rng.normal(0, 1e-3, n).astype(np.float32).astype(np.float64)
        return o, g

    # size the per-step sample so that steps+warmup finish in about two minutes
    probe_n = min(wl.total, 1 << 21)
    o, g = make(probe_n)
    o.step([g], threads=cores)
    t0 = time.perf_counter()
    for _ in range(3):
        o.step([g], threads=cores)
    rate = 3 * probe_n / (time.perf_counter() - t0)
    n = int(min(wl.total, max(4096, rate * 120.0 / (args.steps + args.warmup))))
    o, g = make(n)
    for _ in range(args.warmup):
        o.step([g], threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.step([g], threads=cores)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = (f"first {n} of {wl.total} elements of {wl.name} as one tensor, "
              f"{args.steps} oracle steps, {cores} threads over disjoint ranges")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "params": wl.total, "tensors": len(wl.numel),
                   "lookahead_mode": args.lookahead_mode},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def cpu_baseline(wl, hyper, seconds):
    """Oracle on the host cores for about `seconds` of work on a bounded sample."""
    import numpy as np
    from oracle import novak_oracle as O
    cores = len(os.sched_getaffinity(0))
    n = min(wl.total, 1 << 24)
    rng = np.random.default_rng(1)
    o = O.Oracle(O.Config.from_hyper(hyper), [rng.normal(0, 0.05, n)])
    g = rng.normal(0, 1e-3, n).astype(np.float32).astype(np.float64)
    o.step([g], threads=cores)
    steps, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < seconds and steps < 5000:
        if o.wants_extrapolation():
            o.extrapolated()             # Eq. 10 (the oracle's restore is a no-op)
        o.step([g], threads=cores)
        steps += 1
    dt = time.perf_counter() - t0
    # the same on one thread, a quarter of the time
    steps1, t1 = 0, time.perf_counter()
    while time.perf_counter() - t1 < seconds / 4 and steps1 < 5000:
        if o.wants_extrapolation():
            o.extrapolated()
        o.step([g], threads=1)
        steps1 += 1
    dt1 = time.perf_counter() - t1
    return {"value": n * steps / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "single_thread_value": n * steps1 / dt1,
            "sample": f"{n} elements of {wl.name} as one tensor x {steps} steps "
                      f"({dt:.1f} s), threads over disjoint element ranges; one thread: "
                      f"{steps1} steps ({dt1:.1f} s)"}


def run_zero1(args, rank, world, local):
    """ZeRO-1: the group's optimizer state is split over the ranks; every step
    reduce-scatters the gradients, steps the owned range and all-gathers the
    parameters (NCCL).  Total work is fixed as N grows."""
    import torch
    import torch.distributed as dist
    from paper_2601_07876_b200 import workloads as W
    from paper_2601_07876_b200 import zero1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    wl = W.get_workload(args.config)
    if wl.grad_dtype != torch.float32:
        raise SystemExit("--zero1 reduces fp32 gradients: pick an fp32 workload")
    n = zero1.padded_numel(wl.total, world)
    gen = torch.Generator(device=dev).manual_seed(W.MASTER_SEED)      # same parameters everywhere
    flat_p = torch.zeros(n, device=dev)
    flat_p[:wl.total].normal_(0.0, 0.05, generator=gen)
    gen_g = torch.Generator(device=dev).manual_seed(W.MASTER_SEED + 1 + rank)
    pool = []
    for _ in range(max(1, min(args.pool, int(8e9 // (4 * n)) or 1))):
        g = torch.zeros(n, device=dev)
        g[:wl.total].normal_(0.0, 1e-2, generator=gen_g)
        pool.append(g)
    opt = zero1.ShardedNovak(flat_p, wl.numel, **wl.hyper)
    scratch = torch.empty_like(pool[0])

    def one(i):
        scratch.copy_(pool[i % len(pool)])        # the reduce-scatter may overwrite its input
        opt.step(scratch)

    for i in range(max(3, args.warmup)):
        one(i)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        ev0.record()
        for i in range(args.steps):
            one(i)
        ev1.record()
        dist.barrier()
        torch.cuda.synchronize()
    t = torch.tensor([ev0.elapsed_time(ev1)], device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    if rank == 0:
        info = opt.local.info() if opt.local is not None else {}
        print(json.dumps({
            "metric": METRIC, "value": wl.total * args.steps / (ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "params": wl.total, "tensors": len(wl.numel),
                       "parallelism": f"zero1 x{world}: reduce-scatter(grad, avg) -> novak_step on "
                                      f"the owned 1/{world} -> all-gather(params); the timed step "
                                      "includes one device copy of the gradient buffer",
                       "owned_elements_rank0": opt.hi - opt.lo},
            "gpu_launches": info.get("launches"), "clocks": clocks.summary(),
        }))
    dist.destroy_process_group()


def quantile(sorted_vals, f):
    return sorted_vals[min(len(sorted_vals) - 1, int(f * len(sorted_vals)))] if sorted_vals else None


def timed_repeats(torch, step_fn, steps, repeats, barrier):
    """`repeats` back-to-back regions of exactly `steps` steps, each between two CUDA events
    on the launching stream, a barrier + synchronize before the first and after the last.
    Returns the regions' durations in ms."""
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    barrier()
    evs[0].record()
    i = 0
    for r in range(repeats):
        for _ in range(steps):
            step_fn(i)
            i += 1
        evs[r + 1].record()
    barrier()
    return [evs[r].elapsed_time(evs[r + 1]) for r in range(repeats)]


def repeats_for(ms_per_step_estimate, steps, min_seconds, max_repeats):
    region = max(1e-6, ms_per_step_estimate * steps * 1e-3)
    return int(max(1, min(max_repeats, -(-min_seconds // region))))


def time_one_workload(torch, B, W, dev, index, mode, steps, warmup, min_seconds, max_repeats,
                      pool_want, lib, barrier):
    """One workload in one lookahead mode, everything resident: median ms per step over
    repeated `steps`-step regions, with the algorithmic bytes of exactly those steps."""
    wl = W.get_workload(index)
    hyper = dict(wl.hyper, lookahead_mode=mode)
    k = hyper["lookahead_k"]
    gbytes = 2 if wl.grad_dtype == torch.bfloat16 else 4
    flat_p = W.alloc_flat(wl, torch.float32, dev)
    W.init_params(wl, flat_p)
    params = W.views(flat_p, wl)
    pool_n = max(1, min(pool_want, int(8e9 // (wl.total * gbytes)) or 1))
    src = W.GradSource(wl, dev)
    scratch = W.alloc_flat(wl, torch.float32, dev) if gbytes == 2 else None
    pool_flat = [W.alloc_flat(wl, wl.grad_dtype, dev) for _ in range(pool_n)]
    for gf in pool_flat:
        src.fill(gf, scratch)
    del scratch
    opt = B.NovakOptimizer(params, **hyper, lib=lib)
    pool = [opt.prepare(W.views(gf, wl)) for gf in pool_flat]
    for i in range(max(3, warmup)):
        opt.step(pool[i % pool_n])
    # a short probe sizes the number of repeats
    probe = timed_repeats(torch, lambda i: opt.step(pool[i % pool_n]), steps, 1, barrier)[0] / steps
    repeats = repeats_for(probe, steps, min_seconds, max_repeats)
    t_first = opt.info()["t"] + 1
    times = timed_repeats(torch, lambda i: opt.step(pool[i % pool_n]), steps, repeats, barrier)
    per = sorted(x / steps for x in times)
    ms = quantile(per, 0.5)
    alg = sum(algorithmic_bytes_per_elem(gbytes, k, mode, t)
              for t in range(t_first, t_first + steps * repeats)) / (steps * repeats)
    gbs = alg * wl.total / (ms * 1e-3) / 1e9
    peak, _ = measured_peak()
    out = {"workload": wl.name, "params": wl.total, "tensors": len(wl.numel),
           "grad_dtype": "bf16" if gbytes == 2 else "f32", "lookahead_mode": mode,
           "lookahead_k": k, "steps": steps, "repeats": repeats, "ms_per_step": ms,
           "p10": quantile(per, 0.1), "p90": quantile(per, 0.9),
           "updates_per_s": wl.total / (ms * 1e-3), "algorithmic_bytes_per_elem": alg,
           "hbm_gbs": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0,
           "traffic": ncu_traffic(wl.name, mode, k, t_first, steps * repeats),
           "grad_pool": pool_n, "launches": opt.info()["launches"]}
    del opt, pool, pool_flat, params, flat_p
    torch.cuda.empty_cache()
    return out


# The paths around the plain step, each timed on the headline workload (key per_feature).
# (name, optimizer keywords, bf16 parameter copies, algorithmic-byte keywords)
FEATURES = (
    ("clip", dict(clip_threshold=1.0), False, dict(phase2=True)),
    ("centralize", dict(centralize=True), False, dict()),
    ("clip+centralize", dict(clip_threshold=1.0, centralize=True), False, dict(phase2=True)),
    ("layer_adaptation", dict(layer_adaptation=True), False, dict(trust="fits")),
    ("layer_adaptation, three launches", dict(layer_adaptation=True, layer_adaptation_in_step=0),
     False, dict(trust=1.0)),
    ("clip+centralize+layer_adaptation", dict(clip_threshold=1.0, centralize=True, layer_adaptation=True),
     False, dict(phase2=True, trust="fits")),
    ("bf16 moments", dict(moment_dtype="bf16"), False, dict(moment_bytes=2)),
    ("bf16 parameter copies", dict(), True, dict(copy16=True)),
)


def time_one_feature(torch, B, W, dev, index, mode, feature, steps, warmup, min_seconds,
                     max_repeats, pool_want, lib, barrier):
    """One of FEATURES on one workload, everything resident: median ms per step over
    repeated `steps`-step regions, against the bytes that path has to move."""
    name, kw, copies, alg_kw = feature
    wl = W.get_workload(index)
    hyper = dict(wl.hyper, lookahead_mode=mode)
    k = hyper["lookahead_k"]
    gbytes = 2 if wl.grad_dtype == torch.bfloat16 else 4
    flat_p = W.alloc_flat(wl, torch.float32, dev)
    W.init_params(wl, flat_p)
    params = [v.view(s) for v, s in zip(W.views(flat_p, wl), wl.shapes)]
    pool_n = max(1, min(pool_want, int(8e9 // (wl.total * gbytes)) or 1))
    src = W.GradSource(wl, dev)
    scratch = W.alloc_flat(wl, torch.float32, dev) if gbytes == 2 else None
    pool_flat = [W.alloc_flat(wl, wl.grad_dtype, dev) for _ in range(pool_n)]
    for gf in pool_flat:
        src.fill(gf, scratch)
    del scratch
    opt = B.NovakOptimizer(params, **hyper, **kw, lib=lib)
    pool = [opt.prepare(W.views(gf, wl)) for gf in pool_flat]
    copy_flat = None
    if copies:
        copy_flat = W.alloc_flat(wl, torch.bfloat16, dev)
        opt.set_param_copies(W.views(copy_flat, wl))
    for i in range(max(3, warmup)):
        opt.step(pool[i % pool_n])
    probe = timed_repeats(torch, lambda i: opt.step(pool[i % pool_n]), steps, 1, barrier)[0] / steps
    repeats = repeats_for(probe, steps, min_seconds, max_repeats)
    t_first = opt.info()["t"] + 1
    l0 = opt.info()["launches"]
    times = timed_repeats(torch, lambda i: opt.step(pool[i % pool_n]), steps, repeats, barrier)
    launches = (opt.info()["launches"] - l0) / (steps * repeats)
    per = sorted(x / steps for x in times)
    ms = quantile(per, 0.5)
    alg_kw = dict(alg_kw)
    mbytes = alg_kw.get("moment_bytes", 4)
    if alg_kw.get("trust") == "fits":
        # one launch: only tensors too large to wait in L2 (theta, g, m, v beyond 48 MB) count twice
        per_elem_twice = 4 + 2 * mbytes + gbytes
        alg_kw["trust"] = sum(n for n in wl.numel if n * per_elem_twice > 48e6) / wl.total
    alg = sum(algorithmic_bytes_per_elem(gbytes, k, mode, t, **alg_kw)
              for t in range(t_first, t_first + steps * repeats)) / (steps * repeats)
    gbs = alg * wl.total / (ms * 1e-3) / 1e9
    peak, _ = measured_peak()
    out = {"feature": name, "workload": wl.name, "lookahead_mode": mode, "steps": steps,
           "repeats": repeats, "ms_per_step": ms, "p10": quantile(per, 0.1), "p90": quantile(per, 0.9),
           "updates_per_s": wl.total / (ms * 1e-3), "algorithmic_bytes_per_elem": alg,
           "hbm_gbs": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0,
           "launches_per_step": launches, "warnings": opt.info()["warnings"]}
    del opt, pool, pool_flat, params, flat_p, copy_flat
    torch.cuda.empty_cache()
    return out


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.zero1:
        run_zero1(args, rank, world, local)
        return

    import torch
    import torch.distributed as dist
    from paper_2601_07876_b200 import binding as B
    from paper_2601_07876_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the NOVAK step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    lib = B.load_library(args.lib) if args.lib else None
    wl = W.get_workload(args.config)
    hyper = dict(wl.hyper, lookahead_mode=args.lookahead_mode)
    if args.true_nesterov:
        hyper.update(nesterov="true", true_nesterov_steps=2 ** 31 - 1)
    if args.moment_dtype == "bf16":
        hyper.update(moment_dtype="bf16")
    mbytes = 2 if args.moment_dtype == "bf16" else 4
    k = hyper["lookahead_k"]
    gbytes = 2 if wl.grad_dtype == torch.bfloat16 else 4

    flat_p = W.alloc_flat(wl, torch.float32, dev)
    W.init_params(wl, flat_p)
    params = [v.view(s) for v, s in zip(W.views(flat_p, wl), wl.shapes)]
    phase2 = args.clip > 0 or args.auto_lr        # the whole gradient is read twice
    prepass = phase2 or args.centralize
    pool_n = max(1, min(args.pool, int(8e9 // (wl.total * gbytes)) or 1))
    src = W.GradSource(wl, dev, seed_offset=rank)
    scratch = W.alloc_flat(wl, torch.float32, dev) if gbytes == 2 else None
    pool_base = [torch.zeros(W.element_offsets(wl)[1] + 64, dtype=wl.grad_dtype, device=dev)
                 for _ in range(pool_n)]
    pool_flat = [b[args.grad_offset:args.grad_offset + W.element_offsets(wl)[1]] for b in pool_base]
    for gf in pool_flat:
        src.fill(gf, scratch)
    del scratch
    opt = B.NovakOptimizer(params, **hyper, clip_threshold=args.clip, centralize=args.centralize,
                           layer_adaptation=args.layer_adaptation, adaptive_beta=args.adaptive_beta,
                           auto_lr=args.auto_lr, graph_capturable=args.graph > 0,
                           centralize_in_step=args.centralize_in_step,
                           layer_adaptation_in_step=args.layer_adaptation_in_step,
                           layer_adaptation_lead=args.layer_adaptation_lead,
                           layer_adaptation_group=args.layer_adaptation_group,
                           chunk_elems=args.chunk_elems,
                           ctas_per_sm=args.ctas_per_sm, serpentine=args.serpentine,
                           dependent_launch=args.dependent_launch, lib=lib)
    pool = [opt.prepare(W.views(gf, wl)) for gf in pool_flat]
    if args.bf16_copy:
        copy_flat = W.alloc_flat(wl, torch.bfloat16, dev)
        opt.set_param_copies(W.views(copy_flat, wl))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    plain_step = opt.step
    if args.true_nesterov:
        def true_step(grads):
            opt.extrapolate()            # the caller's closure would run behind this
            if args.restore_pass:
                opt.restore()
            plain_step(grads)
        opt.step = true_step

    # ---------------- resident timing: exactly K steps between two events
    for i in range(max(3, args.warmup)):
        opt.step(pool[i % pool_n])
    graph = None
    if args.graph > 0:
        args.no_e2e = True                 # novak_step_host has no graph-capturable form
        # every pointer list of the pool is resident after the warm-up; capture G steps
        for i in range(pool_n):
            opt.step(pool[i])
        args.steps = max(args.graph, args.steps // args.graph * args.graph)
        torch.cuda.synchronize()
        l0 = opt.info()["launches"]
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(args.graph):
                opt.step(pool[i % pool_n])
        launches_per_graph = opt.info()["launches"] - l0
        for _ in range(3):
            graph.replay()
    if graph is not None:
        step_units = args.steps // args.graph          # one unit = one replay of G steps
        step_fn = lambda i: graph.replay()
    else:
        step_units = args.steps
        step_fn = lambda i: opt.step(pool[i % pool_n])
    # a probe region sizes the number of repeats of the K-step region
    probe_ms = timed_repeats(torch, step_fn, step_units, 1, barrier)[0]
    repeats = repeats_for(probe_ms / args.steps, args.steps, args.min_timed_seconds, args.max_repeats)
    if world > 1:
        r = torch.tensor([repeats], device=dev)
        dist.all_reduce(r, op=dist.ReduceOp.MAX)
        repeats = int(r.item())
    t_first = opt.info()["t"] + 1
    launches0 = opt.info()["launches"]
    uploads0 = opt.info()["record_uploads"]
    with ClockSampler(local) as clocks:
        region_ms = timed_repeats(torch, step_fn, step_units, repeats, barrier)
    grid_timed = opt.info()["grid"]          # before the end-to-end leg launches its runs
    launches = (opt.info()["launches"] - launches0) // repeats
    if graph is not None:
        launches = launches_per_graph * (args.steps // args.graph)
        assert opt.info()["t"] == t_first - 1 + args.steps * repeats   # every replayed step counted
    uploads = opt.info()["record_uploads"] - uploads0
    if world > 1:
        t = torch.tensor(region_ms, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)         # per region, the slowest rank
        region_ms = [float(x) for x in t.tolist()]
    per_region = sorted(x / args.steps for x in region_ms)
    ms_per_step = quantile(per_region, 0.5)
    value = world * wl.total / (ms_per_step * 1e-3)
    n_timed = args.steps * repeats
    # layer adaptation: tensors whose theta, g, m, v exceed 48 MB cannot wait in the 126 MB L2
    # between their statistics and their update
    per_elem_twice = 4 + 2 * mbytes + gbytes
    big = sum(n for n in wl.numel if n * per_elem_twice > 48e6) / wl.total
    trust_share = 0.0 if not args.layer_adaptation else (
        big if args.layer_adaptation_in_step != 0 else 1.0)
    alg = sum(algorithmic_bytes_per_elem(gbytes, k, args.lookahead_mode, t, phase2,
                                         trust_share, args.bf16_copy, args.auto_lr,
                                         ("restore" if args.restore_pass else True) if args.true_nesterov else False,
                                         mbytes)
              for t in range(t_first, t_first + n_timed)) / n_timed
    bytes_per_launch = alg * wl.total
    achieved = bytes_per_launch / (ms_per_step * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    traffic = None if (prepass or args.layer_adaptation or args.bf16_copy or args.true_nesterov
                       or mbytes == 2 or args.grad_offset) else \
        ncu_traffic(wl.name, args.lookahead_mode, k, t_first, n_timed)

    # ---------------- per-step distribution (separate short pass, event per step)
    per = {}
    if rank == 0 and graph is None and args.per_step_steps > 0:
        n_ps = args.per_step_steps
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_ps + 1)]
        t_ps = opt.info()["t"] + 1
        evs[0].record()
        for i in range(n_ps):
            opt.step(pool[i % pool_n])
            evs[i + 1].record()
        torch.cuda.synchronize()
        times = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_ps)]
        sync = sorted(x for i, x in enumerate(times) if k > 0 and (t_ps + i) % k == 0)
        plain = sorted(x for i, x in enumerate(times) if not (k > 0 and (t_ps + i) % k == 0))
        q = quantile
        per = {"non_sync_ms": {"p10": q(plain, .1), "p50": q(plain, .5), "p90": q(plain, .9)},
               "sync_ms": {"p10": q(sync, .1), "p50": q(sync, .5), "p90": q(sync, .9)},
               "steps": n_ps}

    # ---------------- end to end through novak_step_host (pinned host buffers)
    e2e = None
    if not args.no_e2e:
        h_g = W.alloc_flat(wl, wl.grad_dtype, dev, pin=True)
        h_p = W.alloc_flat(wl, torch.float32, dev, pin=True)
        h_g.copy_(pool_flat[0])
        d_g = pool_flat[0]
        offs, _ = W.element_offsets(wl)
        hp = B.ptr_array([h_p.data_ptr() + 4 * o for o in offs])
        hg = B.ptr_array([h_g.data_ptr() + gbytes * o for o in offs])
        dg = B.ptr_array([d_g.data_ptr() + gbytes * o for o in offs])
        stream = torch.cuda.current_stream().cuda_stream
        gdt = B.NOVAK_GRAD_BF16 if gbytes == 2 else B.NOVAK_GRAD_F32

        if args.host_segment_elems is not None:
            opt.handle.set_option(B.NOVAK_OPT_HOST_SEGMENT_ELEMS, args.host_segment_elems)
        launches_e2e = opt.info()["launches"]

        def host_step():
            opt.handle.step_host(hp, hg, opt._params_arr, dg, opt._numel_arr, opt.n, gdt, stream)

        for _ in range(3):
            host_step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(args.e2e_steps):
            host_step()
        e1.record()
        barrier()
        ems = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ems], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ems = float(t.item())
        e2e = {"value": world * wl.total * args.e2e_steps / (ems * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": wl.total * gbytes, "d2h_bytes_per_step": wl.total * 4,
               "ms_per_step": ems / args.e2e_steps, "steps": args.e2e_steps,
               "launches_per_step": (opt.info()["launches"] - launches_e2e) // (args.e2e_steps + 3),
               "host_segment_elems": int(opt.handle.get_option(B.NOVAK_OPT_HOST_SEGMENT_ELEMS)),
               "api": "novak_step_host (pinned host gradients in, parameters out; upload, "
                      "kernel and download pipelined in runs of the chunk table)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wl, hyper, args.cpu_seconds)

    info = opt.info() if rank == 0 else None
    headline_key = (wl.index, args.lookahead_mode)
    plain_headline = not (prepass or args.layer_adaptation or args.bf16_copy or args.true_nesterov
                          or args.adaptive_beta or mbytes == 2 or graph is not None)
    per_workload = None
    if rank == 0 and world == 1 and plain_headline and not args.no_per_workload:
        # every other workload and lookahead mode, one after the other, each freed before the next
        opt_cfg = {"chunk_elems": int(opt.handle.get_option(B.NOVAK_OPT_CHUNK_ELEMS)),
                   "ctas_per_sm": int(opt.handle.get_option(B.NOVAK_OPT_CTAS_PER_SM)),
                   "serpentine": int(opt.handle.get_option(B.NOVAK_OPT_SERPENTINE)),
                   "dependent_launch": int(opt.handle.get_option(B.NOVAK_OPT_DEPENDENT_LAUNCH))}
        del opt, pool, pool_flat, pool_base, params, flat_p
        torch.cuda.empty_cache()
        per_workload = [{
            "workload": wl.name, "params": wl.total, "tensors": len(wl.numel),
            "grad_dtype": "bf16" if gbytes == 2 else "f32", "lookahead_mode": args.lookahead_mode,
            "lookahead_k": k, "steps": args.steps, "repeats": repeats, "ms_per_step": ms_per_step,
            "p10": quantile(per_region, 0.1), "p90": quantile(per_region, 0.9),
            "updates_per_s": value, "algorithmic_bytes_per_elem": alg, "hbm_gbs": achieved,
            "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / 8000.0,
            "traffic": traffic, "grad_pool": pool_n, "headline": True}]
        free_bytes, _ = torch.cuda.mem_get_info()
        for index in range(5):
            for mode in ("last", "traj_mean"):
                if (index, mode) == headline_key:
                    continue
                wl_i = W.get_workload(index)
                if wl_i.total * 4 * 8 > free_bytes:
                    per_workload.append({"workload": wl_i.name, "lookahead_mode": mode,
                                         "skipped": "not enough free device memory"})
                    continue
                # large sets take fewer steps per region: a region of the 1 B set is 0.1 s
                steps_i = args.steps if wl_i.total < 5e8 else min(args.steps, 20)
                per_workload.append(time_one_workload(
                    torch, B, W, dev, index, mode, steps_i, args.warmup, args.min_timed_seconds,
                    args.max_repeats, args.pool, lib, barrier))

    per_feature = None
    if per_workload is not None and not args.no_per_feature:
        per_feature = [time_one_feature(torch, B, W, dev, wl.index, args.lookahead_mode, feat,
                                        args.steps, args.warmup, args.min_timed_seconds / 2,
                                        args.max_repeats, args.pool, lib, barrier)
                       for feat in FEATURES]

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "repeats": repeats, "p10": quantile(per_region, 0.1), "p90": quantile(per_region, 0.9),
            "timed_seconds": sum(region_ms) * 1e-3,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": wl.name, "params": wl.total, "tensors": len(wl.numel),
                "grad_dtype": "bf16" if gbytes == 2 else "f32",
                "lookahead_k": k, "lookahead_mode": args.lookahead_mode,
                "clip_threshold": args.clip, "centralize": bool(args.centralize),
                "layer_adaptation": bool(args.layer_adaptation),
                "layer_adaptation_elements_read_twice": trust_share,
                "adaptive_beta": bool(args.adaptive_beta), "bf16_copy": bool(args.bf16_copy),
                "true_nesterov": bool(args.true_nesterov), "restore_pass": bool(args.restore_pass),
                "moment_dtype": args.moment_dtype,
                "cuda_graph_steps": args.graph,
                "auto_lr": bool(args.auto_lr),
                "grad_pool": pool_n, "grad_offset_elems": args.grad_offset,
                "warnings": info["warnings"],
                "l2": "no flush: working set %.2f GB per step rotates through %d gradient sets, "
                      "larger than the 126 MB L2" % (bytes_per_launch / 1e9, pool_n),
                **(opt_cfg if per_workload is not None else {
                    "chunk_elems": int(opt.handle.get_option(B.NOVAK_OPT_CHUNK_ELEMS)),
                    "ctas_per_sm": int(opt.handle.get_option(B.NOVAK_OPT_CTAS_PER_SM)),
                    "serpentine": int(opt.handle.get_option(B.NOVAK_OPT_SERPENTINE)),
                    "dependent_launch": int(opt.handle.get_option(B.NOVAK_OPT_DEPENDENT_LAUNCH))}),
                "record_uploads_in_timed_region": uploads,
                "grid": grid_timed, "block": info["block"], "n_chunks": info["n_chunks"],
                "replicas": "each rank steps its own replica; no data-path collective",
            },
            "hbm_gbs": achieved,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_source": peak_src,
                         "algorithmic_bytes_per_elem": alg,
                         "traffic": traffic,
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "per_step": per,
            "per_workload": per_workload,
            "per_feature": per_feature,
            "e2e": e2e,
            "cpu_baseline": cpu,
            "gpu_launches": launches,
            "clocks": clocks.summary(),
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
