#!/usr/bin/env python
"""Benchmark of the ApproxIFER encode / decode / locate library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-others] [--no-e2e]

One step = one pass of the hot path over one batch of the largest encode
workload (K=12 queries, W=20 workers, 4,096 groups of 3x224x224 fp32 queries,
1000-class predictions, Bernoulli(0.3) stragglers capped at 8): encode all
groups, then decode all groups.  After the timed steps the decoder is also
timed alone on the largest decode workload (K=16, W=24, 262,144 groups of
1000-class predictions, 16-24 workers present); `roofline.kernels` lists the
three HBM-bound kernels at their largest configurations.  Rank 0 prints ONE
JSON line.  For N > 1 (launched by torchrun) every rank runs the same per-GPU
workload on its own GPU (groups are independent; there is no exchange step)
and the aggregate is reported.

--impl reference times the fp64 CPU checker on a bounded sample of the same
workload on the host cores.

--case NAME times one kernel alone (tuning / profiling); --case grid prints the
decoder's throughput over a grid of payload lengths on 3 GB problems, --case
locategrid the locator over K in {8, 10, 12} x E in {1, 2, 3}.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2109_09868_b200 import workloads as wl  # noqa: E402

METRIC = "encode+decode algorithmic GB/s (fp32 payload bytes read+written / time)"
UNIT = "GB/s"
HEADLINE_CFG = 3
HEADLINE_NAME = "configs[2]: K=12 W=20 D=150528 (3x224x224) C=1000, Bernoulli(0.3) stragglers capped at 8"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# DRAM traffic (ncu dram__bytes_read.sum + dram__bytes_write.sum) of encode_kernel<12, PayloadF32x4, 768> per group of
# the headline workload, from a capture of a reduced launch (profiles/encode_kernel_K12_W20_D150528.md); traffic is
# proportional to the number of groups (every row is touched once).  Set to None when the kernel changes, until
# the counters have been taken again.
ENCODE_TRAFFIC_PER_GROUP = (1387421696 + 2254734336) / 192
ENCODE_TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of a 192-group launch (3.7 GB) of the unchanged kernel, "
                         "per group x groups; the written part misses the ~58 MB of dirty lines still in L2 at kernel end")
E2E_GROUPS = 256
CPU_SAMPLE_GROUPS = 64


# ----------------------------------------------------------------- byte counts

def encode_bytes(w: wl.Workload) -> int:
    return 4 * w.D * (w.K + w.W) * w.G


def present_workers(mask: np.ndarray) -> int:
    return int(np.unpackbits(np.ascontiguousarray(mask).view(np.uint8)).sum())


def decode_bytes(w: wl.Workload, mask: np.ndarray) -> int:
    """Rows of present workers read, K rows written, one mask word per group."""
    return 4 * w.C * (present_workers(mask) + w.K * w.G) + 4 * w.G


def locate_bytes(w: wl.Workload, mask: np.ndarray) -> int:
    return 4 * w.C * present_workers(mask) + 4 * w.G + (4 * w.E + 4) * w.G


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, device copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# --------------------------------------------------------------- clock sampling

class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while a region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.split(",") for r in open(self.path).read().strip().splitlines() if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
                for k, nm in enumerate(names):
                    if r[5 + k].strip().lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                continue
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------- CPU oracle

def oracle_sample(groups: int):
    """Host copies of the first `groups` groups' worth of the headline workload (same generators, same seeds)."""
    w = wl.workload(HEADLINE_CFG, G=groups)
    X = wl.queries(w, "cpu").numpy()
    Yt = wl.gaussian_predictions(w, "cpu").numpy()
    mask = wl.masks(w)
    return w, X, Yt, mask, encode_bytes(w) + decode_bytes(w, mask)


def time_oracle(sample_groups: int = CPU_SAMPLE_GROUPS, min_seconds: float = 12.0, one_core_seconds: float = 6.0):
    """Times the fp64 CPU checker, as it stands, on a bounded sample of the headline workload
    (encode + decode of `sample_groups` groups, repeated), on all host cores and then on one."""
    import oracle

    w, X, Yt, mask, nbytes = oracle_sample(sample_groups)
    oracle.encode(w.K, w.W, X[:1])  # load / first-touch

    def run(seconds):
        reps, t0 = 0, time.perf_counter()
        while True:
            oracle.encode(w.K, w.W, X)
            oracle.decode(w.K, w.W, Yt, mask)
            reps += 1
            dt = time.perf_counter() - t0
            if dt >= seconds or reps >= 2000:
                return reps, dt

    cores = oracle.get_threads()
    reps, dt = run(min_seconds)
    oracle.set_threads(1)
    try:
        reps1, dt1 = run(one_core_seconds)
    finally:
        oracle.set_threads(cores)
    return {
        "value": nbytes * reps / dt / 1e9,
        "unit": UNIT,
        "cores": cores,
        "kind": "oracle",
        "sample": "%d of %d groups of the headline workload, encode+decode, %d repetitions in %.1f s; fp64 C, OpenMP over groups"
                  % (sample_groups, wl.workload(HEADLINE_CFG).G, reps, dt),
        "groups_per_s": sample_groups * reps / dt,
        "seconds": dt,
        "one_core": {"value": nbytes * reps1 / dt1 / 1e9, "unit": UNIT, "cores": 1, "groups_per_s": sample_groups * reps1 / dt1,
                     "seconds": dt1, "repetitions": reps1},
    }


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    sample = CPU_SAMPLE_GROUPS
    ws, X, Yt, mask, nbytes = oracle_sample(sample)

    def step():
        oracle.encode(ws.K, ws.W, X)
        oracle.decode(ws.K, ws.W, Yt, mask)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = nbytes * args.steps / dt / 1e9
    line = {
        "impl": "reference",
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": HEADLINE_NAME + "; each step a %d-group sample of the %d groups" % (sample, wl.workload(HEADLINE_CFG).G)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.get_threads(), "kind": "oracle",
                         "sample": "%d groups per step, encode+decode, fp64 C with OpenMP over groups" % sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "groups_per_s": sample * args.steps / dt,
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------- GPU measuring

def physical_gpu_index(local_rank: int) -> int:
    """nvidia-smi index of this rank's GPU (CUDA_VISIBLE_DEVICES may renumber the devices)."""
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    ids = [v.strip() for v in vis.split(",") if v.strip()]
    if local_rank < len(ids) and ids[local_rank].isdigit():
        return int(ids[local_rank])
    return local_rank


def time_launches(fn, warmup=3, iters=10, all_times=None):
    """Per-launch device time (ms) of fn() on the current stream: median and min."""
    for _ in range(warmup):
        fn()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    torch.cuda.synchronize()
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    if all_times is not None:
        all_times.extend(ms)
    return statistics.median(ms), min(ms)


def fit_groups(w: wl.Workload, bytes_per_group: int, budget: int) -> int:
    return int(max(1, min(w.G, budget // bytes_per_group)))


def kernel_entry(kernel, workload, nbytes, times_ms, peak, groups):
    mean = statistics.mean(times_ms)
    med = statistics.median(times_ms)
    return {"kernel": kernel, "workload": workload, "groups": groups, "launches": len(times_ms),
            "algorithmic_bytes_per_launch": nbytes, "mean_ms": mean, "median_ms": med, "min_ms": min(times_ms),
            "achieved": nbytes / mean / 1e6, "unit": "GB/s", "frac": nbytes / mean / 1e6 / peak,
            "frac_of_8TBps": nbytes / mean / 1e6 / NOMINAL_HBM_GBS, "groups_per_s": groups / mean * 1e3}


def workload4_predictions(ap, dev, w4g):
    """Coded predictions of the decode-heavy workload: a seeded smooth (linear) map of the coded hidden queries."""
    p4 = ap.make_params(w4g.K, w4g.W)
    Xc = ap.approxifer_encode(p4, wl.queries(w4g, dev))
    Yt = torch.empty((w4g.G, w4g.W, w4g.C), device=dev)
    chunk = 16384
    for s in range(0, w4g.G, chunk):
        Yt[s:s + chunk] = wl.apply_model(w4g, Xc[s:s + chunk])
    del Xc
    return Yt


def decode3_alone_entry(ap, dev, peak, seed_offset=0, launches=30):
    """The decoder alone on the headline workload's predictions (K=12, W=20, C=1000, 4,096 groups; 0.43 GB), launches
    back to back.  Taken before the timed steps: a second of encoder steps at the board's power cap lowers the SM
    clock, and a launch this short (its ramp-up and drain are a tenth of it) slows down with the clock."""
    w3 = wl.workload(3)
    p3 = ap.make_params(w3.K, w3.W)
    Yt = wl.gaussian_predictions(w3, dev)
    m3 = wl.masks(w3, seed_offset=seed_offset)
    mt = ap.mask_tensor(m3, dev)
    Yh = torch.empty((w3.G, w3.K, w3.C), device=dev)
    times = []
    time_launches(lambda: ap.approxifer_decode(p3, Yt, mt, Yh), 3, launches, times)
    e = kernel_entry("decode_staged_kernel", HEADLINE_NAME + " (decoder timed alone before the steps, launches back to back)",
                     decode_bytes(w3, m3), times, peak, w3.G)
    del Yt, Yh
    return e


def decode4_entry(ap, dev, peak, launches=40):
    """The decoder alone on the largest decode workload (K=16, W=24, C=1000, 262,144 groups, 16-24 present)."""
    free, _ = torch.cuda.mem_get_info()
    w4 = wl.workload(4)
    G4 = fit_groups(w4, 4 * w4.C * (w4.W + w4.K) * 5 // 4, int(free * 0.85))
    w4g = w4.with_groups(G4)
    p4 = ap.make_params(w4.K, w4.W)
    Yt = workload4_predictions(ap, dev, w4g)
    m4 = wl.masks(w4g)
    mt = ap.mask_tensor(m4, dev)
    Yh = torch.empty((G4, w4.K, w4.C), device=dev)
    times = []
    # back to back: the first launches run at boost clocks, then the board's power cap lowers the SM clock and the
    # launch time settles; the entry's figure is the mean of all of them, both regimes are given
    time_launches(lambda: ap.approxifer_decode(p4, Yt, mt, Yh), 3, launches, times)
    nb = decode_bytes(w4g, m4)
    e = kernel_entry("decode_staged_kernel", "configs[3]: K=16 W=24 C=1000, 16-24 workers present", nb, times, peak, G4)
    e["note"] = "all 262144 groups" if G4 == w4.G else "G reduced to %d to fit free device memory" % G4
    e["first5_GB_per_s"] = nb / statistics.median(times[:5]) / 1e6
    e["last20_GB_per_s"] = nb / statistics.median(times[-20:]) / 1e6
    del Yt, Yh
    torch.cuda.empty_cache()
    return e


def grid_masks(K, W, G, seed):
    """0 .. min(4, W-K) stragglers per group, uniform count, uniform subset (the recipe of workload 2)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n_s = rng.integers(0, min(4, W - K) + 1, size=G)
    rank = rng.random((G, W)).argsort(axis=1).argsort(axis=1)
    present = rank >= n_s[:, None]
    return (present.astype(np.uint64) << np.arange(W, dtype=np.uint64)).sum(axis=1).astype(np.uint32)


def synthetic_decode(ap, dev, K, W, C, G, worker_major=False, iters=10, tuning=None, seed=7):
    """The decoder alone on iid N(0,1) predictions [G][W][C] (or worker-major [W][G][C]) and grid_masks."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    if worker_major:
        Yt = torch.randn((W, G, C), generator=g, device=dev).permute(1, 0, 2)
    else:
        Yt = torch.randn((G, W, C), generator=g, device=dev)
    m = grid_masks(K, W, G, seed)
    mt = ap.mask_tensor(m, dev)
    Yh = torch.empty((G, K, C), device=dev)
    p = ap.make_params(K, W)
    med, mn = time_launches(lambda: ap.approxifer_decode(p, Yt, mt, Yh, tuning=tuning), 3, iters)
    nb = 4 * C * (present_workers(m) + K * G) + 4 * G
    del Yt, Yh
    return {"K": K, "W": W, "C": C, "groups": G, "layout": "[W][G][C]" if worker_major else "[G][W][C]",
            "algorithmic_GB": nb / 1e9, "ms": med, "ms_min": mn, "GB_per_s": nb / med / 1e6,
            "frac_of_8TBps": nb / med / 1e6 / NOMINAL_HBM_GBS, "groups_per_s": G / med * 1e3}


def decode_grid(ap, dev, gigabytes=3.0, worker_major=False):
    """Decoder throughput over payload lengths, on problems of about `gigabytes` GB (far beyond L2)."""
    out = []
    for (K, W) in ((8, 12), (16, 24)):
        for C in (10, 48, 64, 100, 128, 256):
            G = int(gigabytes * 1e9 / (4 * C * (W + K))) // 1024 * 1024
            out.append(synthetic_decode(ap, dev, K, W, C, G, worker_major))
            torch.cuda.empty_cache()
    return out


def fma_peak(ap, dev):
    """fp32 multiply-add issue rate from a register-only loop (the second roof of the weighted sums)."""
    sink = torch.zeros(1, device=dev)
    iters, blocks = 4096, 148 * 8
    med, mn = time_launches(lambda: ap.debug_fma_peak(iters, blocks, sink), 2, 5)
    flop = 2.0 * 64 * iters * 256 * blocks
    return {"fp32_fma_TFLOP_per_s": flop / mn / 1e9, "ms_min": mn, "ms_median": med,
            "nominal_TFLOP_per_s": 148 * 128 * 2 * 1.965e9 / 1e12,
            "note": "register-only loop, 16 independent chains per thread, 8 CTAs of 256 threads per SM; nominal = 148 SMs x 128 lanes x 2 x 1.965 GHz"}


def locate_grid(ap, dev, G=65536, C=10):
    """The locator over the paper's own grid (Section 4.2: K in {8, 10, 12}, E in {1, 2, 3}, no stragglers), linear
    stand-in model, N(0, 10^2) noise on the E adversaries: ms per launch and groups/s."""
    out = []
    for K in (8, 10, 12):
        for E in (1, 2, 3):
            W = 2 * (K + E)
            g = torch.Generator(device=dev)
            g.manual_seed(1000 * K + E)
            p = ap.make_params(K, W, E)
            X = torch.rand((G, K, 64), generator=g, device=dev)
            M = torch.randn((64, C), generator=g, device=dev) / 8.0
            Yt = (ap.approxifer_encode(p, X) @ M).contiguous()
            rng = np.random.Generator(np.random.PCG64(K * 10 + E))
            bad = np.sort(rng.random((G, W)).argsort(axis=1)[:, :E], axis=1)
            rows = torch.arange(G, device=dev)[:, None].expand(G, E)
            Yt[rows, torch.as_tensor(bad, device=dev)] += torch.randn((G, E, C), generator=g, device=dev) * 10.0
            mt = ap.mask_tensor(np.full(G, (1 << W) - 1, dtype=np.uint32), dev)
            adv = torch.empty((G, E), dtype=torch.int32, device=dev)
            trusted = torch.empty((G,), dtype=torch.int32, device=dev)
            med, mn = time_launches(lambda: ap.approxifer_locate(p, Yt, mt, adv, trusted), 3, 10)
            out.append({"K": K, "E": E, "W": W, "groups": G, "C": C, "ms": med, "ms_min": mn, "groups_per_s": G / med * 1e3,
                        "located_equals_injected": float((adv.cpu().numpy() == bad).all(axis=1).mean())})
    return out


def host_cost(ap, dev):
    """Host time of one call (argument checks, plan, launch), from 1000 back-to-back calls on small problems."""
    out = []
    w1 = wl.workload(1)
    p1 = ap.make_params(w1.K, w1.W)
    X1 = wl.queries(w1, dev)
    Xt1 = torch.empty((w1.G, w1.W, w1.D), device=dev)
    w2 = wl.workload(2, G=4096)
    p2 = ap.make_params(w2.K, w2.W)
    Yt2 = wl.gaussian_predictions(w2, dev)
    m2 = ap.mask_tensor(wl.masks(w2), dev)
    Yh2 = torch.empty((w2.G, w2.K, w2.C), device=dev)
    for name, fn in (("approxifer_encode, configs[0] shape", lambda: ap.approxifer_encode(p1, X1, Xt1)),
                     ("approxifer_decode, configs[1] shape, 4096 groups", lambda: ap.approxifer_decode(p2, Yt2, m2, Yh2))):
        for _ in range(20):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(1000):
            fn()
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        out.append({"call": name, "host_us_per_call": (t1 - t0) * 1e3, "note": "python binding + C entry point + launch, 1000 calls back to back"})
    return out


def other_workloads(ap, dev, peak):
    """Kernel-only figures for the other configurations (each timed alone,
    inputs far larger than L2 except where noted)."""
    out = []
    free, _ = torch.cuda.mem_get_info()
    budget = int(free * 0.85)

    def entry(name, nbytes, ms_med, ms_min, G, extra=None):
        e = {"workload": name, "groups": G, "algorithmic_GB": nbytes / 1e9, "ms": ms_med, "ms_min": ms_min,
             "GB_per_s": nbytes / ms_med / 1e6, "frac_of_measured_peak": nbytes / ms_med / 1e6 / peak,
             "frac_of_8TBps": nbytes / ms_med / 1e6 / NOMINAL_HBM_GBS, "groups_per_s": G / ms_med * 1e3}
        if extra:
            e.update(extra)
        out.append(e)

    # workload 2: 3x32x32 queries, 10-class predictions
    w2 = wl.workload(2)
    G2 = fit_groups(w2, 4 * w2.D * (w2.K + w2.W), budget)
    w2g = w2.with_groups(G2)
    p2 = ap.make_params(w2.K, w2.W)
    X = wl.queries(w2g, dev)
    Xt = torch.empty((G2, w2.W, w2.D), device=dev)
    med, mn = time_launches(lambda: ap.approxifer_encode(p2, X, Xt), 3, 20)
    entry("configs[1] encode K=8 W=12 D=3072", encode_bytes(w2g), med, mn, G2)
    # the same encode writing the coded queries worker-major ([W][G][D]: one contiguous batch per worker)
    Xt_wm = Xt.view(w2.W, G2, w2.D).permute(1, 0, 2)
    med, mn = time_launches(lambda: ap.approxifer_encode(p2, X, Xt_wm), 3, 20)
    entry("configs[1] encode, coded queries written worker-major [W][G][D]", encode_bytes(w2g), med, mn, G2)
    del Xt, Xt_wm
    # ... and scattered: every worker's batch a buffer of its own (the layout of peer-resident batches)
    rows = [torch.empty((G2, w2.D), device=dev) for _ in range(w2.W)]
    med, mn = time_launches(lambda: ap.approxifer_encode_scatter(p2, X, rows), 3, 20)
    entry("configs[1] encode, coded queries scattered to one buffer per worker (approxifer_encode_scatter)", encode_bytes(w2g), med, mn, G2)
    del X, rows
    Yt = wl.gaussian_predictions(w2, dev)
    m2 = wl.masks(w2)
    mt = ap.mask_tensor(m2, dev)
    Yh = torch.empty((w2.G, w2.K, w2.C), device=dev)
    med, mn = time_launches(lambda: ap.approxifer_decode(p2, Yt, mt, Yh), 3, 20)
    entry("configs[1] decode K=8 W=12 C=10 (47 MB: L2-resident, launch-bound)", decode_bytes(w2, m2), med, mn, w2.G)
    del Yt, Yh
    torch.cuda.empty_cache()

    # workload 5: Byzantine -- locate, then decode from the trusted workers
    w5 = wl.workload(5)
    p5 = ap.make_params(w5.K, w5.W, w5.E)
    Xh = wl.queries(w5, dev)
    Xc = ap.approxifer_encode(p5, Xh)
    Yt = wl.apply_model(w5, Xc)
    m5 = wl.masks(w5)
    adv_true = wl.adversaries(w5, m5)
    wl.corrupt(w5, Yt, adv_true)
    mt = ap.mask_tensor(m5, dev)
    adv = torch.empty((w5.G, w5.E), dtype=torch.int32, device=dev)
    trusted = torch.empty((w5.G,), dtype=torch.int32, device=dev)
    Yh = torch.empty((w5.G, w5.K, w5.C), device=dev)
    med, mn = time_launches(lambda: ap.approxifer_locate(p5, Yt, mt, adv, trusted), 3, 10)
    recall = float((adv.cpu().numpy() == adv_true).all(axis=1).mean())
    # Algorithm 2 as printed: per class a least-squares problem with n rows and m' = 2(K+E)-1 unknowns,
    # 2 n m'^2 - (2/3) m'^3 flop by Householder QR; fp64 peak = 64 FMA lanes/SM/clock.
    n5, mp5 = w5.W - w5.S, 2 * (w5.K + w5.E) - 1
    flops = w5.G * w5.C * (2.0 * n5 * mp5 * mp5 - (2.0 / 3.0) * mp5 ** 3)
    fp64_peak = 148 * 64 * 2 * 1.965e9 / 1e12
    entry("configs[4] locate K=8 W=24 E=2 C=10 (fp64 solve, ALU-bound; L2-resident input)", locate_bytes(w5, m5), med, mn, w5.G,
          {"located_equals_injected": recall,
           "roofline": {"bound": "alu", "achieved": flops / med / 1e9, "peak": fp64_peak, "unit": "TFLOP/s",
                        "frac": flops / med / 1e9 / fp64_peak,
                        "note": "algorithmic fp64 flop of Algorithm 2's per-class least squares / time; peak = 148 SMs x 64 DFMA/clk x 2 x 1.965 GHz"}})
    Yt_wm = Yt.permute(1, 0, 2).contiguous().permute(1, 0, 2)  # worker-major storage, [G][W][C] view
    med, mn = time_launches(lambda: ap.approxifer_locate(p5, Yt_wm, mt, adv, trusted), 3, 10)
    entry("configs[4] locate, predictions stored worker-major [W][G][C]", locate_bytes(w5, m5), med, mn, w5.G,
          {"located_equals_injected": float((adv.cpu().numpy() == adv_true).all(axis=1).mean())})
    p5h = ap.make_params(w5.K, w5.W, w5.E, 2)
    med, mn = time_launches(lambda: ap.approxifer_locate(p5h, Yt, mt, adv, trusted), 3, 10)
    recall_h = float((adv.cpu().numpy() == adv_true).all(axis=1).mean())
    entry("configs[4] locate, Algorithm 1's homogeneous system (|Q| = 1) per class", locate_bytes(w5, m5), med, mn, w5.G,
          {"located_equals_injected": recall_h})
    med, mn = time_launches(lambda: ap.approxifer_decode_rational(p5, Yt, mt, Yh), 3, 10)
    entry("configs[4] rational decoding (Algorithm 3: P/Q at the alpha nodes, nothing located)",
          locate_bytes(w5, m5) + 4 * w5.G * w5.K * w5.C, med, mn, w5.G)
    ap.approxifer_locate(p5, Yt, mt, adv, trusted)
    t5 = trusted.cpu().numpy().view(np.uint32)
    med, mn = time_launches(lambda: ap.approxifer_decode(p5, Yt, trusted, Yh), 3, 10)
    entry("configs[4] decode from trusted K=8 W=24 C=10 (L2-resident)", decode_bytes(w5, t5), med, mn, w5.G)
    med, mn = time_launches(lambda: ap.approxifer_decode(p5, Yt_wm, trusted, Yh), 3, 10)
    entry("configs[4] decode from trusted, predictions stored worker-major [W][G][C]", decode_bytes(w5, t5), med, mn, w5.G)
    rows5 = [Yt[:, i].contiguous() for i in range(w5.W)]
    med, mn = time_launches(lambda: ap.approxifer_locate_gather(p5, rows5, mt), 3, 10)
    entry("configs[4] locate, predictions gathered from one buffer per worker (approxifer_locate_gather)", locate_bytes(w5, m5), med, mn, w5.G)
    med, mn = time_launches(lambda: ap.approxifer_decode_gather(p5, rows5, trusted, Yh), 3, 10)
    entry("configs[4] decode from trusted, gathered from one buffer per worker (approxifer_decode_gather; host-bound at this size: the binding checks W tensors per call, the kernel is the worker-major one above)", decode_bytes(w5, t5), med, mn, w5.G)
    del rows5
    med, mn = time_launches(lambda: ap.approxifer_locate_decode(p5, Yt, mt, Yh), 3, 10)
    entry("configs[4] locate + decode from trusted through approxifer_locate_decode (two launches at this size)",
          locate_bytes(w5, m5) + 4 * w5.G * w5.K * w5.C, med, mn, w5.G)
    del Yt, Yt_wm, Yh
    # workload 1: tiny, launch-latency bound
    w1 = wl.workload(1)
    p1 = ap.make_params(w1.K, w1.W)
    X1 = wl.queries(w1, dev)
    Xt1 = torch.empty((w1.G, w1.W, w1.D), device=dev)
    med, mn = time_launches(lambda: ap.approxifer_encode(p1, X1, Xt1), 3, 20)
    entry("configs[0] encode K=4 W=5 D=784 (launch-latency bound, L2-resident)", encode_bytes(w1), med, mn, w1.G)
    # bfloat16 payloads (fp32 weights and sums): bytes counted at 2 per element
    w2b = wl.workload(2)
    Xb = wl.queries(w2b, dev).to(torch.bfloat16)
    Xtb = torch.empty((w2b.G, w2b.W, w2b.D), device=dev, dtype=torch.bfloat16)
    p2b = ap.make_params(w2b.K, w2b.W)
    med, mn = time_launches(lambda: ap.approxifer_encode_bf16(p2b, Xb, Xtb), 3, 20)
    entry("configs[1] encode with bfloat16 payloads K=8 W=12 D=3072", encode_bytes(w2b) // 2, med, mn, w2b.G)
    del Xb, Xtb
    torch.cuda.empty_cache()
    w4b = wl.workload(4, G=65536)
    Ytb = workload4_predictions(ap, dev, w4b).to(torch.bfloat16)
    m4b = wl.masks(w4b)
    mtb = ap.mask_tensor(m4b, dev)
    Yhb = torch.empty((w4b.G, w4b.K, w4b.C), device=dev, dtype=torch.bfloat16)
    p4b = ap.make_params(w4b.K, w4b.W)
    med, mn = time_launches(lambda: ap.approxifer_decode_bf16(p4b, Ytb, mtb, Yhb), 3, 10)
    entry("configs[3] decode with bfloat16 payloads K=16 W=24 C=1000, 65536 groups",
          2 * w4b.C * (present_workers(m4b) + w4b.K * w4b.G) + 4 * w4b.G, med, mn, w4b.G)
    del Ytb, Yhb
    torch.cuda.empty_cache()
    # the largest K and W the library takes
    G32 = 8192
    g = torch.Generator(device=dev)
    g.manual_seed(32)
    X32 = torch.rand((G32, 32, 3072), generator=g, device=dev)
    Xt32 = torch.empty((G32, 32, 3072), device=dev)
    p32 = ap.make_params(32, 32)
    med, mn = time_launches(lambda: ap.approxifer_encode(p32, X32, Xt32), 3, 10)
    entry("encode K=32 W=32 D=3072 (64 flop per 8 payload bytes: fp32 issue and HBM both loaded)", 4 * 3072 * 64 * G32, med, mn, G32)
    del X32, Xt32
    torch.cuda.empty_cache()
    e = synthetic_decode(ap, dev, 32, 32, 1000, 16384)
    e["workload"] = "decode K=32 W=32 C=1000, all workers present"
    out.append(e)
    torch.cuda.empty_cache()
    # the paper's own decode shape beyond the cache, predictions stored one batch per worker
    e = synthetic_decode(ap, dev, 8, 12, 10, 3749888, worker_major=True)
    e["workload"] = "decode K=8 W=12 C=10 on a 3 GB problem, predictions stored worker-major [W][G][C], 0-4 stragglers"
    out.append(e)
    torch.cuda.empty_cache()
    return out


def run_case(ap, dev, args):
    """One kernel of one configuration, timed alone (CUDA events per launch)."""
    tuning = ap.decode_tuning(*[int(v) for v in args.dec_config.split(",")]) if args.dec_config else None
    iters = max(args.steps, 1)
    warm = max(args.warmup, 1)
    if args.case == "grid":
        return {"case": "grid", "decode": decode_grid(ap, dev, worker_major=args.worker_major)}
    if args.case == "decode":  # --shape K,W,C,G: iid predictions, 0-4 stragglers
        K, W, C, G = [int(v) for v in args.shape.split(",")]
        e = synthetic_decode(ap, dev, K, W, C, G, args.worker_major, iters, tuning)
        e.update(case="decode", dec_config=args.dec_config, wait_timeouts=ap.device_wait_timeouts())
        return e
    if args.case == "locategrid":
        return {"case": "locategrid", "locate": locate_grid(ap, dev)}
    if args.case == "fmapeak":
        return {"case": "fmapeak", **fma_peak(ap, dev)}
    if args.case == "hostcost":
        return {"case": "hostcost", "calls": host_cost(ap, dev)}
    cfg = int(args.case[-1])
    op = args.case[:-1]
    w = wl.workload(cfg, args.groups)
    p = ap.make_params(w.K, w.W, w.E)
    if op == "locateh":  # the locator with Algorithm 1's homogeneous system
        op, p = "locate", ap.make_params(w.K, w.W, w.E, 2)
    if op == "encode":
        dt = torch.bfloat16 if args.bf16 else torch.float32
        X = wl.queries(w, dev).to(dt)
        Xt = torch.empty((w.G, w.W, w.D), device=dev, dtype=dt)
        if args.worker_major:
            Xt = Xt.view(w.W, w.G, w.D).permute(1, 0, 2)
        enc = ap.approxifer_encode_bf16 if args.bf16 else ap.approxifer_encode
        med, mn = time_launches(lambda: enc(p, X, Xt), warm, iters)
        nbytes = encode_bytes(w) // (2 if args.bf16 else 1)
    else:
        if cfg in (2, 3):
            Yt = wl.gaussian_predictions(w, dev)
        elif cfg == 4:
            Yt = workload4_predictions(ap, dev, w)
        else:
            Yt = wl.apply_model(w, ap.approxifer_encode(p, wl.queries(w, dev)))
        m = wl.masks(w)
        if cfg == 5:
            wl.corrupt(w, Yt, wl.adversaries(w, m))
        if args.worker_major:
            Yt = Yt.permute(1, 0, 2).contiguous().permute(1, 0, 2)
        mt = ap.mask_tensor(m, dev)
        if op == "locate":
            adv = torch.empty((w.G, w.E), dtype=torch.int32, device=dev)
            trusted = torch.empty((w.G,), dtype=torch.int32, device=dev)
            med, mn = time_launches(lambda: ap.approxifer_locate(p, Yt, mt, adv, trusted), warm, iters)
            nbytes = locate_bytes(w, m)
        elif op == "rational":  # Algorithm 3: P/Q at the alpha nodes
            Yh = torch.empty((w.G, w.K, w.C), device=dev)
            med, mn = time_launches(lambda: ap.approxifer_decode_rational(p, Yt, mt, Yh), warm, iters)
            nbytes = locate_bytes(w, m) + 4 * w.G * w.K * w.C
        elif op == "pair":
            Yh = torch.empty((w.G, w.K, w.C), device=dev)
            if args.one_pass is not None:  # 1: the one-pass kernel, 0: the two launches; default: the library's choice
                p = ap.make_params(w.K, w.W, w.E, 4 if args.one_pass else 8)
            med, mn = time_launches(lambda: ap.approxifer_locate_decode(p, Yt, mt, Yh), warm, iters)
            nbytes = locate_bytes(w, m) + 4 * w.G * w.K * w.C
        else:
            Yh = torch.empty((w.G, w.K, w.C), device=dev)
            med, mn = time_launches(lambda: ap.approxifer_decode(p, Yt, mt, Yh, tuning=tuning), warm, iters)
            nbytes = decode_bytes(w, m)
    return {"case": args.case, "groups": w.G, "dec_config": args.dec_config, "worker_major": args.worker_major, "ms": med,
            "ms_min": mn, "GB_per_s": nbytes / med / 1e6, "groups_per_s": w.G / med * 1e3, "algorithmic_GB": nbytes / 1e9,
            "wait_timeouts": ap.device_wait_timeouts()}


def run_e2e(ap, dev, w, steps, warmup):
    """Same metric through the library's host-buffer entry points: every step takes the queries and the
    coded predictions from pinned HOST memory and leaves the coded queries and the decoded predictions
    in pinned host memory (approxifer_encode_host / approxifer_decode_host: chunks of groups staged
    through a device workspace on four streams, so both copy directions and the kernels overlap)."""
    p = ap.make_params(w.K, w.W)
    hX = torch.empty((w.G, w.K, w.D), dtype=torch.float32, pin_memory=True)
    hXt = torch.empty((w.G, w.W, w.D), dtype=torch.float32, pin_memory=True)
    hYt = torch.empty((w.G, w.W, w.C), dtype=torch.float32, pin_memory=True)
    hYh = torch.empty((w.G, w.K, w.C), dtype=torch.float32, pin_memory=True)
    mask_np = wl.masks(w)
    hmask = torch.from_numpy(mask_np.view(np.int32).copy()).pin_memory()
    hX.uniform_(0, 1)
    hYt.normal_(0, 2.0 ** 0.5)
    streams = [torch.cuda.Stream(device=dev) for _ in range(4)]
    ws_enc = torch.empty(512 << 20, dtype=torch.uint8, device=dev)  # small chunks: short pipeline fill and drain
    ws_dec = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
    main = torch.cuda.current_stream()

    def step():
        for st in streams:
            st.wait_stream(main)
        ap.approxifer_encode_host(p, hX, hXt, ws_enc, streams)
        ap.approxifer_decode_host(p, hYt, hmask, hYh, ws_dec, streams[:1])
        for st in streams:
            main.wait_stream(st)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    launches0 = ap.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    h2d = hX.numel() * 4 + hYt.numel() * 4 + hmask.numel() * 4
    d2h = hXt.numel() * 4 + hYh.numel() * 4
    nbytes = encode_bytes(w) + decode_bytes(w, mask_np)
    return ms, h2d, d2h, (ap.launch_count() - launches0) // steps, nbytes


def main():
    ap_ = argparse.ArgumentParser()
    ap_.add_argument("--gpus", type=int, default=1)
    ap_.add_argument("--steps", type=int, default=100)
    ap_.add_argument("--warmup", type=int, default=3)
    ap_.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap_.add_argument("--no-others", action="store_true", help="skip the per-configuration kernel figures")
    ap_.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap_.add_argument("--no-cpu", action="store_true", help="skip timing the CPU checker")
    ap_.add_argument("--groups", type=int, default=None, help="override the number of groups (profiling only)")
    ap_.add_argument("--case", default=None,
                     choices=["decode2", "decode3", "decode4", "decode5", "locate5", "locateh5", "rational5", "pair5", "encode2", "encode3",
                              "decode", "grid", "hostcost", "fmapeak", "locategrid"],
                     help="time one kernel alone (tuning / profiling) and print a short JSON line; `decode` takes --shape, "
                          "`grid` runs the decoder over payload lengths 10..256 on 3 GB problems")
    ap_.add_argument("--shape", default="8,12,64,1048576", help="K,W,C,G for --case decode")
    ap_.add_argument("--one-pass", type=int, default=None, help="--case pair5: 1 forces the one-pass kernel, 0 the two launches")
    ap_.add_argument("--bf16", action="store_true", help="--case encodeN: bfloat16 payloads")
    ap_.add_argument("--worker-major", action="store_true", help="--case: coded rows stored [W][G][*] (one batch per worker)")
    ap_.add_argument("--dec-config", default=None, help="kernel,stages,ctas_per_sm,cols,split for the decoder (--case, tuning)")
    args = ap_.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.warmup < 3:
        args.warmup = max(args.warmup, 1) if (args.groups or args.case) else 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    import torch.distributed as dist

    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    import paper_2109_09868_b200 as ap

    if args.case:
        print(json.dumps(run_case(ap, dev, args)), flush=True)
        return

    # CPU baseline first (rank 0, N = 1 only), before the GPU gets busy
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = time_oracle()

    peak, peak_src = measured_peak()
    # the small decode of the headline workload alone, before the long run of steps pulls the SM clock down
    # (0.43 GB in ~76 us: at that size the kernel's ramp-up and drain depend on the clock)
    dec3_alone = decode3_alone_entry(ap, dev, peak, seed_offset=rank) if (rank == 0 and args.groups is None) else None
    torch.cuda.empty_cache()
    w_full = wl.workload(HEADLINE_CFG)
    free, _ = torch.cuda.mem_get_info()
    G = args.groups or fit_groups(w_full, 4 * w_full.D * (w_full.K + w_full.W) + 4 * w_full.C * (w_full.K + w_full.W) + 4,
                                  int(free * 0.9))
    w = w_full.with_groups(G)
    p = ap.make_params(w.K, w.W)
    X = wl.queries(w, dev, seed_offset=rank)
    Xt = torch.empty((w.G, w.W, w.D), device=dev)
    Yt = wl.gaussian_predictions(w, dev)
    mask_np = wl.masks(w, seed_offset=rank)
    mask = ap.mask_tensor(mask_np, dev)
    Yh = torch.empty((w.G, w.K, w.C), device=dev)
    enc_b, dec_b = encode_bytes(w), decode_bytes(w, mask_np)

    def step(evs=None):
        if evs:
            evs[0].record()
        ap.approxifer_encode(p, X, Xt)
        if evs:
            evs[1].record()
        ap.approxifer_decode(p, Yt, mask, Yh)
        if evs:
            evs[2].record()

    for _ in range(args.warmup):
        step()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    time.sleep(0.2)  # let the sampler take its first readings
    launches0 = ap.launch_count()
    e_begin.record()
    for s in range(args.steps):
        step(evs[s])
    e_end.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = ap.launch_count() - launches0
    clocks = sampler.stop()
    total_ms = e_begin.elapsed_time(e_end)
    if world > 1:
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    enc_times = [e[0].elapsed_time(e[1]) for e in evs]
    dec_times = [e[1].elapsed_time(e[2]) for e in evs]
    ms_per_step = total_ms / args.steps
    value = world * (enc_b + dec_b) / ms_per_step / 1e6
    wait_timeouts = ap.device_wait_timeouts()
    del X, Xt, Yt, Yh
    torch.cuda.empty_cache()

    kernels = [
        kernel_entry("encode_kernel", HEADLINE_NAME + " (inside the timed steps)", enc_b, enc_times, peak, w.G),
        kernel_entry("decode_staged_kernel", HEADLINE_NAME + " (inside the timed steps, right after the encoder)", dec_b, dec_times, peak, w.G),
    ]
    if rank == 0 and args.groups is None:
        kernels.append(dec3_alone)
        kernels.append(decode4_entry(ap, dev, peak))

    # end to end through the host-buffer entry points, on every rank (max over ranks, like the device figure)
    e2e = None
    if not args.no_e2e and args.groups is None:
        we = w_full.with_groups(min(E2E_GROUPS, w.G))
        try:
            ms, h2d, d2h, l_e2e, nb_e2e = run_e2e(ap, dev, we, steps=3, warmup=1)
        except RuntimeError as exc:  # e.g. not enough pinned host memory for every rank
            ms, h2d, d2h, l_e2e, nb_e2e = float("inf"), 0, 0, 0, 0
            sys.stderr.write("rank %d: end-to-end measurement failed: %s\n" % (rank, exc))
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        if ms != float("inf"):
            e2e = {"value": world * nb_e2e / ms / 1e6, "unit": UNIT, "ms_per_step": ms,
                   "h2d_bytes_per_step": world * h2d, "d2h_bytes_per_step": world * d2h, "gpu_launches_per_step": world * l_e2e,
                   "groups_per_step": world * we.G,
                   "note": "approxifer_encode_host + approxifer_decode_host on every rank, pinned host buffers, 512 MiB device "
                           "workspace, 4 streams; PCIe-bound.  Each end-to-end step takes %d of the %d groups of the headline "
                           "workload: pinned host buffers for all of them would be 79 GB per rank, and the rate of a "
                           "PCIe-bound pipeline does not depend on the number of groups" % (we.G, w_full.G)}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    enc = kernels[0]
    line = {}
    if not args.no_others and world == 1 and args.groups is None:
        line["others"] = other_workloads(ap, dev, peak)
        line["decode_grid_3GB"] = decode_grid(ap, dev)
        line["locate_grid"] = locate_grid(ap, dev)
        line["host_cost"] = host_cost(ap, dev)
        line["fma_peak"] = fma_peak(ap, dev)
    line.update({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": HEADLINE_NAME + "; G=%d groups per GPU; step = encode + decode" % w.G,
                   "groups_per_gpu": w.G,
                   "l2": "inputs (29.6 GB of queries, 0.33 GB of predictions per step) are far larger than the 126 MB L2; no flush needed",
                   "parallelism": "groups sharded over GPUs, no collective" if world > 1 else "1 GPU"},
        "groups_per_s": world * w.G / ms_per_step * 1e3,
        "frac_of_8TBps": value / world / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "encode_kernel", "achieved": enc["achieved"], "peak": peak, "unit": "GB/s",
                     "frac": enc["frac"], "frac_of_8TBps": enc["frac_of_8TBps"], "peak_source": peak_src,
                     "traffic": ENCODE_TRAFFIC_PER_GROUP * w.G if ENCODE_TRAFFIC_PER_GROUP else None,
                     "traffic_source": ENCODE_TRAFFIC_SOURCE,
                     "algorithmic_bytes_per_launch": enc_b,
                     "kernels": kernels},
        "clocks": clocks,
        "gpu_launches": launches,
        "wait_timeouts": wait_timeouts,
    })
    if cpu is not None:
        line["cpu_baseline"] = cpu
    line["e2e"] = e2e
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
