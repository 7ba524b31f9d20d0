#!/usr/bin/env python
"""Benchmark of the fused lossy aggregate + step + broadcast (+ drift) pass.

Headline: one "step" = one call of lossy_fused_step over one LLaMA-2-7B-decoder-layer-shaped bucket
(W=8 workers, bf16 gradients, fp32 master + Adam, bf16 replicas, packets of 2048 elements,
Bernoulli drop p=0.1) with all state resident in HBM. The metric is algorithmic HBM bytes
moved per second:

    bytes/step = (1-p)*W*n*gb + 24*n + W*n*rb      (delivered gradient packets are read once,
                                                    theta/m/v are read and written, every
                                                    replica packet is either written or read;
                                                    with owner-elided replicas W-1 instead of W)

Prints ONE JSON line. After the headline the same process measures the other benchmark
configurations and adds them to the line as `configs` (each with its own time, GB/s, fractions of the
measured and of the datasheet peak, the kernel build that ran and the sampled clocks):
    1  W=4 fp32 SGD, 40 MB per step (L2-resident, launch-bound): steps/s eager and as a CUDA graph
    3  W=64 on the layer bucket at p = 0.01 and 0.1
    4  the full 7B-shaped parameter set, 34 buckets streamed with owner-elided replicas (178 GB resident)
    5  W=16: packet size {256,1024,2048,4096} x p {0,0.01,0.05,0.1,0.3}, plus few-worker small-packet points
`--configs` picks the groups (also: wsweep, alg1, unfused, closed_loop; `none` = headline only).

`--impl reference` times the CPU oracle (as it stands) on a bounded sample. With --gpus N > 1 (torchrun,
one process per GPU) every rank runs its own bucket (weak scaling, no data-path collective); the W squared
drift sums are all-reduced once per timed region.
"""
from __future__ import annotations

import argparse
import concurrent.futures
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

import torch  # noqa: E402

import workload  # noqa: E402

METRIC = "lossy aggregate+step+broadcast HBM GB/s"
WORKLOAD = "cfg2_w8_layer_adam"
FALLBACK_HBM_GBS = 6650.0
DATASHEET_HBM_GBS = 8000.0
CPU_SAMPLE_PACKETS = 16384
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "fused_step_dram_traffic.txt")


def algorithmic_bytes(w: workload.Workload, n: int | None = None, *, elided: bool = False, alg1: bool = False) -> float:
    n = w.n if n is None else n
    gb = 2 if w.grad_dtype == "bf16" else 4
    rb = 2 if w.replica_dtype == "bf16" else 4
    opt = 24 if w.optimizer == "adam" else 8
    copies = w.W - 1 if elided else w.W           # owner-elided replicas: the owner keeps no copy of its shard
    # Algorithm 1 mode: the saved aggregate is read on a drop and written on a keep: 4 more bytes per element
    return (1.0 - w.p) * w.W * n * gb + opt * n + copies * n * rb + (4 * n if alg1 else 0)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def ncu_traffic(plan: str, w: workload.Workload):
    """DRAM bytes of one launch from the committed ncu summary, scaled by elements; None (with the reason)
    when the summary was taken on another kernel build or another workload shape than the one that ran."""
    try:
        rows = [ln.split("|") for ln in open(TRAFFIC_FILE) if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None, "no ncu summary committed"
    for r in rows:
        f = [x.strip() for x in r]
        if len(f) < 7:
            continue
        wl, build, elems, dram = f[0], f[1], int(f[2]), float(f[3])
        if wl == f"W={w.W} P={w.packet_elems} p={w.p} {w.grad_dtype}/{w.replica_dtype} {w.optimizer}":
            if build != plan:
                return None, f"the committed ncu capture is of build '{build}', this run used '{plan}'"
            return dram * w.n / elems, f"ncu small case of {elems} elements scaled by elements (commit {f[5]})"
    return None, "no ncu capture of this workload shape"


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region (read-only query)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


def gen_grads(w, step, device, e0=0, e1=None):
    e1 = w.n if e1 is None else e1
    return [workload.grad_slab(w, step, i, e0, e1, device) for i in range(w.W)]


def tdt(name):
    return torch.bfloat16 if name == "bf16" else torch.float32


def static_config(w, world=1, strong=False, full_n=None):
    """What is measured, in words and numbers that do not depend on the run (both arms print the same)."""
    B = algorithmic_bytes(w)
    return {"workload": w.name, "W": w.W, "n": w.n, "packet_elems": w.packet_elems, "p": w.p,
            "optimizer": w.optimizer, "grad_dtype": w.grad_dtype, "replica_dtype": w.replica_dtype,
            "bytes_per_step": B,
            "parallelism": (f"one bucket in {world} packet ranges, one per GPU" if strong
                            else f"{world} independent bucket(s), one per GPU"),
            "l2": "no flush: each step streams %.1f GB of state, far larger than the 126 MB L2; "
                  "two gradient sets alternate" % (B / 1e9)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the one place besides the tests and the smoke check that runs oracle/)
# ------------------------------------------------------------------------------------------------
def _np_grads(gs):
    return [x.cpu().view(torch.int16).numpy().view("uint16") if x.dtype == torch.bfloat16 else x.cpu().numpy()
            for x in gs]


def _make_oracle(w, k0, n_slab, dev):
    from oracle import oracle as O

    e0 = k0 * w.packet_elems
    th = workload.theta0_slab(w, e0, e0 + n_slab, dev).cpu().numpy()
    return O.Oracle(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                    grad_dtype=O.BF16 if w.grad_dtype == "bf16" else O.F32,
                    replica_dtype=O.BF16 if w.replica_dtype == "bf16" else O.F32,
                    optimizer=O.ADAM if w.optimizer == "adam" else O.SGD, theta0=th, lr=w.lr, beta1=w.beta1,
                    beta2=w.beta2, eps=w.eps, k0=k0, n_slab=n_slab)


def oracle_arm(w, steps, warmup, sample_packets):
    """Time the CPU oracle, as it stands, single-threaded, on the first `sample_packets` packets."""
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    n_slab = min(w.n, sample_packets * w.packet_elems)
    orc = _make_oracle(w, 0, n_slab, dev)
    sets = [_np_grads(gen_grads(w, s, dev, 0, n_slab)) for s in (1, 2)]
    for t in range(1, warmup + 1):
        orc.step(t, sets[t % 2], want_ghat=False)
    t0 = time.perf_counter()
    for t in range(warmup + 1, warmup + steps + 1):
        orc.step(t, sets[t % 2], want_ghat=False)
    dt = time.perf_counter() - t0
    gbs = algorithmic_bytes(w, n_slab) * steps / dt / 1e9
    sample = (f"first {n_slab // w.packet_elems} of {w.K} packets ({n_slab} elements x {w.W} workers), "
              f"{steps} steps, one thread, {dt:.1f} s of CPU work")
    return {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
            "ms_per_step": dt / steps * 1e3}


def oracle_all_cores(w, steps, slab_packets, max_threads=128):
    """The same unchanged oracle on every host core: disjoint packet slabs (packets are independent), one
    thread per slab; the C routine runs outside the interpreter lock."""
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    threads = max(1, min(cores, max_threads, w.K // slab_packets))
    n_slab = slab_packets * w.packet_elems
    jobs = []
    for r in range(threads):
        k0 = r * slab_packets
        e0 = k0 * w.packet_elems
        sets = [_np_grads(gen_grads(w, s, dev, e0, e0 + n_slab)) for s in (1, 2)]
        jobs.append((_make_oracle(w, k0, n_slab, dev), sets))

    def work(job):
        orc, sets = job
        for t in range(1, steps + 1):
            orc.step(t, sets[t % 2], want_ghat=False)

    with concurrent.futures.ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, [(j[0], j[1]) for j in jobs[:1]]))          # first touch / warm-up of one slab
        t0 = time.perf_counter()
        list(ex.map(work, jobs))
        dt = time.perf_counter() - t0
    gbs = algorithmic_bytes(w, n_slab) * threads * steps / dt / 1e9
    return {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": (f"{threads} threads (host reports {cores} usable cores), each its own slab of {slab_packets} "
                       f"packets ({n_slab} elements x {w.W} workers), {steps} steps, {dt:.1f} s wall")}


# ------------------------------------------------------------------------------------------------
# GPU measurement helpers
# ------------------------------------------------------------------------------------------------
class Bucket:
    """Device state of one bucket; reusable for several workloads of the same n and up to `W` workers."""

    def __init__(self, n, W, gdt, rdt, adam, dev, elided_for=None):
        self.n, self.W, self.dev = n, W, dev
        self.master = torch.empty(n, dtype=torch.float32, device=dev)
        self.m = torch.zeros(n, dtype=torch.float32, device=dev) if adam else None
        self.v = torch.zeros(n, dtype=torch.float32, device=dev) if adam else None
        self.rdt = rdt
        self.replicas = None if elided_for is not None else [torch.empty(n, dtype=rdt, device=dev) for _ in range(W)]
        self.norms = torch.zeros(W, dtype=torch.float32, device=dev)
        self.sumsq = torch.zeros(W, dtype=torch.float64, device=dev)

    def reset(self, w, L=None, ctx=None):
        """theta_0 of the workload, zero moments, synchronised replicas (drift 0)."""
        self.master.copy_(workload.theta0_slab(w, 0, w.n, self.dev))
        if self.m is not None:
            self.m.zero_(); self.v.zero_()
        wire = self.master.to(self.rdt)
        if ctx is not None:        # owner-elided: replica i is the bucket without the packets worker i owns
            pps = (w.K + w.W - 1) // w.W
            self.replicas = []
            for i in range(w.W):
                lo, hi = min(w.n, i * pps * w.packet_elems), min(w.n, (i + 1) * pps * w.packet_elems)
                r = torch.cat([wire[:lo], wire[hi:]])
                assert r.numel() == L.lossy_replica_elems(ctx, i)
                self.replicas.append(r)
        else:
            for i in range(w.W):
                self.replicas[i].copy_(wire)
        del wire


def make_ctx(L, w, flags=0, **kw):
    return L.lossy_init(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                        grad_dtype=tdt(w.grad_dtype), replica_dtype=tdt(w.replica_dtype), optimizer=w.optimizer,
                        lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, packet_base=w.packet_base, flags=flags, **kw)


def time_point(L, w, bucket, grad_sets, steps, warmup=3, *, flags=0, alg1=False, graph=False, peak=FALLBACK_HBM_GBS):
    """One workload on a prepared bucket: `steps` fused steps with drift norms between two CUDA events."""
    ctx = make_ctx(L, w, flags)
    bucket.reset(w)
    reps, W = bucket.replicas[:w.W], w.W
    norms, worst = bucket.norms[:W], torch.zeros(W, device=bucket.dev)
    prev = torch.zeros_like(bucket.master) if alg1 else None
    stream = torch.cuda.current_stream()

    # the arguments of a step are marshalled once per gradient set (the binding's prepared call): a step is then
    # one foreign call, which is what a launch-bound bucket needs
    calls = [L.lossy_fused_step_prepared(ctx, gs[:W], bucket.master, bucket.m, bucket.v, reps, norms=norms,
                                         ghat_prev=prev, stream=stream) for gs in grad_sets]

    def step(t):
        calls[t % len(calls)](t)

    t = 0
    for _ in range(max(3, warmup)):
        t += 1
        step(t)
        torch.maximum(worst, norms, out=worst)
    torch.cuda.synchronize()
    # an event after every step (per-step minimum), except in the launch-bound case, where recording it costs a
    # fifth of a step: there only the two ends are recorded
    every = not graph
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1 if every else 2)]
    ev[0].record(stream)
    for i in range(steps):
        t += 1
        step(t)
        if every:
            ev[i + 1].record(stream)
    if not every:
        ev[1].record(stream)
    torch.cuda.synchronize()
    torch.maximum(worst, norms, out=worst)
    L.lossy_device_status(ctx)
    ms = ev[0].elapsed_time(ev[-1]) / steps
    per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)] if every else [ms]
    out = {"workload": w.name + ("[alg1]" if alg1 else ""), "W": W, "P": w.packet_elems, "p": w.p, "n": w.n,
           "steps": steps, "ms_per_step": ms, "min_ms": min(per), "steps_per_s": 1e3 / ms}
    B = algorithmic_bytes(w, alg1=alg1)
    out.update({"GBps": B / (ms * 1e-3) / 1e9, "frac": B / (ms * 1e-3) / 1e9 / peak,
                "frac_datasheet": B / (ms * 1e-3) / 1e9 / DATASHEET_HBM_GBS,
                "max_drift_norm": float(worst.max()), "build": L.lossy_describe_plan(ctx, True)})
    if graph:
        # launch-bound case: capture `steps` consecutive steps once, replay them as one graph launch
        side = torch.cuda.Stream()
        side_calls = [L.lossy_fused_step_prepared(ctx, gs[:W], bucket.master, bucket.m, bucket.v, reps, norms=norms,
                                                  ghat_prev=prev, stream=side) for gs in grad_sets]
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    side_calls[(t + 1 + i) % len(side_calls)](t + 1 + i)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nrep = 20
        e0.record()
        for _ in range(nrep):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        L.lossy_device_status(ctx)
        out["steps_per_s_cuda_graph"] = nrep * steps / (e0.elapsed_time(e1) * 1e-3)
        out["us_per_step_cuda_graph"] = e0.elapsed_time(e1) * 1e3 / (nrep * steps)
        del g
    L.lossy_destroy(ctx)
    return out


def free_device():
    import gc

    gc.collect()
    torch.cuda.empty_cache()


def group_small_and_w64(L, dev, peak, which):
    """Configuration 1 (L2-resident, launch-bound) and configuration 3 (W = 64 on the layer bucket)."""
    cfg = workload.baseline_workloads()
    out = []
    if "1" in which:
        w = cfg["cfg1_w4_sgd_f32"]
        b = Bucket(w.n, w.W, torch.float32, torch.float32, False, dev)
        sets = [gen_grads(w, s, dev) for s in (1, 2)]
        r = time_point(L, w, b, sets, w.steps, graph=True, peak=peak)
        r["note"] = ("40 MB per step: L2-resident and launch-bound; the figure of merit is steps/s (eager: one launch per "
                     "step through the binding; CUDA graph: the configuration's 10 steps captured and replayed)")
        out.append(r)
        del b, sets
        free_device()
    if "3" in which:
        b = sets = None
        for name in ("cfg3_w64_layer_p01", "cfg3_w64_layer_p10"):
            w = cfg[name]
            if b is None:
                b = Bucket(w.n, w.W, torch.bfloat16, torch.bfloat16, True, dev)
                sets = [gen_grads(w, 1, dev)]          # 26 GB: one set (every step streams 54 GB, far beyond L2)
            out.append(time_point(L, w, b, sets, 5, peak=peak))
        del b, sets
        free_device()
    return out


def group_sweep(L, dev, peak, full=True):
    """Configuration 5 (W = 16: packet size x drop rate) and the few-worker / small-packet / high-loss points."""
    base = workload.baseline_workloads()["cfg5_w16_layer_sweep"]
    n, Wmax = workload.LAYER_ELEMS, 17
    b = Bucket(n, Wmax, torch.bfloat16, torch.bfloat16, True, dev)
    wgen = workload.scaled(base, n, W=Wmax)
    sets = [gen_grads(wgen, s, dev) for s in (1, 2)]
    out = []
    pts = [(16, P, p) for P in (256, 1024, 2048, 4096) for p in (0.0, 0.01, 0.05, 0.1, 0.3)]
    extra = [(W, P, p) for W in (2, 3, 4) for P in (256, 512) for p in (0.1, 0.3)] + [(8, 512, 0.3), (16, 256, 0.2), (17, 2048, 0.5)]
    for W, P, p in pts + (extra if full else []):
        w = workload.scaled(base, n, W=W, packet_elems=P, p=p,
                            name=f"cfg5_w16_P{P}_p{p}" if W == 16 and (W, P, p) in pts else f"extra_w{W}_P{P}_p{p}")
        out.append(time_point(L, w, b, sets, base.steps, peak=peak))
    del b, sets
    free_device()
    return out


def group_wsweep(L, dev, peak):
    """The config-2 bucket with the worker count varied, at two loss rates."""
    base = workload.baseline_workloads()["cfg2_w8_layer_adam"]
    out = []
    for W in (1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64):
        b = Bucket(base.n, W, torch.bfloat16, torch.bfloat16, True, dev)
        wg = workload.scaled(base, base.n, W=W)
        sets = [gen_grads(wg, s, dev) for s in ((1, 2) if W <= 32 else (1,))]
        for p in (0.1, 0.3):
            out.append(time_point(L, workload.scaled(base, base.n, W=W, p=p, name=f"w{W}_p{p}"), b, sets, 10, peak=peak))
        del b, sets
        free_device()
    return out


def group_alg1(L, dev, peak):
    """Algorithm 1 mode on the config-2 bucket: packet-granular and shard-granular (P = n / W) drops."""
    base = workload.baseline_workloads()["cfg2_w8_layer_adam"]
    b = Bucket(base.n, base.W, torch.bfloat16, torch.bfloat16, True, dev)
    sets = [gen_grads(base, s, dev) for s in (1, 2)]
    out = []
    for P in (2048, workload.LAYER_ELEMS // 8):
        for p in (0.1, 0.3):
            w = workload.scaled(base, base.n, packet_elems=P, p=p, name=f"cfg2_w8_P{P}_p{p}")
            out.append(time_point(L, w, b, sets, 30, alg1=True, peak=peak))
    del b, sets
    free_device()
    return out


def group_unfused(L, dev, peak, elements=0, steps=20, warmup=3):
    """Each unfused entry point on its own: time and algorithmic GB/s of aggregate, step, broadcast, drift."""
    w = workload.baseline_workloads()["cfg2_w8_layer_adam"]
    if elements:
        w = workload.scaled(w, elements)
    gb, rb = (2 if w.grad_dtype == "bf16" else 4), (2 if w.replica_dtype == "bf16" else 4)
    adam = w.optimizer == "adam"
    ctx = make_ctx(L, w)
    b = Bucket(w.n, w.W, tdt(w.grad_dtype), tdt(w.replica_dtype), adam, dev)
    b.reset(w)
    grads = gen_grads(w, 1, dev)
    ghat = torch.zeros_like(b.master)
    count = torch.zeros(w.K, dtype=torch.uint8, device=dev)
    n, W, p = w.n, w.W, w.p
    calls = {
        "lossy_aggregate": (lambda t: L.lossy_aggregate(ctx, t, grads, ghat, count), (1 - p) * W * n * gb + 4 * n),
        "lossy_step": (lambda t: L.lossy_step(ctx, t, ghat, count, b.master, b.m, b.v), (28 if adam else 12) * n),
        "lossy_broadcast": (lambda t: L.lossy_broadcast(ctx, t, b.master, b.replicas), 4 * n + ((W - 1) * (1 - p) + 1) * n * rb),
        "drift_norms": (lambda t: L.drift_norms(ctx, b.master, b.replicas, b.norms), 4 * n + W * n * rb),
    }
    out = []
    for name, (fn, nbytes) in calls.items():
        for t in range(1, warmup + 1):
            fn(t)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(warmup + 1, warmup + steps + 1):
            fn(t)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        out.append({"workload": w.name, "call": name, "ms": ms, "GBps": nbytes / (ms * 1e-3) / 1e9,
                    "frac": nbytes / (ms * 1e-3) / 1e9 / peak})
    L.lossy_device_status(ctx)
    L.lossy_destroy(ctx)
    del b, grads, ghat
    free_device()
    return out


def group_full_model(L, dev, peak, steps=20, warmup=2, layers=32, elide=True):
    """Configuration 4: the full LLaMA-2-7B-shaped parameter set (32 decoder-layer buckets + embedding + head)
    streamed bucket by bucket. One context per bucket with its own shard map and a running global packet id;
    owner-elided replicas (worker i keeps no copy of its own shard) make the whole model fit one GPU. One
    gradient buffer is reused for every bucket (the masks still differ: they hash the global packet id).
    Model-level drift = sqrt of the squared sums added over the buckets."""
    base = workload.baseline_workloads()["cfg4_w8_full_model"]
    emb = 32000 * 4096
    sizes = [workload.LAYER_ELEMS] * layers + [emb, emb]
    flags = L.LOSSY_REPLICA_SKIP_OWNER if elide else 0
    free0, total = torch.cuda.mem_get_info()
    ctxs, state, pb = [], [], 0
    note = None
    try:
        big = workload.scaled(base, workload.LAYER_ELEMS)
        grads = gen_grads(big, 1, dev)
        for bi, n in enumerate(sizes):
            w = workload.scaled(base, n, packet_base=pb, seed=base.seed + bi, name=f"cfg4_bucket{bi}")
            ctx = make_ctx(L, w, flags)
            b = Bucket(n, w.W, torch.bfloat16, torch.bfloat16, True, dev, elided_for=ctx if elide else None)
            b.reset(w, L, ctx if elide else None)
            ctxs.append((ctx, w))
            state.append(b)
            pb += w.K
            if bi % 8 == 7:
                torch.cuda.empty_cache()
        torch.cuda.empty_cache()
        free1, _ = torch.cuda.mem_get_info()
        sumsq = torch.zeros(base.W, dtype=torch.float64, device=dev)
        worst = torch.zeros(base.W, dtype=torch.float64, device=dev)
        total_bytes = sum(algorithmic_bytes(w, elided=elide) for _, w in ctxs)

        def model_step(t):
            sumsq.zero_()
            for (ctx, w), b in zip(ctxs, state):
                L.lossy_fused_step(ctx, t, [g[:w.n] for g in grads], b.master, b.m, b.v, b.replicas, sumsq=sumsq)
            torch.maximum(worst, sumsq, out=worst)

        t = 0
        for _ in range(warmup):
            t += 1
            model_step(t)
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            t += 1
            model_step(t)
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = ev[0].elapsed_time(ev[-1]) / steps
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        for ctx, _ in ctxs:
            L.lossy_device_status(ctx)
        gbs = total_bytes / (ms * 1e-3) / 1e9
        res = {"workload": "cfg4_w8_full_model" if layers == 32 else f"cfg4_cut_{layers}_layers_plus_embedding_and_head",
               "W": base.W, "P": base.packet_elems, "p": base.p, "buckets": len(sizes), "n": sum(sizes),
               "replica_layout": "owner-elided (LOSSY_REPLICA_SKIP_OWNER)" if elide else "full",
               "steps": steps, "launches_per_step": len(sizes), "ms_per_step": ms, "min_ms": min(per),
               "steps_per_s": 1e3 / ms, "GBps": gbs, "frac": gbs / peak, "frac_datasheet": gbs / DATASHEET_HBM_GBS,
               "bytes_per_step": total_bytes, "max_drift_norm": float(worst.max().sqrt()),
               "build": L.lossy_describe_plan(ctxs[0][0], True),
               "device_memory": {"total_GB": total / 1e9, "free_before_GB": free0 / 1e9, "free_resident_GB": free1 / 1e9,
                                 "resident_GB": (free0 - free1) / 1e9},
               "gradients": "one reusable W x bucket buffer (3.24 GB), the same values for every bucket; the drop masks "
                            "differ per bucket (they hash the global packet id)"}
    except torch.OutOfMemoryError as e:          # the allocation was refused: report it, the caller may try a cut
        res = {"workload": "cfg4_w8_full_model", "refused": f"device memory: {str(e)[:200]}", "layers": layers,
               "device_memory": {"total_GB": total / 1e9, "free_before_GB": free0 / 1e9}}
    finally:
        for ctx, _ in ctxs:
            L.lossy_destroy(ctx)
        state.clear()
        grads = None
        free_device()
    if note:
        res["note"] = note
    return res


def closed_loop_run(p, *, W, n, P, steps, optimizer, lr, gdt, rdt, seed=0, sigma_noise=1.0):
    """The method in closed loop on a synthetic objective (the paper's Table 1 trend in miniature): every step
    worker i evaluates the gradient of 1/2 sum a (theta - x*)^2 at ITS OWN replica (stale where broadcasts were
    lost) plus fresh noise (lossy_closed_loop_grads), then the fused lossy step aggregates, updates and broadcasts.
    Returns (objective at the owners' parameters, objective at the replicas, largest drift norm), the objectives
    averaged over the last quarter of the run."""
    import paper_2507_07114_b200 as L

    dev = torch.device("cuda")
    ctx = L.lossy_init(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=gdt, replica_dtype=rdt,
                       optimizer=optimizer, lr=lr, beta1=0.9, beta2=0.95, eps=1e-8)
    curv = 0.5 + (workload.normal_f32(seed, 4000, 0, 0, n, 1.0, dev).abs() % 1.0)          # a in [0.5, 1.5)
    target = workload.normal_f32(seed, 4001, 0, 0, n, 1.0, dev)
    master = target + workload.normal_f32(seed, 4002, 0, 0, n, 1.0, dev)
    adam = optimizer == "adam"
    m = torch.zeros_like(master) if adam else None
    v = torch.zeros_like(master) if adam else None
    reps = [master.to(rdt) for _ in range(W)]
    grads = [torch.empty(n, dtype=gdt, device=dev) for _ in range(W)]
    norms = torch.zeros(W, device=dev)
    worst = 0.0
    tail_owner, tail_rep = [], []
    for t in range(1, steps + 1):
        noise = [workload.normal_f32(seed, 5000 + i, t, 0, n, sigma_noise, dev).to(gdt) for i in range(W)]
        L.lossy_closed_loop_grads(ctx, curv, target, noise, reps, grads)
        L.lossy_fused_step(ctx, t, grads, master, m, v, reps, norms=norms)
        worst = max(worst, float(norms.max()))
        if t > steps - steps // 4:
            tail_owner.append(float(0.5 * (curv * (master - target) ** 2).mean()))
            tail_rep.append(float(sum(0.5 * (curv * (r.float() - target) ** 2).mean() for r in reps) / W))
    L.lossy_device_status(ctx)
    L.lossy_destroy(ctx)
    return sum(tail_owner) / len(tail_owner), sum(tail_rep) / len(tail_rep), worst


def group_closed_loop(elements=2048 * 4096, steps=200, W=8, P=2048):
    out = []
    for name, opt, lr, gdt, rdt in (("sgd_fp32", "sgd", 0.1, torch.float32, torch.float32),
                                    ("adam_bf16", "adam", 3e-3, torch.bfloat16, torch.bfloat16)):
        base = None
        for p in (0.0, 0.1, 0.2, 0.3, 0.4):
            owner, rep, drift = closed_loop_run(p, W=W, n=elements, P=P, steps=steps, optimizer=opt, lr=lr, gdt=gdt, rdt=rdt)
            base = base or (owner, rep)
            out.append({"run": name, "p": p, "objective_owner": owner, "change_vs_lossless_pct": 100 * (owner / base[0] - 1),
                        "objective_replicas": rep, "replica_change_pct": 100 * (rep / base[1] - 1), "max_drift_norm": drift})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD)
    ap.add_argument("--elements", type=int, default=0, help="override the bucket size (profiling of a small case)")
    ap.add_argument("--p", type=float, default=None, help="override the drop probability")
    ap.add_argument("--workers", type=int, default=0, help="override W")
    ap.add_argument("--packet-elems", type=int, default=0, help="override the packet size")
    ap.add_argument("--strong", action="store_true",
                    help="N > 1: split ONE bucket into packet ranges, one per rank (default: one bucket per rank)")
    ap.add_argument("--range", default="", metavar="R/G",
                    help="single process: run only packet range R of G of the bucket (what rank R of a G-GPU --strong job runs)")
    ap.add_argument("--register-path", action="store_true", help="time the register-path kernel, not the bulk-copy pipeline")
    ap.add_argument("--skip-owner", action="store_true", help="headline with owner-elided replicas (LOSSY_REPLICA_SKIP_OWNER)")
    ap.add_argument("--gather-path", action="store_true", help="small packets: force the gather pipeline (LOSSY_GATHER_PATH)")
    ap.add_argument("--e2e-steps", type=int, default=-1, help="steps of the host-buffer leg (default: min(steps, 10))")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-timed-region", action="store_true",
                    help="bracket the headline's timed region with cudaProfilerStart/Stop (for ncu --profile-from-start off)")
    ap.add_argument("--cpu-sample-packets", type=int, default=CPU_SAMPLE_PACKETS)
    ap.add_argument("--configs", default=None,
                    help="comma list of the further configurations measured after the headline: 1,3,4,5 (default for the "
                         "unmodified headline on one GPU), wsweep, alg1, unfused, closed_loop; 'none' = headline only")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world == 1 and "RANK" not in os.environ:
        # convenience: relaunch under torchrun, one process per GPU
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), *sys.argv]
        raise SystemExit(subprocess.call(cmd))

    w = workload.baseline_workloads()[args.workload]
    if args.elements:
        w = workload.scaled(w, args.elements)
    if args.p is not None:
        w = workload.scaled(w, w.n, p=args.p)
    if args.workers:
        w = workload.scaled(w, w.n, W=args.workers)
    if args.packet_elems:
        w = workload.scaled(w, w.n, packet_elems=args.packet_elems)
    warmup = max(3, args.warmup)
    pristine = (args.workload == WORKLOAD and not args.elements and args.p is None and not args.workers
                and not args.packet_elems and not args.register_path and not args.range and not args.skip_owner)
    dtypes = {"grad": w.grad_dtype, "replica": w.replica_dtype, "master_and_moments": "f32", "accumulate": "f32"}

    if args.impl == "reference":
        if rank != 0:
            return
        r = oracle_arm(w, args.steps, warmup, args.cpu_sample_packets)
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "GB/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "dtypes": dtypes, "data": "synthetic",
                "config": static_config(w, max(1, args.gpus)),
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
                "e2e": {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import paper_2507_07114_b200 as L

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1 or "WORLD_SIZE" in os.environ:         # under torchrun, also with a single rank
        import torch.distributed as dist
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)

    full_w, full_n, e_off, rng_kw = w, w.n, 0, {}
    strong = args.strong and world > 1
    if strong or args.range:
        # strong scaling: the ranks share one bucket, each a contiguous packet range for all W workers
        r_, g_ = (int(x) for x in args.range.split("/")) if args.range else (rank, world)
        pr = L.packet_range_config(w.n, w.packet_elems, r_, g_)
        e_off = pr["e0"]
        rng_kw = {"shard_packet0": pr["shard_packet0"], "bucket_packets": pr["bucket_packets"]}
        w = workload.scaled(w, pr["n"])
    else:
        # weak scaling: every rank simulates its own bucket; global packet ids continue across ranks
        w = workload.scaled(w, w.n, packet_base=rank * w.K, seed=w.seed)
    gdt, rdt = tdt(w.grad_dtype), tdt(w.replica_dtype)
    adam = w.optimizer == "adam"
    flags = ((L.LOSSY_REGISTER_PATH if args.register_path else 0) | (L.LOSSY_REPLICA_SKIP_OWNER if args.skip_owner else 0)
             | (L.LOSSY_GATHER_PATH if args.gather_path else 0))
    ctx = make_ctx(L, w, flags, **rng_kw)
    plan = L.lossy_describe_plan(ctx, True)       # the build the library's launch policy picks for this workload
    master = workload.theta0_slab(w, e_off, e_off + w.n, dev)
    m = torch.zeros_like(master) if adam else None
    v = torch.zeros_like(master) if adam else None
    if args.skip_owner:
        Kb = rng_kw.get("bucket_packets", w.K)
        pps = (Kb + w.W - 1) // w.W
        owner = (rng_kw.get("shard_packet0", 0) + torch.arange(w.n, device=dev) // w.packet_elems) // pps
        wire = master.to(rdt)
        replicas = [wire[owner != i].clone() for i in range(w.W)]
        del owner, wire
    else:
        replicas = [master.to(rdt) for _ in range(w.W)]
    norms = torch.zeros(w.W, dtype=torch.float32, device=dev)
    sumsq = torch.zeros(w.W, dtype=torch.float64, device=dev)
    grad_sets = [gen_grads(w, s, dev, e_off, e_off + w.n) for s in (1, 2)]   # 2 sets, each larger than L2, alternate
    stream = torch.cuda.current_stream()

    def one_step(t):
        L.lossy_fused_step(ctx, t, grad_sets[t % 2], master, m, v, replicas, norms=norms, sumsq=sumsq)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    t = 0
    for _ in range(warmup):
        t += 1
        one_step(t)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = L.lossy_kernel_launches(ctx)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    if args.profile_timed_region:        # a profiler started with --profile-from-start off sees the timed region only
        torch.cuda.profiler.start()
    ev[0].record(stream)
    for i in range(args.steps):
        t += 1
        one_step(t)
        ev[i + 1].record(stream)
    if dist is not None:
        dist.all_reduce(sumsq, op=dist.ReduceOp.SUM)        # the only exchange: W doubles per job
    barrier()
    if args.profile_timed_region:
        torch.cuda.profiler.stop()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_launch_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    launches = L.lossy_kernel_launches(ctx) - launches0
    clocks = sampler.stop()

    tmax = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    total_ms = float(tmax.item())
    B = algorithmic_bytes(w, elided=args.skip_owner)          # this rank's bytes per step
    B_job = algorithmic_bytes(full_w, full_n, elided=args.skip_owner) if strong else B * world
    value = B_job * args.steps / (total_ms * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    avg_launch_ms = sum(per_launch_ms) / len(per_launch_ms)
    achieved = B / (avg_launch_ms * 1e-3) / 1e9

    # ---- end to end: gradients start in pinned host memory, norms end in host memory ----------
    e2e_steps = args.e2e_steps if args.e2e_steps >= 0 else min(args.steps, 10)
    e2e = None
    if e2e_steps > 0:
        host_grads = [g.cpu().pin_memory() for g in grad_sets[0]]
        host_norms = torch.zeros(w.W, dtype=torch.float32).pin_memory()
        dev_grads = None                                        # pinned buffers are read in place over PCIe
        for _ in range(2):
            t += 1
            L.lossy_fused_step_host(ctx, t, host_grads, dev_grads, master, m, v, replicas, norms, host_norms)
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            t += 1
            L.lossy_fused_step_host(ctx, t, host_grads, dev_grads, master, m, v, replicas, norms, host_norms)
        e1.record(stream)
        barrier()
        e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3 if world == 1 else 0.0)
        tm = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        e2e_ms = float(tm.item())
        e2e = {"value": B_job * e2e_steps / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
               # pinned gradients are read by the kernel itself: only delivered packets cross PCIe
               "h2d_bytes_per_step": int((1.0 - w.p) * sum(g.numel() * g.element_size() for g in host_grads)),
               "d2h_bytes_per_step": host_norms.numel() * 4, "steps": e2e_steps,
               "ms_per_step": e2e_ms / e2e_steps,
               "api": "lossy_fused_step_host (pinned host gradients read in place by the fused kernel, "
                      "dropped packets never transferred; norms -> host)"}
        del host_grads
    final_norm_max = float(norms.max().item())
    L.lossy_device_status(ctx)
    L.lossy_destroy(ctx)
    traffic, traffic_note = ncu_traffic(plan, w) if not (args.register_path or args.skip_owner or args.range) else (None, "non-default launch")

    # ---- the other benchmark configurations, in the same process ----------------------------------
    which = args.configs if args.configs is not None else ("1,3,4,5" if pristine and world == 1 else "none")
    which = set() if which == "none" else set(which.split(","))
    configs, extra = [], {}
    if which and rank == 0 and world == 1:
        del master, m, v, replicas, grad_sets
        free_device()

        def sampled(fn, *a, **k):
            s = ClockSampler(local_rank).start()
            try:
                rows = fn(*a, **k)
            except Exception as e:          # one group failing must not lose the headline
                rows = [{"error": f"{type(e).__name__}: {str(e)[:300]}"}]
                free_device()
            ck = s.stop()
            rows = rows if isinstance(rows, list) else [rows]
            for r in rows:
                r["clocks"] = ck
            return rows

        if which & {"1", "3"}:
            configs += sampled(group_small_and_w64, L, dev, peak, which)
        if "5" in which:
            configs += sampled(group_sweep, L, dev, peak)
        if "4" in which:
            rows = sampled(group_full_model, L, dev, peak)
            if "refused" in rows[0]:
                # the whole model was refused: the largest layer count that the free memory allows, as a cut
                free, _ = torch.cuda.mem_get_info()
                per_layer = workload.LAYER_ELEMS * (12 + 14)
                layers = int((free - 2 * 32000 * 4096 * 26 - 3.3e9 - 3e9) // per_layer)
                rows += sampled(group_full_model, L, dev, peak, layers=max(1, min(31, layers)))
            configs += rows
        if "wsweep" in which:
            extra["worker_sweep"] = sampled(group_wsweep, L, dev, peak)
        if "alg1" in which:
            extra["alg1"] = sampled(group_alg1, L, dev, peak)
        if "unfused" in which:
            extra["unfused"] = sampled(group_unfused, L, dev, peak, args.elements, steps=min(args.steps, 20))
        if "closed_loop" in which:
            extra["closed_loop"] = sampled(group_closed_loop)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        one = oracle_arm(w, 20, 1, args.cpu_sample_packets)
        allc = oracle_all_cores(w, 20, 1024)
        cpu = {k: allc[k] for k in ("value", "unit", "cores", "kind", "sample")}
        cpu["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if strong else "weak",
            "vs_baseline": None, "dtype": "f32", "dtypes": dtypes, "data": "synthetic",
            "steps_per_s": args.steps * (1 if strong else world) / (total_ms * 1e-3),
            "pct_of_hbm_peak": 100.0 * value / world / peak,
            "config": static_config(full_w if strong else workload.scaled(w, w.n, packet_base=0), world, strong),
            "observed": {"drift_norm_max_last_step": final_norm_max, "rank_elements": w.n,
                         "replica_layout": "owner-elided" if args.skip_owner else "full"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "frac_datasheet": achieved / DATASHEET_HBM_GBS,
                         "datasheet_peak": DATASHEET_HBM_GBS,
                         "traffic": traffic, "traffic_source": traffic_note,
                         "frac_of_traffic": (traffic / (avg_launch_ms * 1e-3) / 1e9 / peak) if traffic else None,
                         "peak_source": peak_src + " (MEASURED_PEAKS.json hbm_gbs)" if peak_src == "measured"
                         else peak_src, "kernel": ("lossy_kernel<AGG|STEP|BCAST|DRIFT>" if plan.startswith("register") else "lossy_fused_tma_kernel")
                         + " (drift norms finalised by its last block)", "build": plan,
                         "algorithmic_bytes_per_launch": B,
                         "avg_launch_ms": avg_launch_ms, "min_launch_ms": min(per_launch_ms)},
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "cpu_baseline": cpu,
        }
        if configs:
            line["configs"] = configs
        line.update(extra)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
