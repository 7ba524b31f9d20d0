"""Throughput and drift of the fused step over the benchmark configurations.

    python -m paper_2507_07114_b200.sweep [--configs 1,2,3,4,5,alg1,unfused] [--steps N]

Prints one line per point: algorithmic GB/s, fraction of the measured HBM copy peak, steps/s and the
largest per-replica drift norm seen. Inputs are the seeded synthetic workloads; state stays in HBM.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

import workload
from . import binding as L

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def algorithmic_bytes(w, alg1=False):
    gb = 2 if w.grad_dtype == "bf16" else 4
    rb = 2 if w.replica_dtype == "bf16" else 4
    b = (1.0 - w.p) * w.W * w.n * gb + (24 if w.optimizer == "adam" else 8) * w.n + w.W * w.n * rb
    # Algorithm 1 mode: the saved aggregate is read on a drop and written on a keep: 4 bytes per element
    return b + (4 * w.n if alg1 else 0)


def run_point(w, steps, warmup=3, grad_sets=2, alg1=False, graph=False):
    dev = torch.device("cuda")
    gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    rdt = torch.bfloat16 if w.replica_dtype == "bf16" else torch.float32
    adam = w.optimizer == "adam"
    ctx = L.lossy_init(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                       grad_dtype=gdt, replica_dtype=rdt, optimizer=w.optimizer, lr=w.lr, beta1=w.beta1,
                       beta2=w.beta2, eps=w.eps)
    master = workload.theta0_slab(w, 0, w.n, dev)
    m = torch.zeros_like(master) if adam else None
    v = torch.zeros_like(master) if adam else None
    reps = [master.to(rdt) for _ in range(w.W)]
    norms = torch.zeros(w.W, device=dev)
    worst = torch.zeros(w.W, device=dev)
    prev = torch.zeros_like(master) if alg1 else None

    def step(t):
        if alg1:
            L.lossy_fused_step_alg1(ctx, t, sets[t % grad_sets], prev, master, m, v, reps, norms=norms)
        else:
            L.lossy_fused_step(ctx, t, sets[t % grad_sets], master, m, v, reps, norms=norms)

    sets = [[workload.grad_slab(w, s, i, 0, w.n, dev) for i in range(w.W)] for s in range(1, grad_sets + 1)]
    t = 0
    for _ in range(warmup):
        t += 1
        step(t)
        torch.maximum(worst, norms, out=worst)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        t += 1
        step(t)
        torch.maximum(worst, norms, out=worst)
    e1.record()
    torch.cuda.synchronize()
    L.lossy_device_status(ctx)
    ms = e0.elapsed_time(e1) / steps
    graph_sps = None
    if graph:
        # launch-bound case: capture `steps` consecutive steps once, replay them as one graph launch
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    step(t + 1 + i)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        reps = 20
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        graph_sps = reps * steps / (e0.elapsed_time(e1) * 1e-3)
        L.lossy_device_status(ctx)
    plan = L.lossy_describe_plan(ctx, True)
    L.lossy_destroy(ctx)
    gbs = algorithmic_bytes(w, alg1) / (ms * 1e-3) / 1e9
    return {"workload": w.name + ("[alg1]" if alg1 else ""), "W": w.W, "P": w.packet_elems, "p": w.p, "ms_per_step": ms, "GBps": gbs,
            "frac_of_measured_peak": gbs / _peak(), "steps_per_s": 1e3 / ms, "max_drift_norm": float(worst.max()),
            "build": plan, **({"steps_per_s_cuda_graph": graph_sps} if graph_sps else {})}


def run_unfused(w, steps=20, warmup=3):
    """Each unfused entry point on its own: time and algorithmic GB/s of aggregate, step, broadcast, drift."""
    dev = torch.device("cuda")
    gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    rdt = torch.bfloat16 if w.replica_dtype == "bf16" else torch.float32
    gb, rb = (2 if w.grad_dtype == "bf16" else 4), (2 if w.replica_dtype == "bf16" else 4)
    adam = w.optimizer == "adam"
    ctx = L.lossy_init(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                       grad_dtype=gdt, replica_dtype=rdt, optimizer=w.optimizer, lr=w.lr, beta1=w.beta1,
                       beta2=w.beta2, eps=w.eps)
    master = workload.theta0_slab(w, 0, w.n, dev)
    m = torch.zeros_like(master) if adam else None
    v = torch.zeros_like(master) if adam else None
    reps = [master.to(rdt) for _ in range(w.W)]
    grads = [workload.grad_slab(w, 1, i, 0, w.n, dev) for i in range(w.W)]
    ghat = torch.zeros_like(master)
    count = torch.zeros(w.K, dtype=torch.uint8, device=dev)
    norms = torch.zeros(w.W, device=dev)
    n, W, p = w.n, w.W, w.p
    calls = {
        "lossy_aggregate": (lambda t: L.lossy_aggregate(ctx, t, grads, ghat, count), (1 - p) * W * n * gb + 4 * n),
        "lossy_step": (lambda t: L.lossy_step(ctx, t, ghat, count, master, m, v), (28 if adam else 12) * n),
        "lossy_broadcast": (lambda t: L.lossy_broadcast(ctx, t, master, reps), 4 * n + ((W - 1) * (1 - p) + 1) * n * rb),
        "drift_norms": (lambda t: L.drift_norms(ctx, master, reps, norms), 4 * n + W * n * rb),
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
                    "frac_of_measured_peak": nbytes / (ms * 1e-3) / 1e9 / _peak()})
    L.lossy_destroy(ctx)
    return out


def run_model_streamed(base, layers, steps, warmup=2):
    """Configuration 4's mechanism at (nearly) full scale: a model streamed bucket by bucket. One context per
    bucket with its own shard map and a running global packet id; one gradient buffer is reused for every bucket
    (the masks still differ: they hash the global packet id). Model-level drift = sqrt of the summed squares."""
    dev = torch.device("cuda")
    emb = 32000 * 4096
    sizes = [workload.LAYER_ELEMS] * layers + [emb, emb]
    ctxs, state, pb = [], [], 0
    for b, n in enumerate(sizes):
        w = workload.scaled(base, n, packet_base=pb, seed=base.seed + b)
        ctx = L.lossy_init(W=w.W, n=n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                           grad_dtype=torch.bfloat16, replica_dtype=torch.bfloat16, optimizer="adam", lr=w.lr,
                           beta1=w.beta1, beta2=w.beta2, eps=w.eps, packet_base=pb)
        master = workload.theta0_slab(w, 0, n, dev)
        state.append((master, torch.zeros_like(master), torch.zeros_like(master),
                      [master.to(torch.bfloat16) for _ in range(w.W)]))
        ctxs.append((ctx, w))
        pb += w.K
    big = workload.scaled(base, workload.LAYER_ELEMS)
    grads = [workload.grad_slab(big, 1, i, 0, big.n, dev) for i in range(base.W)]
    sumsq = torch.zeros(base.W, dtype=torch.float64, device=dev)
    worst = torch.zeros(base.W, dtype=torch.float64, device=dev)
    total_bytes = sum(algorithmic_bytes(w) for _, w in ctxs)

    def model_step(t):
        sumsq.zero_()
        for (ctx, w), (master, m, v, reps) in zip(ctxs, state):
            L.lossy_fused_step(ctx, t, [g[:w.n] for g in grads], master, m, v, reps, sumsq=sumsq)
        torch.maximum(worst, sumsq, out=worst)

    t = 0
    for _ in range(warmup):
        t += 1
        model_step(t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        t += 1
        model_step(t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    for ctx, _ in ctxs:
        L.lossy_device_status(ctx)
        L.lossy_destroy(ctx)
    gbs = total_bytes / (ms * 1e-3) / 1e9
    return {"workload": f"cfg4_cut_{layers}_layers_plus_embedding_and_head", "W": base.W, "P": base.packet_elems,
            "p": base.p, "buckets": len(sizes), "elements": sum(sizes), "resident_GB": round(sum(sizes) * 28 / 1e9, 1),
            "ms_per_step": ms, "GBps": gbs, "frac_of_measured_peak": gbs / _peak(), "steps_per_s": 1e3 / ms,
            "max_drift_norm": float(worst.max().sqrt())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,5")
    ap.add_argument("--steps", type=int, default=0, help="0 = each configuration's own step count")
    ap.add_argument("--elements", type=int, default=0, help="unfused: bucket size override (small case for profiling)")
    args = ap.parse_args()
    cfg = workload.baseline_workloads()
    want = set(args.configs.split(","))
    points = []
    if "1" in want:
        points.append(cfg["cfg1_w4_sgd_f32"])
    if "2" in want:
        points.append(cfg["cfg2_w8_layer_adam"])
    if "3" in want:
        points += [cfg["cfg3_w64_layer_p01"], cfg["cfg3_w64_layer_p10"]]
    if "5" in want:
        for P in (256, 1024, 2048, 4096):
            for p in (0.0, 0.01, 0.05, 0.1, 0.3):
                points.append(workload.scaled(cfg["cfg5_w16_layer_sweep"], workload.LAYER_ELEMS, packet_elems=P, p=p,
                                              name=f"cfg5_w16_P{P}_p{p}"))
    for w in points:
        r = run_point(w, args.steps or w.steps, grad_sets=1 if w.W >= 64 else 2, graph=w.n <= (1 << 22))
        print(json.dumps(r), flush=True)
    if "4" in want:
        # the full model (32 layers) needs 189 GB resident and does not fit one GPU: 24 layers + embedding + head
        print(json.dumps(run_model_streamed(cfg["cfg4_w8_full_model"], 24, args.steps or 20)), flush=True)
    if "unfused" in want:
        base2 = cfg["cfg2_w8_layer_adam"]
        if args.elements:
            base2 = workload.scaled(base2, args.elements)
        for r in run_unfused(base2, steps=args.steps or 20):
            print(json.dumps(r), flush=True)
    if "alg1" in want:
        # Algorithm 1 mode on the config-2 bucket: packet-granular and shard-granular (P = n / W) drops
        base = cfg["cfg2_w8_layer_adam"]
        for P in (2048, workload.LAYER_ELEMS // 8):
            for p in (0.1, 0.3):
                w = workload.scaled(base, base.n, packet_elems=P, p=p, name=f"cfg2_w8_P{P}_p{p}")
                print(json.dumps(run_point(w, args.steps or 30, alg1=True)), flush=True)


if __name__ == "__main__":
    main()
