#!/usr/bin/env python
"""Benchmark of the fused lossy aggregate + step + broadcast (+ drift) pass.

One "step" = one call of lossy_fused_step over one LLaMA-2-7B-decoder-layer-shaped bucket
(W=8 workers, bf16 gradients, fp32 master + Adam, bf16 replicas, packets of 2048 elements,
Bernoulli drop p=0.1) with all state resident in HBM. The metric is algorithmic HBM bytes
moved per second:

    bytes/step = (1-p)*W*n*gb + 24*n + W*n*rb      (delivered gradient packets are read once,
                                                    theta/m/v are read and written, every
                                                    replica packet is either written or read)

Prints ONE JSON line. `--impl reference` times the CPU oracle (as it stands) on a bounded sample.
With --gpus N > 1 (torchrun, one process per GPU) every rank runs its own bucket (weak scaling,
no data-path collective); the W squared drift sums are all-reduced once per timed region.
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

import torch  # noqa: E402

import workload  # noqa: E402

METRIC = "lossy aggregate+step+broadcast HBM GB/s"
WORKLOAD = "cfg2_w8_layer_adam"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the fused kernel, from the ncu capture
# of a small case of the same kernel (Nsight Compute, --set full): 1770.4 MB on a 33,554,432-element cut of the
# workload, scaled by the elements processed (traffic is proportional to them).
NCU_TRAFFIC_SMALL_CASE = (1770.4e6, 33554432)


def algorithmic_bytes(w: workload.Workload, n: int | None = None) -> float:
    n = w.n if n is None else n
    gb = 2 if w.grad_dtype == "bf16" else 4
    rb = 2 if w.replica_dtype == "bf16" else 4
    opt = 24 if w.optimizer == "adam" else 8
    return (1.0 - w.p) * w.W * n * gb + opt * n + w.W * n * rb


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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


def oracle_arm(w, steps, warmup, sample_packets, emit=True):
    """Time the CPU oracle, as it stands, on the first `sample_packets` packets of the workload."""
    from oracle import oracle as O

    dev = "cuda" if torch.cuda.is_available() else "cpu"
    n_slab = min(w.n, sample_packets * w.packet_elems)
    th = workload.theta0_slab(w, 0, n_slab, dev).cpu().numpy()
    orc = O.Oracle(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                   grad_dtype=O.BF16 if w.grad_dtype == "bf16" else O.F32,
                   replica_dtype=O.BF16 if w.replica_dtype == "bf16" else O.F32,
                   optimizer=O.ADAM if w.optimizer == "adam" else O.SGD, theta0=th, lr=w.lr, beta1=w.beta1,
                   beta2=w.beta2, eps=w.eps, k0=0, n_slab=n_slab)
    sets = []
    for s in (1, 2):
        g = gen_grads(w, s, dev, 0, n_slab)
        sets.append([x.cpu().view(torch.int16).numpy().view("uint16") if x.dtype == torch.bfloat16
                     else x.cpu().numpy() for x in g])
    for t in range(1, warmup + 1):
        orc.step(t, sets[t % 2], want_ghat=False)
    t0 = time.perf_counter()
    for t in range(warmup + 1, warmup + steps + 1):
        orc.step(t, sets[t % 2], want_ghat=False)
    dt = time.perf_counter() - t0
    gbs = algorithmic_bytes(w, n_slab) * steps / dt / 1e9
    sample = (f"first {n_slab // w.packet_elems} of {w.K} packets ({n_slab} elements x {w.W} workers), "
              f"{steps} steps, {dt:.1f} s of CPU work")
    return {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
            "ms_per_step": dt / steps * 1e3, "steps_per_s_full_bucket_equiv": steps / dt * n_slab / w.n}


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
    ap.add_argument("--e2e-steps", type=int, default=-1, help="steps of the host-buffer leg (default: min(steps, 10))")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-packets", type=int, default=16384)
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
    # the stored ncu traffic figure belongs to the unmodified default workload on the default kernel
    pristine = (args.workload == WORKLOAD and args.p is None and not args.workers and not args.packet_elems
                and not args.register_path and not args.range)

    if args.impl == "reference":
        if rank != 0:
            return
        r = oracle_arm(w, args.steps, warmup, min(args.cpu_sample_packets, 4096))
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "GB/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name, "W": w.W, "n": w.n, "packet_elems": w.packet_elems, "p": w.p,
                           "optimizer": w.optimizer, "note": "each step is a bounded sample of the bucket"},
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

    full_n, e_off, rng_kw = w.n, 0, {}
    if (args.strong and world > 1) or args.range:
        # strong scaling: the ranks share one bucket, each a contiguous packet range for all W workers
        r_, g_ = (int(x) for x in args.range.split("/")) if args.range else (rank, world)
        pr = L.packet_range_config(w.n, w.packet_elems, r_, g_)
        e_off = pr["e0"]
        rng_kw = {"shard_packet0": pr["shard_packet0"], "bucket_packets": pr["bucket_packets"]}
        w = workload.scaled(w, pr["n"])
    else:
        # weak scaling: every rank simulates its own bucket; global packet ids continue across ranks
        w = workload.scaled(w, w.n, packet_base=rank * w.K, seed=w.seed)
    gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    rdt = torch.bfloat16 if w.replica_dtype == "bf16" else torch.float32
    adam = w.optimizer == "adam"
    ctx = L.lossy_init(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p, p_param=w.p, seed=w.seed,
                       grad_dtype=gdt, replica_dtype=rdt, optimizer=w.optimizer, lr=w.lr, beta1=w.beta1,
                       beta2=w.beta2, eps=w.eps, packet_base=w.packet_base,
                       flags=L.LOSSY_REGISTER_PATH if args.register_path else 0, **rng_kw)
    plan = L.lossy_describe_plan(ctx, True)       # the build the library's launch policy picks for this workload
    master = workload.theta0_slab(w, e_off, e_off + w.n, dev)
    m = torch.zeros_like(master) if adam else None
    v = torch.zeros_like(master) if adam else None
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
    ev[0].record(stream)
    for i in range(args.steps):
        t += 1
        one_step(t)
        ev[i + 1].record(stream)
    if dist is not None:
        dist.all_reduce(sumsq, op=dist.ReduceOp.SUM)        # the only exchange: W doubles per job
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_launch_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    launches = L.lossy_kernel_launches(ctx) - launches0
    clocks = sampler.stop()

    tmax = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    total_ms = float(tmax.item())
    B = algorithmic_bytes(w)                                  # this rank's bytes per step
    strong = args.strong and world > 1
    B_job = algorithmic_bytes(w, full_n) if strong else B * world
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

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = oracle_arm(w, 20, 1, args.cpu_sample_packets)
        cpu = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if strong else "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "steps_per_s": args.steps * (1 if strong else world) / (total_ms * 1e-3),
            "pct_of_hbm_peak": 100.0 * value / world / peak,
            "config": {"workload": w.name, "W": w.W, "n": w.n, "packet_elems": w.packet_elems, "p": w.p,
                       "optimizer": w.optimizer, "grad_dtype": w.grad_dtype, "replica_dtype": w.replica_dtype,
                       "bytes_per_step": B, "parallelism": (f"one bucket in {world} packet ranges, one per GPU" if strong
                                       else f"{world} independent bucket(s), one per GPU"),
                       "l2": "no flush: each step streams %.1f GB of state, far larger than the 126 MB L2; "
                             "two gradient sets alternate" % (B / 1e9),
                       "drift_norm_max_last_step": final_norm_max},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak,
                         "traffic": (NCU_TRAFFIC_SMALL_CASE[0] * w.n / NCU_TRAFFIC_SMALL_CASE[1]
                                     if pristine else None),
                         "peak_source": peak_src + " (MEASURED_PEAKS.json hbm_gbs)" if peak_src == "measured"
                         else peak_src, "kernel": ("lossy_kernel<AGG|STEP|BCAST|DRIFT>" if plan.startswith("register") else "lossy_fused_tma_kernel")
                         + " (drift norms finalised by its last block)", "build": plan,
                         "avg_launch_ms": avg_launch_ms, "min_launch_ms": min(per_launch_ms)},
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    L.lossy_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
