"""The method in closed loop on a synthetic objective: the paper's Table 1 trend in miniature.

    python -m paper_2507_07114_b200.closed_loop [--elements N] [--steps T] [--workers W]

Every step, worker i evaluates the gradient of 1/2 sum a (theta - x*)^2 at ITS OWN replica (stale
where broadcasts were lost) plus fresh noise (lossy_closed_loop_grads), then the fused lossy step
aggregates, updates and broadcasts. For each drop rate the module prints the objective at the
owners' parameters averaged over the last quarter of the run, its change against the lossless run,
the largest drift norm, and the same for the objective seen by the replicas.
"""
from __future__ import annotations

import argparse
import json

import torch

import workload
from . import binding as L


def run(p, *, W, n, P, steps, optimizer, lr, gdt, rdt, seed=0, sigma_noise=1.0):
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--elements", type=int, default=2048 * 4096)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--workers", type=int, default=8)
    ap.add_argument("--packet-elems", type=int, default=2048)
    args = ap.parse_args()
    for name, opt, lr, gdt, rdt in (("sgd_fp32", "sgd", 0.1, torch.float32, torch.float32),
                                    ("adam_bf16", "adam", 3e-3, torch.bfloat16, torch.bfloat16)):
        base = None
        for p in (0.0, 0.1, 0.2, 0.3, 0.4):
            owner, rep, drift = run(p, W=args.workers, n=args.elements, P=args.packet_elems, steps=args.steps,
                                    optimizer=opt, lr=lr, gdt=gdt, rdt=rdt)
            base = base or (owner, rep)
            print(json.dumps({"run": name, "p": p, "objective_owner": owner,
                              "change_vs_lossless_pct": 100 * (owner / base[0] - 1), "objective_replicas": rep,
                              "replica_change_pct": 100 * (rep / base[1] - 1), "max_drift_norm": drift}), flush=True)


if __name__ == "__main__":
    main()
