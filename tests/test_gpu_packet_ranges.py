"""One bucket simulated as several packet ranges (the multi-GPU partition, run here on one GPU one range
after the other): bit-identical to the single-context run, and to the oracle's slabs."""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from paper_2507_07114_b200.sharding import packet_range_config
from parity_util import GpuRun, assert_rel, assert_same, make_oracle, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("W,n,P,world", [(8, 2048 * 37 + 1003, 2048, 3), (5, 1024 * 11, 1024, 4), (16, 256 * 50 + 8, 256, 2)])
def test_packet_ranges_reproduce_the_whole_bucket(W, n, P, world, monkeypatch):
    w = workload.Workload("ranges", W, n, P, 0.25, "adam", 3e-4, "bf16", "bf16", 5, seed=17)
    whole = GpuRun(w)
    parts = []
    orig_init = L.lossy_init
    for r in range(world):
        cfg = packet_range_config(n, P, r, world)

        def init_with_range(**kw):
            kw.update(shard_packet0=cfg["shard_packet0"], bucket_packets=cfg["bucket_packets"])
            return orig_init(**kw)

        monkeypatch.setattr(L, "lossy_init", init_with_range)
        sub = workload.scaled(w, cfg["n"])
        parts.append((cfg, GpuRun(sub, theta0=workload.theta0_slab(w, cfg["e0"], cfg["e0"] + cfg["n"]))))
    monkeypatch.setattr(L, "lossy_init", orig_init)
    orcs = [make_oracle(w, k0=cfg["shard_packet0"], n_slab=cfg["n"], e0=cfg["e0"]) for cfg, _ in parts]
    for t in range(1, 6):
        gd = [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)]
        whole.step_fused(t, gd)
        tot = torch.zeros(W, dtype=torch.float64, device="cuda")
        for (cfg, run), orc in zip(parts, orcs):
            e0, e1 = cfg["e0"], cfg["e0"] + cfg["n"]
            run.step_fused(t, [g[e0:e1] for g in gd])
            tot += run.sumsq
            ref = orc.step(t, [to_np(g[e0:e1]) for g in gd])
            k0 = cfg["shard_packet0"]
            torch.cuda.synchronize()
            assert torch.equal(run.master, whole.master[e0:e1]) and torch.equal(run.v, whole.v[e0:e1])
            for i in range(W):
                assert torch.equal(run.replicas[i], whole.replicas[i][e0:e1])
            assert torch.equal(run.recv, whole.recv[k0:k0 + run.w.K]) and torch.equal(run.stale, whole.stale[k0:k0 + run.w.K])
            assert torch.equal(run.count, whole.count[k0:k0 + run.w.K])
            assert_same(to_np(run.master), orc.master, f"range {k0} step {t} master vs oracle slab")
            assert_same(to_np(run.recv).view(np.uint64), ref["recv_bits"], f"range {k0} step {t} recv bits")
        torch.cuda.synchronize()
        # the one exchange of the multi-GPU path: the squared drift sums add up
        assert_rel(tot.cpu().numpy(), whole.sumsq.cpu().numpy(), f"step {t} summed drift", tol=1e-6)


def test_bad_ranges_are_rejected():
    kw = dict(W=4, n=1024 * 4, packet_elems=1024, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
              replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
    for bad in (dict(shard_packet0=3, bucket_packets=6), dict(shard_packet0=1, bucket_packets=0),
                dict(n=1024 * 4 - 8, shard_packet0=0, bucket_packets=9)):
        k = dict(kw)
        k.update(bad)
        with pytest.raises(L.LossyError):
            L.lossy_init(**k)
    ctx = L.lossy_init(**dict(kw, shard_packet0=2, bucket_packets=6))
    L.lossy_destroy(ctx)
