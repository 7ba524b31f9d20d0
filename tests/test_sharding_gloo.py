"""The N>1 path on CPU: ranks take contiguous bucket ranges, run independently (no data-path
collective) and only the per-replica squared drift sums are all-reduced. world_size 2, gloo."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workload
from paper_2507_07114_b200.sharding import packet_range_config, shard_range
from parity_util import make_oracle, to_np


def test_shard_range_partitions_exactly():
    for units in (0, 1, 7, 8, 34):
        for world in (1, 2, 3, 8):
            got = [shard_range(units, r, world) for r in range(world)]
            assert got[0][0] == 0 and got[-1][1] == units
            assert all(a[1] == b[0] for a, b in zip(got[:-1], got[1:]))
            sizes = [b - a for a, b in got]
            assert max(sizes) - min(sizes) <= 1


def test_packet_ranges_tile_the_bucket():
    for n, P in ((2048 * 37 + 1003, 2048), (1024 * 11, 1024), (100, 256)):
        K = (n + P - 1) // P
        for world in (1, 2, 3, 8):
            cfgs = [packet_range_config(n, P, r, world) for r in range(world)]
            assert cfgs[0]["e0"] == 0 and sum(c["n"] for c in cfgs) == n
            for a, b in zip(cfgs[:-1], cfgs[1:]):
                assert a["e0"] + a["n"] == b["e0"]
                assert a["n"] % P == 0 or b["n"] == 0            # only the last non-empty range may be ragged
                assert b["shard_packet0"] * P == b["e0"] or b["n"] == 0
            assert all(c["bucket_packets"] == K for c in cfgs)


BUCKETS = [512 * 9, 512 * 7 + 40, 512 * 12, 512 * 5, 512 * 3 + 8]


def _bucket_workloads():
    base = workload.baseline_workloads()["cfg4_w8_full_model"]
    out, pb = [], 0
    for b, n in enumerate(BUCKETS):
        w = workload.scaled(base, n, packet_elems=512, packet_base=pb, name=f"bucket{b}")
        out.append(w)
        pb += w.K
    return out


def _run_buckets(ws, steps):
    tot = np.zeros(8)
    for w in ws:
        o = make_oracle(w)
        for t in range(1, steps + 1):
            r = o.step(t, [to_np(workload.grad_slab(w, t, i, 0, w.n)) for i in range(w.W)])
        tot += r["sumsq"]
    return tot


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ws = _bucket_workloads()
    lo, hi = shard_range(len(ws), rank, world)
    mine = torch.from_numpy(_run_buckets(ws[lo:hi], 3))
    dist.all_reduce(mine, op=dist.ReduceOp.SUM)          # the only exchange: W doubles
    t = torch.tensor([1.0 + rank])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)              # bench timing rule: max over ranks
    if rank == 0:
        q.put((mine.numpy(), float(t)))
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_drift():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got, tmax = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = _run_buckets(_bucket_workloads(), 3)
    assert np.allclose(got, want, rtol=1e-12)
    assert tmax == 2.0


def _range_worker(rank, world, port, q):
    """One bucket in `world` packet ranges with owner-elided replicas: a range holds all, part or none of a
    worker's shard, and replica i of that range leaves out exactly that part."""
    from oracle import oracle as O

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workload.Workload("range_bucket", 5, 512 * 23 + 40, 512, 0.3, "adam", 3e-4, "bf16", "bf16", 3, seed=9)
    cfg = packet_range_config(w.n, w.packet_elems, rank, world)
    e0, e1 = cfg["e0"], cfg["e0"] + cfg["n"]
    o = make_oracle(w, flags=O.REPLICA_SKIP_OWNER, k0=cfg["shard_packet0"], n_slab=cfg["n"], e0=e0)
    for t in range(1, 4):
        r = o.step(t, [to_np(workload.grad_slab(w, t, i, e0, e1)) for i in range(w.W)])
    mine = torch.from_numpy(r["sumsq"].copy())
    dist.all_reduce(mine, op=dist.ReduceOp.SUM)
    kept = torch.tensor([float(sum(x.size for x in o.replicas))])
    dist.all_reduce(kept, op=dist.ReduceOp.SUM)
    if rank == 0:
        q.put((mine.numpy(), float(kept)))
    dist.destroy_process_group()


def test_two_ranks_of_packet_ranges_with_owner_elided_replicas():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_range_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got, kept = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = workload.Workload("range_bucket", 5, 512 * 23 + 40, 512, 0.3, "adam", 3e-4, "bf16", "bf16", 3, seed=9)
    o = make_oracle(w)                                   # the whole bucket, full replicas
    for t in range(1, 4):
        r = o.step(t, [to_np(workload.grad_slab(w, t, i, 0, w.n)) for i in range(w.W)])
    assert np.allclose(got, r["sumsq"], rtol=1e-12) and got.max() > 0
    assert kept == (w.W - 1) * w.n                       # every element is stored W - 1 times over the ranks
