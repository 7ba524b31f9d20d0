"""Owner-elided replicas (LOSSY_REPLICA_SKIP_OWNER) on every kernel build, element by element against the
oracle's elided layout: replica i holds the bucket without the packets worker i owns (Section 3 step (4):
the broadcast goes to all OTHER workers)."""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from paper_2507_07114_b200.sharding import packet_range_config
from parity_util import GpuRun, REL_TOL, assert_rel, assert_same, make_oracle, run_parity, to_np

pytestmark = pytest.mark.gpu
ELIDE, REG, SKIP, LOSSLESS = L.LOSSY_REPLICA_SKIP_OWNER, L.LOSSY_REGISTER_PATH, L.LOSSY_ZERO_SKIP, L.LOSSY_SELF_LOSSLESS
PACKED = L.LOSSY_PACKED_BULK

CASES = [
    # name, W, n, P, p, opt, gd, rd, extra flags, expected start of the plan (None = any)
    ("wide_group4_ragged", 8, 2048 * 37 + 1003, 2048, 0.1, "adam", "bf16", "bf16", 0, "bulk-copy wide group=4"),
    ("wide_group8_early", 16, 2048 * 33, 2048, 0.3, "adam", "bf16", "bf16", 0, "bulk-copy wide group=8 stale=early"),
    ("twin_w64", 64, 4096 * 70 + 40, 4096, 0.1, "adam", "bf16", "bf16", 0, "bulk-copy twin group=8 stale=late"),
    ("twin_split_staged_w64", 64, 1024 * 130 + 8, 1024, 0.3, "adam", "bf16", "bf16", 0, "bulk-copy twin group=8 stale=staged split"),
    ("twin_split_early_w24", 24, 1024 * 75, 1024, 0.2, "sgd", "f32", "f32", 0, "bulk-copy twin group=8 stale=early split"),
    ("gather_wide_256", 16, 256 * 61 + 40, 256, 0.1, "adam", "bf16", "bf16", 0, "gather wide packets/tile=8"),
    ("gather_twin_128_w40", 40, 128 * 90 + 8, 128, 0.1, "sgd", "bf16", "bf16", 0, "gather twin packets/tile=8"),
    ("gather_twin_512_w3_f32", 3, 512 * 21, 512, 0.4, "adam", "f32", "f32", SKIP, "gather twin packets/tile=2"),
    ("gather_shards_inside_a_tile", 8, 256 * 10, 256, 0.3, "adam", "bf16", "bf16", 0, "gather wide"),      # pps = 2: four owners per tile
    ("gather_twin_w2_mixed", 2, 256 * 33 + 24, 256, 0.3, "adam", "bf16", "f32", 0, "gather twin packets/tile=4"),
    ("packed_wide_256", 16, 256 * 61 + 40, 256, 0.1, "adam", "bf16", "bf16", PACKED, "bulk-copy wide group=8 stale=late packed"),
    ("packed_twin_128_w40", 40, 128 * 90 + 8, 128, 0.3, "sgd", "bf16", "bf16", PACKED, "bulk-copy twin group=8 stale=late packed"),
    ("packed_512_w3_f32", 3, 512 * 21, 512, 0.4, "adam", "f32", "f32", SKIP | PACKED, None),
    ("packed_shards_inside_a_tile", 8, 256 * 10, 256, 0.3, "adam", "bf16", "bf16", PACKED, None),
    ("register_path", 8, 2048 * 9 + 5, 2048, 0.3, "adam", "bf16", "bf16", REG, "register kernel"),
    ("register_small_packets_w17", 17, 264 * 50, 264, 0.2, "adam", "bf16", "f32", 0, "register kernel"),
    ("fewer_packets_than_workers", 8, 3 * 512 - 100, 512, 0.2, "adam", "f32", "bf16", 0, None),
    ("one_worker_holds_nothing", 1, 5000, 256, 0.3, "adam", "bf16", "bf16", 0, None),
    ("single_short_packet", 4, 5, 1024, 0.3, "sgd", "bf16", "bf16", 0, None),
    ("self_lossless_zero_skip", 5, 1032 * 33 + 16, 1032, 0.45, "adam", "f32", "bf16", LOSSLESS | SKIP, None),
    ("w63_tiny_packets", 63, 8 * 700 + 3, 8, 0.2, "sgd", "f32", "f32", 0, None),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("fused", [True, False])
def test_elided_replicas_match_the_oracle(case, fused):
    name, W, n, P, p, opt, gd, rd, flags, plan = case
    w = workload.Workload(name, W, n, P, p, opt, 1e-2 if opt == "sgd" else 3e-4, gd, rd, 5, seed=21)
    gpu, orc = run_parity(w, 5, fused=fused, flags=flags | ELIDE)
    if plan is not None:
        assert L.lossy_describe_plan(gpu.ctx).startswith(plan), L.lossy_describe_plan(gpu.ctx)
    if W > 1 and n > 1000:
        assert float(gpu.norms.max()) > 0.0
    # the standalone drift entry points read the same layout
    want = orc.drift_sumsq()
    got = torch.zeros(W, dtype=torch.float64, device="cuda")
    L.drift_norms(gpu.ctx, gpu.master, gpu.replicas, None, got)
    assert_rel(got.cpu().numpy(), want, f"{name} drift_norms", tol=2 * REL_TOL)
    got.zero_()
    L.drift_norms_static(W=W, n=n, packet_elems=P, replica_dtype=gpu.replicas[0].dtype, master=gpu.master,
                         replicas=gpu.replicas, sumsq=got, flags=ELIDE)
    assert_rel(got.cpu().numpy(), want, f"{name} drift_norms_static", tol=2 * REL_TOL)
    d2 = torch.zeros(W * W, dtype=torch.float64, device="cuda")
    L.drift_pairwise(gpu.ctx, gpu.replicas, d2)
    off = ~np.eye(W, dtype=bool)        # fp32 squares of eight elements at a time, then fp64: the same bound as the norms
    assert_rel(d2.cpu().numpy().reshape(W, W)[off], orc.pairwise_sumsq()[off], f"{name} pairwise", tol=2 * REL_TOL)


def test_elided_equals_the_full_layout_on_everything_a_worker_does_not_own():
    """Same run with and without the flag: identical masks, parameters and norms; each elided replica is the full
    one with the owner's range cut out."""
    w = workload.scaled(workload.baseline_workloads()["cfg2_w8_layer_adam"], 2048 * 300 + 24)
    a, b = GpuRun(w), GpuRun(w, flags=ELIDE)
    K, W, P = w.K, w.W, w.packet_elems
    pps = (K + W - 1) // W
    for t in range(1, 5):
        gd = [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(W)]
        a.step_fused(t, gd)
        b.step_fused(t, gd)
        torch.cuda.synchronize()
        assert torch.equal(a.master, b.master) and torch.equal(a.m, b.m) and torch.equal(a.v, b.v)
        assert torch.equal(a.recv, b.recv) and torch.equal(a.stale, b.stale) and torch.equal(a.count, b.count)
        assert torch.equal(a.norms, b.norms) and torch.equal(a.sumsq, b.sumsq)
        for i in range(W):
            lo, hi = min(w.n, i * pps * P), min(w.n, (i + 1) * pps * P)
            assert torch.equal(b.replicas[i], torch.cat([a.replicas[i][:lo], a.replicas[i][hi:]]))


BAND, POISON = 4096, 0x5A


@pytest.mark.parametrize("W,n,P,p,flags", [(8, 2048 * 19 + 1003, 2048, 0.2, 0), (16, 256 * 45 + 40, 256, 0.1, 0),
                                           (16, 256 * 45 + 40, 256, 0.1, PACKED), (3, 128 * 77 + 8, 128, 0.3, 0),
                                           (64, 1024 * 70 + 16, 1024, 0.3, 0), (8, 2048 * 7 + 5, 2048, 0.3, REG)])
def test_elided_replicas_between_guard_bands(W, n, P, p, flags):
    """Every replica is exactly lossy_replica_elems long and sits between two poisoned bands: the owner's range
    does not exist, so a kernel that addressed it would write into a band (or into the neighbour)."""
    w = workload.Workload("guard_elided", W, n, P, p, "adam", 3e-4, "bf16", "bf16", 3, seed=8)
    ctx = L.lossy_init(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=8, grad_dtype=torch.bfloat16,
                       replica_dtype=torch.bfloat16, optimizer="adam", lr=3e-4, flags=flags | ELIDE)
    th = workload.theta0_slab(w, 0, n, "cuda")
    master, m, v = th.clone(), torch.zeros_like(th), torch.zeros_like(th)
    raws, reps = [], []
    for i in range(W):
        ne = L.lossy_replica_elems(ctx, i)
        raw = torch.full((2 * BAND + 2 * ne,), POISON, dtype=torch.uint8, device="cuda")
        raws.append((raw, 2 * ne))
        reps.append(raw[BAND:BAND + 2 * ne].view(torch.bfloat16))
        reps[-1].zero_()
    norms = torch.zeros(W, device="cuda")
    stale = torch.zeros(w.K, dtype=torch.int64, device="cuda")
    for t in range(1, 4):
        gd = [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)]
        L.lossy_fused_step(ctx, t, gd, master, m, v, reps, norms=norms)
        L.lossy_broadcast(ctx, t, master, reps, stale)
        L.drift_norms(ctx, master, reps, norms)
        L.lossy_device_status(ctx)
        for i, (raw, nb) in enumerate(raws):
            assert bool((raw[:BAND] == POISON).all()) and bool((raw[BAND + nb:] == POISON).all()), f"replica {i} step {t}"
    L.lossy_destroy(ctx)


@pytest.mark.parametrize("W,n,P,world", [(8, 2048 * 37 + 1003, 2048, 3), (5, 1024 * 11, 1024, 4), (16, 256 * 50 + 8, 256, 2)])
def test_elided_packet_ranges_reproduce_the_whole_bucket(W, n, P, world):
    """Packet-range sharding with owner-elided replicas: a range may hold all, part or none of worker i's shard,
    and replica i of that range leaves out exactly that part."""
    w = workload.Workload("ranges_elided", W, n, P, 0.25, "adam", 3e-4, "bf16", "bf16", 4, seed=17)
    whole = GpuRun(w)                                       # full layout, the reference for every range
    K = w.K
    pps = (K + W - 1) // W
    parts = []
    for r in range(world):
        cfg = packet_range_config(n, P, r, world)
        sub = workload.scaled(w, cfg["n"])
        run = GpuRun(sub, flags=ELIDE, theta0=workload.theta0_slab(w, cfg["e0"], cfg["e0"] + cfg["n"]),
                     shard_packet0=cfg["shard_packet0"], bucket_packets=cfg["bucket_packets"])
        orc = make_oracle(w, flags=ELIDE, k0=cfg["shard_packet0"], n_slab=cfg["n"], e0=cfg["e0"])
        parts.append((cfg, run, orc))
    for t in range(1, 5):
        gd = [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)]
        whole.step_fused(t, gd)
        tot = torch.zeros(W, dtype=torch.float64, device="cuda")
        for cfg, run, orc in parts:
            e0, e1 = cfg["e0"], cfg["e0"] + cfg["n"]
            run.step_fused(t, [g[e0:e1] for g in gd])
            tot += run.sumsq
            orc.step(t, [to_np(g[e0:e1]) for g in gd])
            torch.cuda.synchronize()
            assert torch.equal(run.master, whole.master[e0:e1])
            owner = (torch.arange(e0, e1, device="cuda") // P) // pps
            for i in range(W):
                assert torch.equal(run.replicas[i], whole.replicas[i][e0:e1][owner != i]), f"range {cfg['shard_packet0']} replica {i}"
                assert_same(to_np(run.replicas[i]), orc.replicas[i], f"range {cfg['shard_packet0']} replica {i} vs oracle")
        torch.cuda.synchronize()
        assert_rel(tot.cpu().numpy(), whole.sumsq.cpu().numpy(), f"step {t} summed drift", tol=1e-6)


def test_replica_elems_and_rejections():
    kw = dict(W=4, n=1024 * 10 + 8, packet_elems=1024, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
              replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
    ctx = L.lossy_init(**kw)
    assert [L.lossy_replica_elems(ctx, i) for i in range(5)] == [kw["n"]] * 4 + [0]
    L.lossy_destroy(ctx)
    ctx = L.lossy_init(flags=ELIDE, **kw)           # K = 11, shards of 3 packets, the last one 2 (one of them short)
    assert [L.lossy_replica_elems(ctx, i) for i in range(4)] == [kw["n"] - 3072] * 3 + [kw["n"] - 1024 - 8]
    z = [torch.zeros(kw["n"], device="cuda") for _ in range(4)]
    with pytest.raises(L.LossyError) as ei:         # the closed-loop gradient stand-in needs full replicas
        L.lossy_closed_loop_grads(ctx, z[0], z[0], z, z, z)
    assert ei.value.code == L.LOSSY_EINVAL
    L.lossy_destroy(ctx)
