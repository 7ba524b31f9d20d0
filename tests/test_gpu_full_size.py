"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run a whole 202-million-element bucket in seconds, but packets evolve
independently: the GPU runs the full bucket, and the oracle re-runs sampled slabs of packets
(first, last, shard boundaries, random) from regenerated inputs, element by element. The
drift norms are checked on EVERY element: the oracle's drift routine reads the full GPU
state copied to the host.
"""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import (GpuRun, assert_rel, assert_same, compare_state, make_oracle, to_np)

pytestmark = pytest.mark.gpu
CFG = workload.baseline_workloads()


def _slabs(w, rng, n_random, width):
    K = w.K
    pps = (K + w.W - 1) // w.W
    starts = {0, max(0, K - width), max(0, pps - width // 2), max(0, min(K - width, (w.W - 1) * pps - 1))}
    starts |= {int(x) for x in rng.integers(0, max(1, K - width), n_random)}
    return sorted(starts)


def _run_full(w, steps, slab_packets, n_random, full_drift, flags=0):
    gpu = GpuRun(w, flags=flags)
    rng = np.random.default_rng(0)
    slabs = _slabs(w, rng, n_random, slab_packets)
    P = w.packet_elems
    oracles = []
    for k0 in slabs:
        e0, e1 = k0 * P, min(w.n, (k0 + slab_packets) * P)
        oracles.append((k0, e0, e1, make_oracle(w, k0=k0, n_slab=e1 - e0, e0=e0)))
    for t in range(1, steps + 1):
        gd = [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)]
        gpu.step_fused(t, gd)                       # the call bench.py times (with every optional output)
        out = gpu.outputs()
        # masks, received counts and stale sets of EVERY packet of the bucket, bit for bit
        recv_all, stale_all, count_all = oracles[0][3].masks(t, 0, w.K)
        assert_same(out["recv_bits"], recv_all, f"{w.name} step {t} recv_bits of all {w.K} packets")
        assert_same(out["stale_bits"], stale_all, f"{w.name} step {t} stale_bits of all {w.K} packets")
        assert_same(out["count"], count_all, f"{w.name} step {t} counts of all {w.K} packets")
        for k0, e0, e1, orc in oracles:
            ref = orc.step(t, [to_np(g[e0:e1]) for g in gd])
            k1 = k0 + orc.packets
            what = f"{w.name} step {t} packets [{k0},{k1})"
            assert_same(out["count"][k0:k1], ref["count"], what + " count")
            assert_same(out["recv_bits"][k0:k1], ref["recv_bits"], what + " recv_bits")
            assert_same(out["stale_bits"][k0:k1], ref["stale_bits"], what + " stale_bits")
            assert_rel(out["ghat"][e0:e1], ref["ghat"], what + " ghat")
            compare_state(gpu, orc, what, e0, e1)
        del gd
    L.lossy_device_status(gpu.ctx)
    if full_drift:
        # every element: oracle drift routine on the full GPU state
        # (a small oracle object is re-pointed at the full arrays; its drift routine only needs
        # the replica dtype, W and the element count)
        drift_orc = make_oracle(workload.scaled(w, 8 * w.W, packet_elems=8), theta0=torch.zeros(8 * w.W))
        drift_orc.n_slab = w.n
        drift_orc.master = to_np(gpu.master)
        drift_orc.replicas = [to_np(r) for r in gpu.replicas]
        want = np.sqrt(drift_orc.drift_sumsq())
        assert_rel(out["norms"], want, f"{w.name} drift norms over all elements")
        assert float(want.max()) > 0.0
    # conservation over the whole bucket: counts are the popcounts of the receive bits
    pop = np.array([bin(int(b)).count("1") for b in out["recv_bits"][:5000]])
    assert_same(out["count"][:5000], pop.astype(np.uint8), "count vs popcount")
    return gpu


def test_config2_full_layer_bucket():
    w = CFG["cfg2_w8_layer_adam"]
    _run_full(w, steps=3, slab_packets=6, n_random=6, full_drift=True)


def test_config2_full_layer_unfused_calls_match_the_fused_step():
    """The four single-phase calls at full size, each on its own bulk-copy pipeline: the same masks,
    parameters, moments, replicas and estimate as the fused step (itself checked against the oracle
    above), bit for bit; drift norms to rounding (another summation order)."""
    w = CFG["cfg2_w8_layer_adam"]
    a, b = GpuRun(w), GpuRun(w)
    for t in (1, 2):
        gd = [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)]
        a.step_fused(t, gd)
        b.step_unfused(t, gd)
        oa, ob = a.outputs(), b.outputs()
        for key in ("count", "recv_bits", "stale_bits"):
            assert_same(ob[key], oa[key], f"step {t} {key}")
        assert torch.equal(a.ghat, b.ghat) and torch.equal(a.master, b.master)
        assert torch.equal(a.m, b.m) and torch.equal(a.v, b.v)
        for i in range(w.W):
            assert torch.equal(a.replicas[i], b.replicas[i]), f"step {t} replica {i}"
        assert_rel(ob["norms"], oa["norms"], f"step {t} norms", tol=2e-6)
        del gd
    L.lossy_device_status(a.ctx)
    L.lossy_device_status(b.ctx)


def test_config3_full_w64_sampled():
    w = CFG["cfg3_w64_layer_p10"]
    _run_full(w, steps=2, slab_packets=3, n_random=3, full_drift=False)


def test_w64_high_loss_full_size_split_build_with_staged_stale_copies():
    # W = 64 at p = 0.3: state slots apart from the stages, stale replicas' old copies as pipeline stages
    w = workload.scaled(CFG["cfg3_w64_layer_p10"], workload.LAYER_ELEMS, p=0.3)
    gpu = _run_full(w, steps=2, slab_packets=3, n_random=3, full_drift=False)
    assert L.lossy_describe_plan(gpu.ctx) == "bulk-copy twin group=8 stale=staged split stages=4"


def test_config5_point_full_size_small_packets_register_path():
    # the register-path kernel at full size (what P = 256 ran on at high loss before the drift-warp build; still the
    # kernel of many workers at high loss)
    w = workload.scaled(CFG["cfg5_w16_layer_sweep"], workload.LAYER_ELEMS, packet_elems=256, p=0.3)
    gpu = _run_full(w, steps=2, slab_packets=24, n_random=4, full_drift=False, flags=L.LOSSY_REGISTER_PATH)
    assert L.lossy_describe_plan(gpu.ctx) == "register kernel"


def test_config5_point_full_size_small_packets_high_loss_drift_warps():
    # P = 256, p = 0.3: the wide gather build whose drift warps read the stale copies
    w = workload.scaled(CFG["cfg5_w16_layer_sweep"], workload.LAYER_ELEMS, packet_elems=256, p=0.3)
    gpu = _run_full(w, steps=2, slab_packets=24, n_random=4, full_drift=True)
    assert L.lossy_describe_plan(gpu.ctx) == "gather wide packets/tile=8 stages=3 drift-warps"


def test_config5_point_full_size_small_packets_gather_pipeline():
    # P=256 at low and moderate loss takes the gather pipeline (eight whole packets per tile) at full size
    w = workload.scaled(CFG["cfg5_w16_layer_sweep"], workload.LAYER_ELEMS, packet_elems=256, p=0.1)
    gpu = _run_full(w, steps=2, slab_packets=24, n_random=4, full_drift=True)
    assert L.lossy_describe_plan(gpu.ctx) == "gather wide packets/tile=8 stages=3"


def test_few_workers_small_packets_full_size_gather_twin():
    # W = 3, P = 256 at high loss: the twin gather build whose replica warps also read the stale copies
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], workload.LAYER_ELEMS, W=3, packet_elems=256, p=0.3)
    gpu = _run_full(w, steps=2, slab_packets=24, n_random=4, full_drift=True)
    assert L.lossy_describe_plan(gpu.ctx) == "gather twin packets/tile=4 stages=4"


def test_drift_is_order_one_and_matches_the_stationary_constant_at_scale():
    """Bounded Model Drift at scale, as a property that holds at any size: with SGD and gradients
    redrawn i.i.d. every step, a replica's squared distance from the owners' values settles at
    (elements it does not own) * p/(1-p) * sigma^2, sigma^2 = lr^2 sigma_g^2 E[1/c; c>0] — the
    replica-vs-owner form of the theorem's constant — and does not grow with t."""
    from math import comb

    W, p, lr, sg = 8, 0.3, 1e-2, 1e-3
    n = 2048 * 24000
    w = workload.Workload("drift_at_scale", W, n, 2048, p, "sgd", lr, "bf16", "f32", 60, grad_sigma=sg, seed=4)
    gpu = GpuRun(w)
    hist = []
    for t in range(1, 61):
        gd = [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)]
        gpu.step_fused(t, gd, outputs=False)
        hist.append(gpu.norms.double().cpu().numpy() ** 2)
        del gd
    L.lossy_device_status(gpu.ctx)
    inv_c = sum(comb(W, c) * (1 - p) ** c * p ** (W - c) / c for c in range(1, W + 1))
    sigma2 = (lr * sg) ** 2 * inv_c
    K = w.K
    pps = (K + W - 1) // W
    own = np.array([min(K, (i + 1) * pps) - min(K, i * pps) for i in range(W)]) * 2048
    want = (n - own) * p / (1 - p) * sigma2
    late = np.mean(hist[30:], axis=0)
    assert np.all(np.abs(late / want - 1) < 0.03), (late / want)
    first, second = np.mean(hist[20:40], axis=0), np.mean(hist[40:], axis=0)
    assert np.all(np.abs(second / first - 1) < 0.03)                 # O(1): no growth with t
    paper = (n - own) * 2 * p / (1 + p) * sigma2                     # the printed pairwise constant, for scale
    assert np.all(late < 2.0 * paper)
