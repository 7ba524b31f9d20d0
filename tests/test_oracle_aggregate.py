"""Pins for the oracle's unbiased aggregation (Section 3 step (2); "Unbiased Gradient
Aggregation" and its Corollary). CPU only."""
import itertools

import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import ADAM, BF16, F32, SGD, Oracle

f32 = np.float32


def _mk(W, n, P, p, *, seed=0, gd=F32, rd=F32, opt=SGD, lr=1e-2, flags=0, theta=None, f64=False, **kw):
    theta = np.zeros(n, f32) if theta is None else theta
    return Oracle(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=gd, replica_dtype=rd,
                  optimizer=opt, theta0=theta, lr=lr, flags=flags, f64=f64, **kw)


def _rand_grads(rng, W, n, sigma=1e-3):
    return [(rng.standard_normal(n) * sigma).astype(f32) for _ in range(W)]


def test_p_zero_is_the_plain_mean_bit_exact():
    """With every indicator 1 the estimator is the ordinary mean (Section 3 step (2))."""
    rng = np.random.default_rng(0)
    for W, n, P in ((1, 40, 8), (3, 1000, 64), (8, 5000, 256), (64, 700, 16)):
        theta = (rng.standard_normal(n) * 0.02).astype(f32)
        o = _mk(W, n, P, 0.0, theta=theta)
        g = _rand_grads(rng, W, n)
        r = o.step(1, g)
        acc = np.zeros(n, f32)
        for i in range(W):                       # (((g0+g1)+g2)+...) in fp32
            acc = (acc + g[i]).astype(f32)
        plain = (acc / f32(W)).astype(f32)
        assert np.array_equal(r["ghat"], plain)
        dmean = np.mean(np.stack(g).astype(np.float64), axis=0)
        assert np.max(np.abs(r["ghat"] - dmean)) <= 1e-6 * np.max(np.abs(dmean))
        assert np.all(r["count"] == W)
        assert np.all(r["recv_bits"] == np.uint64((1 << W) - 1))
        assert np.all(r["stale_bits"] == 0)
        assert np.all(r["sumsq"] == 0.0)
        for rep in o.replicas:                   # lossless broadcast: every copy is the owner's value
            assert np.array_equal(rep, o.master)
        assert np.array_equal(o.master, (theta - (f32(1e-2) * plain).astype(f32)).astype(f32))


def test_worker_order_is_ascending_in_fp32():
    g = [np.full(8, v, f32) for v in (1e8, 1.0, -1e8)]
    o = _mk(3, 8, 8, 0.0)
    r = o.step(1, g)
    assert np.all(r["ghat"] == f32((f32(1e8) + f32(1.0)) + f32(-1e8)) / f32(3))   # = 0, not 1/3


@pytest.mark.parametrize("W,K", [(1, 1), (2, 2), (3, 2), (4, 2), (4, 1)])
def test_all_delivery_patterns_enumerated(W, K):
    """Every one of the 2^(W*K) receive patterns gives masked-sum / count, zero when nothing arrived,
    and the pattern-weighted average is (1 - p^W) * mean (unbiased given that something arrived)."""
    rng = np.random.default_rng(W * 10 + K)
    P, p = 8, 0.3
    n = K * P
    g = _rand_grads(rng, W, n, 1.0)
    G = np.stack(g).astype(np.float64)
    mean = G.mean(axis=0)
    expect = np.zeros(n)
    for pattern in itertools.product(range(1 << W), repeat=K):
        o = _mk(W, n, P, p, f64=True)
        r = o.step(1, g, recv_force=np.array(pattern, np.uint64))
        prob = 1.0
        for k, bits in enumerate(pattern):
            sel = [i for i in range(W) if (bits >> i) & 1]
            prob *= (1 - p) ** len(sel) * p ** (W - len(sel))
            want = G[sel, k * P:(k + 1) * P].sum(axis=0) / len(sel) if sel else np.zeros(P)
            assert np.allclose(r["ghat"][k * P:(k + 1) * P], want, rtol=1e-13, atol=0)
            assert r["count"][k] == len(sel)
        expect += prob * r["ghat"]
    assert np.allclose(expect, (1 - p ** W) * mean, rtol=1e-12, atol=1e-15)


def test_unbiased_over_seeds_with_hashed_masks():
    """Corollary: E[ghat | something arrived] equals the lossless mean, for FIXED heterogeneous
    worker gradients; unconditioned it is (1 - p^W) times that (zero fallback)."""
    W, P, K, p = 4, 8, 4, 0.3
    n = P * K
    rng = np.random.default_rng(5)
    shared = rng.standard_normal(n)
    g = [(shared + 0.5 * rng.standard_normal(n)).astype(f32) for _ in range(W)]
    mean = np.stack(g).astype(np.float64).mean(axis=0)
    seeds = 6000
    tot = np.zeros(n)
    tot2 = np.zeros(n)
    cond = np.zeros(n)
    cond_n = np.zeros(n)
    for s in range(seeds):
        o = _mk(W, n, P, p, seed=s, f64=True)
        r = o.step(1, g)
        gh = r["ghat"]
        tot += gh
        tot2 += gh * gh
        got = np.repeat(r["count"] > 0, P)
        cond += np.where(got, gh, 0.0)
        cond_n += got
    se = np.sqrt((tot2 / seeds - (tot / seeds) ** 2) / seeds) + 1e-12
    assert np.all(np.abs(cond / cond_n - mean) < 4.5 * se * np.sqrt(seeds / cond_n))
    assert np.all(np.abs(tot / seeds - (1 - p ** W) * mean) < 4.5 * se)
    # and the received fraction itself
    assert abs(cond_n.mean() / seeds - (1 - p ** W)) < 4 * np.sqrt(p ** W / (seeds * K))


def test_nothing_received_fallback_and_zero_skip():
    W, P = 3, 8
    n = 2 * P
    rng = np.random.default_rng(1)
    theta = rng.standard_normal(n).astype(f32)
    g = _rand_grads(rng, W, n, 1.0)
    force = np.array([0, 0b101], np.uint64)          # packet 0 receives nothing
    for opt in (SGD, ADAM):
        o = _mk(W, n, P, 0.5, opt=opt, theta=theta)
        o.step(1, g, recv_force=np.array([0b111, 0b111], np.uint64))
        th1, m1, v1 = o.master.copy(), o.m.copy(), o.v.copy()
        r = o.step(2, g, recv_force=force)
        assert np.all(r["ghat"][:P] == 0) and r["count"][0] == 0
        if opt == SGD:
            assert np.array_equal(o.master[:P], th1[:P])          # theta - lr*0
        else:
            # the unmodified optimizer still runs on ghat = 0: moments decay, theta moves
            assert np.array_equal(o.m[:P], (f32(0.9) * m1[:P]).astype(f32))
            assert np.array_equal(o.v[:P], (f32(0.95) * v1[:P]).astype(f32))
            assert not np.array_equal(o.master[:P], th1[:P])
        # ZERO_SKIP leaves the packet's state untouched
        o2 = _mk(W, n, P, 0.5, opt=opt, theta=theta, flags=oracle.ZERO_SKIP)
        o2.step(1, g, recv_force=np.array([0b111, 0b111], np.uint64))
        a, b, c = o2.master.copy(), o2.m.copy(), o2.v.copy()
        o2.step(2, g, recv_force=force)
        assert np.array_equal(o2.master[:P], a[:P]) and np.array_equal(o2.m[:P], b[:P])
        assert np.array_equal(o2.v[:P], c[:P])
        assert not np.array_equal(o2.master[P:], a[P:])


def test_self_lossless_flag_always_delivers_the_owners_piece():
    W, P, K = 4, 8, 64
    n = P * K
    g = _rand_grads(np.random.default_rng(2), W, n)
    o = _mk(W, n, P, 0.6, flags=oracle.SELF_LOSSLESS)
    r = o.step(1, g)
    o0 = _mk(W, n, P, 0.6)
    r0 = o0.step(1, g)
    for k in range(K):
        j = o.owner(k)
        assert (int(r["recv_bits"][k]) >> j) & 1
        assert int(r["recv_bits"][k]) == int(r0["recv_bits"][k]) | (1 << j)
    assert any(not (int(r0["recv_bits"][k]) >> o0.owner(k)) & 1 for k in range(K))


def test_masks_counts_follow_the_hash_and_shard_map():
    """recv bit i of packet k is the (src=i, dst=owner(k)) draw; stale bit i the (src=owner, dst=i) draw;
    shards are contiguous runs of ceil(K/W) packets (ragged tail, possibly empty shards)."""
    for W, n, P, base in ((4, 1000, 64, 0), (5, 8 * 7, 8, 1234567), (8, 8 * 3, 8, 5)):
        K = (n + P - 1) // P
        pps = (K + W - 1) // W
        o = _mk(W, n, P, 0.25, seed=9, packet_base=base)
        g = _rand_grads(np.random.default_rng(3), W, n)
        r = o.step(4, g)
        for k in range(K):
            j = k // pps
            assert o.owner(k) == j
            bits = sum(oracle.delivered(9, 4, i, j, base + k, 0.25) << i for i in range(W))
            assert int(r["recv_bits"][k]) == bits
            assert r["count"][k] == bin(bits).count("1")
            st = sum((1 - oracle.delivered(9, 4, j, i, base + k, 0.25)) << i for i in range(W) if i != j)
            assert int(r["stale_bits"][k]) == st


def test_fp32_contract_path_tracks_the_fp64_path():
    W, n, P = 8, 4096 + 24, 256
    rng = np.random.default_rng(4)
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    for opt, lr in ((SGD, 1e-2), (ADAM, 3e-4)):
        a = _mk(W, n, P, 0.1, opt=opt, lr=lr, theta=theta, gd=BF16, rd=BF16)
        b = _mk(W, n, P, 0.1, opt=opt, lr=lr, theta=theta, gd=BF16, rd=BF16, f64=True)
        for t in range(1, 21):
            g = [torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
                 for x in _rand_grads(rng, W, n)]
            ra, rb = a.step(t, g), b.step(t, g)
            assert np.array_equal(ra["recv_bits"], rb["recv_bits"])
            assert np.max(np.abs(ra["ghat"] - rb["ghat"])) <= 2e-7 * np.max(np.abs(rb["ghat"]))
        assert np.max(np.abs(a.master - b.master)) <= 1e-6 * np.max(np.abs(b.master))
        assert np.max(np.abs(a.m - b.m)) <= 1e-5 * np.max(np.abs(b.m))
        assert np.max(np.abs(a.v - b.v)) <= 1e-5 * np.max(np.abs(b.v))


def test_slab_by_slab_equals_whole_bucket():
    W, P = 4, 16
    n = P * 37 + 8                               # ragged last packet, K = 38, pps = 10
    rng = np.random.default_rng(6)
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    grads = [[_rand_grads(rng, W, n)] for _ in range(3)]
    whole = _mk(W, n, P, 0.2, opt=ADAM, lr=3e-4, theta=theta, rd=BF16)
    cuts = [0, 7, 20, 38]
    slabs = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        e0, e1 = a * P, min(n, b * P)
        slabs.append((e0, e1, Oracle(W=W, n=n, packet_elems=P, p_grad=0.2, p_param=0.2, seed=0, grad_dtype=F32,
                                     replica_dtype=BF16, optimizer=ADAM, theta0=theta[e0:e1], lr=3e-4,
                                     k0=a, n_slab=e1 - e0)))
    for t, (g,) in enumerate(grads, start=1):
        rw = whole.step(t, g)
        tot = np.zeros(W)
        for e0, e1, o in slabs:
            r = o.step(t, [x[e0:e1] for x in g])
            assert np.array_equal(r["ghat"], rw["ghat"][e0:e1])
            assert np.array_equal(o.master, whole.master[e0:e1])
            for i in range(W):
                assert np.array_equal(o.replicas[i], whole.replicas[i][e0:e1])
            tot += r["sumsq"]
        assert np.allclose(tot, rw["sumsq"], rtol=1e-12)


def test_mask_only_routine_agrees_with_the_step():
    W, P, K = 7, 8, 500
    n = P * K - 3
    o = _mk(W, n, P, 0.3, seed=21, flags=oracle.SELF_LOSSLESS, packet_base=77)
    g = _rand_grads(np.random.default_rng(0), W, n)
    for t in (1, 2, 9):
        r = o.step(t, g)
        recv, stale, count = o.masks(t)
        assert np.array_equal(recv, r["recv_bits"]) and np.array_equal(stale, r["stale_bits"])
        assert np.array_equal(count, r["count"])
        recv2, stale2, count2 = o.masks(t, k0=100, packets=50)
        assert np.array_equal(recv2, recv[100:150]) and np.array_equal(stale2, stale[100:150])
