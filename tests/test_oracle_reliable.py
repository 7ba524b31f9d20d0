"""Pins for the oracle's hybrid reliable/unreliable transport (the paper's first Future Direction:
important traffic on a reliable channel, the long tail best-effort) and the per-packet gradient norms
an importance rule starts from. CPU only."""
import numpy as np

from oracle import oracle
from oracle.oracle import F32, SGD, Oracle

f32 = np.float32


def _mk(W, K, P, p, seed=0, **kw):
    n = K * P
    return Oracle(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=F32, replica_dtype=F32,
                  optimizer=SGD, theta0=np.zeros(n, f32), lr=1e-2, **kw), n


def test_reliable_links_are_never_lost_and_the_others_are_unchanged():
    W, K, P, p = 5, 300, 8, 0.4
    rng = np.random.default_rng(0)
    a, n = _mk(W, K, P, p, seed=3)
    b, _ = _mk(W, K, P, p, seed=3)
    g = [rng.standard_normal(n).astype(f32) for _ in range(W)]
    rel = rng.integers(0, 1 << W, (2, K)).astype(np.uint64)
    ra, rb = a.step(1, g, reliable=rel), b.step(1, g)
    all_w = np.uint64((1 << W) - 1)
    assert np.array_equal(ra["recv_bits"], rb["recv_bits"] | (rel[0] & all_w))
    assert np.array_equal(ra["stale_bits"], rb["stale_bits"] & ~rel[1])
    # everything reliable = the lossless step; nothing reliable = the plain lossy step
    c, _ = _mk(W, K, P, p, seed=3)
    d, _ = _mk(W, K, P, 0.0, seed=3)
    rc = c.step(1, g, reliable=np.full((2, K), all_w, np.uint64))
    rd = d.step(1, g)
    assert np.array_equal(rc["ghat"], rd["ghat"]) and np.all(rc["stale_bits"] == 0)
    e, _ = _mk(W, K, P, p, seed=3)
    re = e.step(1, g, reliable=np.zeros((2, K), np.uint64))
    assert np.array_equal(re["ghat"], rb["ghat"]) and np.array_equal(re["stale_bits"], rb["stale_bits"])


def test_algorithm1_mode_uses_bit_zero():
    W, K, P = 3, 200, 8
    o, n = _mk(W, K, P, 0.6, seed=1, alg1=True)
    g = [np.ones(n, f32) for _ in range(W)]
    rel = np.zeros((2, K), np.uint64)
    rel[0, ::2] = 1
    r = o.step(1, g, reliable=rel)
    assert np.all(r["count"][::2] == W)
    assert 0 < (r["count"][1::2] == 0).sum() < K // 2


def test_packet_norms_against_direct_sums():
    W, K, P = 4, 37, 16
    o, n = _mk(W, K, P, 0.1)
    n_r = n - 5                                   # ragged last packet
    o2 = Oracle(W=W, n=n_r, packet_elems=P, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=F32, replica_dtype=F32,
                optimizer=SGD, theta0=np.zeros(n_r, f32), lr=1e-2)
    rng = np.random.default_rng(2)
    g = [rng.standard_normal(n_r).astype(f32) for _ in range(W)]
    got = o2.packet_sqnorms(g)
    for i in range(W):
        for k in range(K):
            want = float((g[i][k * P:(k + 1) * P].astype(np.float64) ** 2).sum())
            assert np.isclose(got[i, k], want, rtol=1e-14)
