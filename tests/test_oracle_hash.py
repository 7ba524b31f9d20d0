"""Pins for the oracle's delivery-indicator hash (Section 3: s, r ~ Bernoulli(1-p);
Algorithm 1: Uniform(0,1) < p). CPU only."""
import os

import numpy as np

from oracle import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_mix64_matches_published_splitmix64_vectors():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "splitmix64_vectors.txt")) if not l.startswith("#")]
    assert len(rows) >= 3
    for _, state, out in rows:
        assert oracle.mix64(int(state, 16)) == int(out, 16)


def test_threshold_is_floor_p_times_2_32():
    assert oracle.threshold(0.0) == 0
    assert oracle.threshold(0.5) == 1 << 31
    assert oracle.threshold(0.25) == 1 << 30
    assert oracle.threshold(0.1) == 429496729          # floor(0.1 * 2^32) = floor(429496729.6)
    assert oracle.threshold(1.0 - 2.0 ** -32) == (1 << 32) - 1


def test_p_zero_never_drops():
    for k in range(2000):
        assert oracle.delivered(7, 1 + k % 5, k % 8, (k // 8) % 8, k, 0.0) == 1


def test_deterministic_replay_and_seed_sensitivity():
    a = [oracle.hash_u32(3, 9, 1, 2, k) for k in range(256)]
    assert a == [oracle.hash_u32(3, 9, 1, 2, k) for k in range(256)]
    b = [oracle.hash_u32(4, 9, 1, 2, k) for k in range(256)]
    assert sum(x == y for x, y in zip(a, b)) == 0
    # direction matters: (src,dst) and (dst,src) are different transmissions
    c = [oracle.hash_u32(3, 9, 2, 1, k) for k in range(256)]
    assert sum(x == y for x, y in zip(a, c)) == 0


def _bits(seed, steps, srcs, dsts, packets, p):
    out = np.empty((len(steps), len(srcs), len(dsts), len(packets)), np.uint8)
    for a, t in enumerate(steps):
        for b, s in enumerate(srcs):
            for c, d in enumerate(dsts):
                for e, k in enumerate(packets):
                    out[a, b, c, e] = oracle.delivered(seed, t, s, d, k, p)
    return out


def test_drop_frequency_per_stream_within_binomial_bounds():
    for p in (0.01, 0.1, 0.3):
        steps, packets = range(1, 41), range(0, 400)
        bits = _bits(11, steps, range(4), range(4), packets, p)
        nper = len(steps) * len(packets)
        drops = (1 - bits.astype(np.int64)).sum(axis=(0, 3))       # per (src,dst) stream
        sd = np.sqrt(nper * p * (1 - p))
        assert np.all(np.abs(drops - nper * p) < 4.5 * sd), (p, drops)
        tot = drops.sum()
        assert abs(tot - 16 * nper * p) < 4 * np.sqrt(16 * nper * p * (1 - p))


def test_uniformity_of_u32_chi_square():
    vals = np.array([oracle.hash_u32(5, 1 + (k >> 12), k & 7, (k >> 3) & 7, k >> 6) for k in range(1 << 16)],
                    dtype=np.uint64)
    hist = np.bincount((vals >> 24).astype(np.int64), minlength=256)   # top byte, 256 bins
    expect = len(vals) / 256
    chi2 = ((hist - expect) ** 2 / expect).sum()
    # chi2 with 255 dof: mean 255, sd 22.6
    assert 255 - 5 * 22.6 < chi2 < 255 + 5 * 22.6
    low = np.bincount((vals & 0xFF).astype(np.int64), minlength=256)   # low byte of the 32-bit value
    chi2 = ((low - expect) ** 2 / expect).sum()
    assert 255 - 5 * 22.6 < chi2 < 255 + 5 * 22.6


def test_no_lag1_correlation_along_any_counter():
    p = 0.3
    bits = _bits(2, range(1, 33), range(8), range(8), range(64), p).astype(np.float64) - (1 - p)
    var = p * (1 - p)
    for axis in range(4):
        a = np.take(bits, range(0, bits.shape[axis] - 1), axis=axis)
        b = np.take(bits, range(1, bits.shape[axis]), axis=axis)
        r = (a * b).mean() / var
        assert abs(r) < 5.0 / np.sqrt(a.size), (axis, r)


def test_gradient_and_broadcast_draws_are_distinct_streams():
    # grad tuple (i, owner) and broadcast tuple (owner, i) coincide only at i == owner
    p = 0.5
    same = 0
    tot = 0
    for k in range(500):
        for i in range(1, 4):
            tot += 1
            same += oracle.delivered(1, 3, i, 0, k, p) == oracle.delivered(1, 3, 0, i, k, p)
    assert abs(same - tot / 2) < 4 * np.sqrt(tot / 4)
