"""Pins for the oracle's Algorithm 1 mode (the paper's "Drop simulation on worker n"): the gradient
reduce is reliable, one draw per packet either keeps the fresh aggregate (saving it as g_prev) or
falls back to g_prev; the parameter half is the stale-retaining broadcast. CPU only."""
import numpy as np

from oracle import oracle
from oracle.oracle import ADAM, BF16, F32, SGD, Oracle

f32 = np.float32


def _mk(W, n, P, pg, pp, *, seed=0, opt=SGD, lr=1e-2, alg1=True, f64=False, theta=None, rd=F32, flags=0):
    theta = np.zeros(n, f32) if theta is None else theta
    return Oracle(W=W, n=n, packet_elems=P, p_grad=pg, p_param=pp, seed=seed, grad_dtype=F32, replica_dtype=rd,
                  optimizer=opt, theta0=theta, lr=lr, alg1=alg1, f64=f64, flags=flags)


def _grads(rng, W, n, sigma=1.0, mean=None):
    base = 0.0 if mean is None else mean
    return [(base + rng.standard_normal(n) * sigma).astype(f32) for _ in range(W)]


def test_no_loss_equals_the_section3_path_and_prev_tracks_the_aggregate():
    rng = np.random.default_rng(0)
    W, P, K = 5, 16, 13
    n = P * K + 8
    theta = rng.standard_normal(n).astype(f32)
    a = _mk(W, n, P, 0.0, 0.2, theta=theta, opt=ADAM, lr=3e-4, rd=BF16)
    b = _mk(W, n, P, 0.0, 0.2, theta=theta, opt=ADAM, lr=3e-4, rd=BF16, alg1=False)
    for t in range(1, 7):
        g = _grads(rng, W, n, 1e-3)
        ra, rb = a.step(t, g), b.step(t, g)
        assert np.array_equal(ra["ghat"], rb["ghat"]) and np.array_equal(a.master, b.master)
        assert np.array_equal(a.ghat_prev, ra["ghat"])
        assert np.array_equal(ra["stale_bits"], rb["stale_bits"])
        for x, y in zip(a.replicas, b.replicas):
            assert np.array_equal(x, y)
        assert np.all(ra["count"] == W)


def test_dropped_packet_reuses_the_last_surviving_aggregate():
    """g <- g_prev on a drop, g_prev <- g otherwise; before anything survived g_prev is zero."""
    rng = np.random.default_rng(1)
    W, P, K, T = 3, 8, 6, 12
    n = P * K
    o = _mk(W, n, P, 0.5, 0.0, f64=True)
    last = np.zeros(n)
    keep_hist = rng.integers(0, 2, (T, K))
    keep_hist[0, 0] = 0                                   # a first-step drop: nothing saved yet
    for t in range(1, T + 1):
        g = _grads(rng, W, n)
        fresh = np.mean(np.stack(g).astype(np.float64), axis=0)
        prev_before = o.ghat_prev.copy()
        r = o.step(t, g, recv_force=keep_hist[t - 1].astype(np.uint64))
        for k in range(K):
            sl = slice(k * P, (k + 1) * P)
            if keep_hist[t - 1, k]:
                assert np.allclose(r["ghat"][sl], fresh[sl], rtol=1e-14)
                last[sl] = r["ghat"][sl]
                assert r["count"][k] == W and int(r["recv_bits"][k]) == (1 << W) - 1
            else:
                assert np.array_equal(r["ghat"][sl], last[sl])
                assert np.array_equal(o.ghat_prev[sl], prev_before[sl])      # untouched on a drop
                assert r["count"][k] == 0 and int(r["recv_bits"][k]) == 0
        assert np.array_equal(o.ghat_prev, last)
    assert np.all(last[:P] != 0) or keep_hist[:, 0].sum() == 0


def test_one_draw_per_packet_with_the_stated_rate_and_independent_of_the_broadcast_draws():
    W, P, K, pg, pp = 4, 8, 3000, 0.2, 0.3
    n = P * K
    o = _mk(W, n, P, pg, pp, seed=5)
    g = [np.zeros(n, f32) for _ in range(W)]
    r = o.step(1, g)
    kept = r["count"] == W
    assert set(np.unique(r["count"])) <= {0, W}
    assert abs((~kept).sum() - K * pg) < 4.5 * np.sqrt(K * pg * (1 - pg))
    # the draw is the (owner, owner) link of the hash
    for k in range(0, K, 97):
        j = o.owner(k)
        assert kept[k] == bool(oracle.delivered(5, 1, j, j, k, pg))
    stale_any = np.array([int(b) != 0 for b in r["stale_bits"]])
    both = (stale_any & ~kept).sum()
    expect = K * pg * (1 - (1 - pp) ** (W - 1))
    assert abs(both - expect) < 5 * np.sqrt(expect)


def test_reuse_keeps_the_mean_and_has_lag_one_correlation_p():
    """With a stationary gradient (fixed mean + fresh noise) the reused aggregate has the same mean,
    and consecutive aggregates coincide with probability p: their correlation is p."""
    rng = np.random.default_rng(2)
    W, P, K, T, pg = 4, 4, 2048, 120, 0.3
    n = P * K
    mean = rng.standard_normal(n)
    o = _mk(W, n, P, pg, 0.0, f64=True, seed=9)
    hist = []
    for t in range(1, T + 1):
        r = o.step(t, _grads(rng, W, n, 1.0, mean))
        hist.append(r["ghat"].copy())
    H = np.stack(hist[20:]) - mean                         # after the zero-initialised prev has washed out
    var = (H ** 2).mean()
    assert abs(var / (1.0 / W) - 1) < 0.03                 # variance of a W-worker mean
    assert abs(H.mean()) < 4 * np.sqrt(var / H.size * (1 + pg) / (1 - pg))
    lag1 = (H[1:] * H[:-1]).mean() / var
    assert abs(lag1 - pg) < 0.02
    lag2 = (H[2:] * H[:-2]).mean() / var
    assert abs(lag2 - pg ** 2) < 0.02


def test_fp32_contract_path_tracks_fp64_in_alg1_mode():
    rng = np.random.default_rng(3)
    W, P, K = 8, 64, 40
    n = P * K
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    a = _mk(W, n, P, 0.2, 0.2, theta=theta, opt=ADAM, lr=3e-4)
    b = _mk(W, n, P, 0.2, 0.2, theta=theta, opt=ADAM, lr=3e-4, f64=True)
    for t in range(1, 16):
        g = _grads(rng, W, n, 1e-3)
        ra, rb = a.step(t, g), b.step(t, g)
        assert np.array_equal(ra["count"], rb["count"])
        assert np.max(np.abs(ra["ghat"] - rb["ghat"])) <= 3e-7 * np.max(np.abs(rb["ghat"]))
    assert np.max(np.abs(a.master - b.master)) <= 1e-6 * np.max(np.abs(b.master))
