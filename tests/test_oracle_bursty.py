"""Pins for the oracle's bursty loss: a two-state (Gilbert-Elliott) chain per link and packet, the
correlated-loss regime the paper's Limitations leave open. CPU only."""
import numpy as np

from oracle import oracle
from oracle.oracle import F32, SGD, Oracle

f32 = np.float32


def _mk(W, K, P, burst, *, seed=0, p=0.0, lr=1e-2, alg1=False, flags=0, track_age=False):
    n = K * P
    return Oracle(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=F32, replica_dtype=F32,
                  optimizer=SGD, theta0=np.zeros(n, f32), lr=lr, burst=burst, alg1=alg1, flags=flags,
                  track_age=track_age), n


def _bits(a, W):
    return ((a[:, None] >> np.arange(W, dtype=np.uint64)) & np.uint64(1)).astype(np.int8)


def test_chain_follows_the_recurrence_on_the_hash():
    W, K, P, T, a, b = 3, 5, 8, 20, 0.3, 0.4
    o, n = _mk(W, K, P, (a, b), seed=13)
    Te, Tl = oracle.threshold(a), oracle.threshold(1 - b)
    gstate = np.zeros((K, W), int)
    pstate = np.zeros((K, W), int)
    g = [np.zeros(n, f32) for _ in range(W)]
    for t in range(1, T + 1):
        prev = o.burst_state.copy()
        r = o.step(t, g)
        for k in range(K):
            j = o.owner(k)
            for i in range(W):
                u = oracle.hash_u32(13, t, i, j, k)
                gstate[k, i] = int(u < Tl) if gstate[k, i] else int(u < Te)
                assert ((int(r["recv_bits"][k]) >> i) & 1) == 1 - gstate[k, i]
                if i != j:
                    u = oracle.hash_u32(13, t, j, i, k)
                    pstate[k, i] = int(u < Tl) if pstate[k, i] else int(u < Te)
                    assert ((int(r["stale_bits"][k]) >> i) & 1) == pstate[k, i]
        assert np.array_equal(_bits(o.burst_state[0], W), gstate)
        assert np.array_equal(_bits(o.burst_state[1], W), pstate)
        assert not np.array_equal(prev, o.burst_state) or t > 1


def test_stationary_loss_rate_and_burst_lengths():
    W, K, P, T = 4, 600, 8, 300
    for a, b in ((0.05, 0.25), (0.2, 0.8), (0.1, 0.5)):
        o, n = _mk(W, K, P, (a, b), seed=3)
        g = [np.zeros(n, f32) for _ in range(W)]
        lost = []
        for t in range(1, T + 1):
            r = o.step(t, g)
            lost.append(1 - _bits(r["recv_bits"], W))
        L = np.stack(lost[50:]).astype(np.float64)              # [T', K, W] after the all-good start has mixed
        pi_b = a / (a + b)
        assert abs(L.mean() / pi_b - 1) < 0.03
        # a burst (run of lost steps on one link) is geometric with mean 1 / P(bad->good)
        x = np.stack(lost).reshape(T, -1).T                    # one row per (packet, link)
        starts = ((x[:, 1:] == 1) & (x[:, :-1] == 0)).sum()
        runs_total = x[:, 1:].sum()
        assert abs(runs_total / starts * b - 1) < 0.05
        # lag-1 correlation of the loss indicator is 1 - a - b
        c = ((L[1:] - pi_b) * (L[:-1] - pi_b)).mean() / (pi_b * (1 - pi_b))
        assert abs(c - (1 - a - b)) < 0.03


def test_independent_special_case_has_the_bernoulli_statistics():
    """P(good->bad) = p, P(bad->good) = 1 - p makes the chain memoryless: loss rate p, no correlation."""
    W, K, P, T, p = 4, 500, 8, 120, 0.2
    o, n = _mk(W, K, P, (p, 1 - p), seed=8)
    g = [np.zeros(n, f32) for _ in range(W)]
    lost = np.stack([1 - _bits(o.step(t, g)["recv_bits"], W) for t in range(1, T + 1)]).astype(np.float64)
    assert abs(lost.mean() / p - 1) < 0.03
    c = ((lost[1:] - p) * (lost[:-1] - p)).mean() / (p * (1 - p))
    assert abs(c) < 0.01


def test_drift_under_bursts_matches_the_mean_age():
    """With i.i.d. increments a replica's squared distance from the owner is sigma^2 times its mean age;
    for the chain the mean age is pi_bad / P(bad->good) (p/(1-p) in the memoryless case)."""
    W, K, P, T, a, b = 4, 4096, 4, 260, 0.1, 0.3
    n = K * P
    rng = np.random.default_rng(0)
    o = Oracle(W=W, n=n, packet_elems=P, p_grad=0.0, p_param=0.0, seed=2, grad_dtype=F32, replica_dtype=F32,
               optimizer=SGD, theta0=np.zeros(n, f32), lr=1e-2, burst=(a, b), track_age=True)
    ratios, sig2, ages = [], [], []
    keep = np.repeat(np.array([o.owner(k) != 1 for k in range(K)]), P)
    for t in range(1, T + 1):
        prev = o.master.copy()
        # lossless-looking gradients are not available here (gradient links are bursty too), so use
        # increments whose size does not depend on the received count: identical workers
        gi = (rng.standard_normal(n) * 1e-1).astype(f32)
        o.step(t, [gi] * W)
        if t > 60:
            d = (o.replicas[1].astype(np.float64) - o.master.astype(np.float64))[keep]
            ratios.append(np.mean(d ** 2))
            sig2.append(np.mean((o.master.astype(np.float64) - prev)[keep] ** 2))
            ages.append(np.mean(o.age[1][np.array([o.owner(k) != 1 for k in range(K)])]))
    mean_age = (a / (a + b)) / b
    assert abs(np.mean(ages) / mean_age - 1) < 0.04
    assert abs(np.mean(ratios) / (np.mean(sig2) * mean_age) - 1) < 0.06


def test_algorithm1_mode_uses_one_chain_per_packet():
    W, K, P, T = 3, 800, 8, 200
    o, n = _mk(W, K, P, (0.1, 0.4), seed=4, alg1=True)
    g = [np.zeros(n, f32) for _ in range(W)]
    kept = np.stack([o.step(t, g)["count"] == W for t in range(1, T + 1)])[40:]
    assert abs((1 - kept.mean()) / (0.1 / 0.5) - 1) < 0.04
    assert np.all(o.burst_state[0] <= 1)                         # only bit 0 is used
