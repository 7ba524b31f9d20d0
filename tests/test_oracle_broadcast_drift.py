"""Pins for the oracle's lossy broadcast and drift (Section 3 step (4); Theorem "Bounded Model
Drift" and the four-case rule in its proof). CPU only."""
import os

import numpy as np

from oracle import oracle
from oracle.oracle import BF16, F32, SGD, Oracle

f32 = np.float32
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _closed_forms():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "drift_closed_forms.txt")) if not l.startswith("#")]
    return {float(r[0]): tuple(float(x) for x in r[1:]) for r in rows}


def _run(W, K, P, p, steps, *, rd=F32, seed=0, lr=1e-2, sigma_g=1e-3, p_grad=None):
    n = K * P
    rng = np.random.default_rng(seed)
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    o = Oracle(W=W, n=n, packet_elems=P, p_grad=p if p_grad is None else p_grad, p_param=p, seed=seed,
               grad_dtype=F32, replica_dtype=rd, optimizer=SGD, theta0=theta, lr=lr, track_age=True)
    return o, rng, n


def test_stale_retention_history_invariant():
    """Replica i's packet k is exactly the wire value the owner sent `age` steps ago."""
    W, K, P, p = 5, 23, 8, 0.35
    for rd in (F32, BF16):
        o, rng, n = _run(W, K, P, p, 0, rd=rd)
        hist = [oracle.cast_wire(o.master.astype(f32), rd)]
        for t in range(1, 31):
            g = [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)]
            r = o.step(t, g)
            hist.append(oracle.cast_wire(o.master.astype(f32), rd))
            for i in range(W):
                for k in range(K):
                    a = int(o.age[i][k])
                    assert a <= t
                    assert np.array_equal(o.replicas[i][k * P:(k + 1) * P], hist[t - a][k * P:(k + 1) * P])
                    if o.owner(k) == i:
                        assert a == 0 and not (int(r["stale_bits"][k]) >> i) & 1


def test_four_case_rule_of_the_drift_proof():
    """D_{t+1} between two replicas: 0 if both received; D_t if both missed; new value minus the
    loser's old copy if exactly one received."""
    W, K, P, p = 4, 40, 8, 0.4
    o, rng, n = _run(W, K, P, p, 0)
    seen = set()
    for t in range(1, 16):
        before = [r.copy() for r in o.replicas]
        g = [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)]
        res = o.step(t, g)
        new = o.master
        for k in range(K):
            sl = slice(k * P, (k + 1) * P)
            st = int(res["stale_bits"][k])
            for i in range(W):
                for q in range(i + 1, W):
                    si, sq = not (st >> i) & 1, not (st >> q) & 1
                    D = o.replicas[i][sl] - o.replicas[q][sl]
                    if si and sq:
                        assert np.all(D == 0)
                    elif not si and not sq:
                        assert np.array_equal(D, before[i][sl] - before[q][sl])
                    elif si:
                        assert np.array_equal(D, new[sl] - before[q][sl])
                    else:
                        assert np.array_equal(D, before[i][sl] - new[sl])
                    seen.add((si, sq))
    assert len(seen) == 4


def test_drift_sumsq_matches_brute_force_and_standalone():
    W, K, P, p = 6, 31, 16, 0.3
    for rd in (F32, BF16):
        o, rng, n = _run(W, K, P, p, 0, rd=rd)
        for t in range(1, 9):
            g = [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)]
            r = o.step(t, g)
            wire = oracle.cast_wire(o.master.astype(f32), rd)
            x = oracle.bf16_bits_to_f32(wire).astype(np.float64) if rd == BF16 else wire.astype(np.float64)
            for i in range(W):
                rep = o.replicas[i]
                rep = oracle.bf16_bits_to_f32(rep).astype(np.float64) if rd == BF16 else rep.astype(np.float64)
                want = float(((rep - x) ** 2).sum())
                assert np.isclose(r["sumsq"][i], want, rtol=1e-12, atol=0)
            assert np.allclose(o.drift_sumsq(), r["sumsq"], rtol=1e-12, atol=0)
            assert np.allclose(r["norms"], np.sqrt(r["sumsq"]))


def test_stationary_drift_is_order_one_and_matches_exact_constants():
    """Bounded Model Drift: E[D^2] does not grow with t. For i.i.d. zero-mean increments of variance
    sigma^2 the four-case rule gives the stationary values 2p/(1-p^2) sigma^2 (replica pair) and
    p/(1-p) sigma^2 (replica vs owner); the theorem's printed 2p/(1+p) sigma^2 is their first-order
    form and is reported beside them."""
    forms = _closed_forms()
    W, K, P, T = 4, 4096, 4, 200
    for p in (0.1, 0.3):
        paper, pair_c, owner_c = forms[p]
        # lossless gradients (p_grad = 0) make the increments exactly i.i.d. across steps
        o, rng, n = _run(W, K, P, p, 0, seed=int(p * 100), p_grad=0.0)
        pair, own, sig2 = [], [], []
        for t in range(1, T + 1):
            prev = o.master.copy()
            g = [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)]
            o.step(t, g)
            sig2.append(np.mean((o.master.astype(np.float64) - prev) ** 2))
            # only packets where neither replica is the owner (the theorem's i, k are receivers)
            keep = np.repeat(np.array([o.owner(k) not in (1, 2) for k in range(K)]), P)
            d = o.replicas[1].astype(np.float64) - o.replicas[2].astype(np.float64)
            pair.append(np.mean(d[keep] ** 2))
            keep0 = np.repeat(np.array([o.owner(k) != 1 for k in range(K)]), P)
            d0 = o.replicas[1].astype(np.float64) - o.master.astype(np.float64)
            own.append(np.mean(d0[keep0] ** 2))
        s2 = np.mean(sig2)
        pair, own = np.array(pair) / s2, np.array(own) / s2
        assert abs(pair[40:].mean() / pair_c - 1) < 0.03, (p, pair[40:].mean(), pair_c, paper)
        assert abs(own[40:].mean() / owner_c - 1) < 0.03, (p, own[40:].mean(), owner_c)
        # O(1): no growth between the two halves of the run, and never far above the constant
        assert abs(pair[40:120].mean() / pair[120:].mean() - 1) < 0.08
        assert pair.max() < 1.6 * pair_c
        # the printed constant is the small-p form: below the exact value by the factor (1 - p)
        assert np.isclose(paper / pair_c, 1 - p, rtol=1e-9)


def test_drift_transient_follows_the_recurrence():
    """E_t from a synchronised start (E_0 = 0) follows the proof's recurrence with the loser's
    staleness kept: A_{t+1} = p (A_t + s2), E_{t+1} = p^2 E_t + 2p(1-p)(s2 + A_t)."""
    W, K, P, p, T = 3, 8192, 2, 0.3, 12
    o, rng, n = _run(W, K, P, p, 0, seed=77, p_grad=0.0)
    E, A, s2s, meas = 0.0, 0.0, [], []
    keep = np.repeat(np.array([o.owner(k) == 0 for k in range(K)]), P)   # receivers 1 and 2
    for t in range(1, T + 1):
        prev = o.master.copy()
        g = [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)]
        o.step(t, g)
        s2s.append(np.mean((o.master.astype(np.float64) - prev)[keep] ** 2))
        d = (o.replicas[1].astype(np.float64) - o.replicas[2].astype(np.float64))[keep]
        meas.append(np.mean(d ** 2))
    s2 = np.mean(s2s)
    for t in range(T):
        E, A = p * p * E + 2 * p * (1 - p) * (s2 + A), p * (A + s2)
        assert abs(meas[t] / E - 1) < 0.12, (t, meas[t], E)


def test_stale_fraction_is_binomial():
    W, K, P, p = 8, 4000, 8, 0.1
    o, rng, n = _run(W, K, P, p, 0, seed=3)
    g = [(rng.standard_normal(n) * 1e-3).astype(f32) for _ in range(W)]
    r = o.step(1, g)
    pps = (K + W - 1) // W
    for i in range(W):
        stale_i = sum((int(b) >> i) & 1 for b in r["stale_bits"])
        trials = K - pps
        assert abs(stale_i - trials * p) < 4.5 * np.sqrt(trials * p * (1 - p))
    assert int(r["count"].sum()) == sum(bin(int(b)).count("1") for b in r["recv_bits"])


def test_pairwise_drift_matrix_against_direct_sums_and_the_pair_constant():
    """The theorem's own quantity between two receivers: symmetric, zero diagonal, equal to the direct
    sum of squared differences, and stationary at 2p/(1-p^2) sigma^2 per element where neither owns."""
    forms = _closed_forms()
    W, K, P, p, T = 4, 4096, 4, 0.3, 160
    o, rng, n = _run(W, K, P, p, 0, seed=12, p_grad=0.0)
    acc, sig2 = [], []
    keep = np.repeat(np.array([o.owner(k) not in (1, 2) for k in range(K)]), P)
    for t in range(1, T + 1):
        prev = o.master.copy()
        o.step(t, [(rng.standard_normal(n) * 1e-1).astype(f32) for _ in range(W)])
        if t > 40:
            sig2.append(np.mean((o.master.astype(np.float64) - prev) ** 2))
            d2 = o.pairwise_sumsq()
            assert np.allclose(d2, d2.T, rtol=1e-14) and np.all(np.diag(d2) == 0)
            R = np.stack([r.astype(np.float64) for r in o.replicas])
            want = ((R[:, None, :] - R[None, :, :]) ** 2).sum(axis=2)
            assert np.allclose(d2, want, rtol=1e-12)
            # the part of D^2(1,2) over packets that neither 1 nor 2 owns
            acc.append(np.sum((R[1] - R[2])[keep] ** 2) / keep.sum())
    assert abs(np.mean(acc) / (np.mean(sig2) * forms[p][1]) - 1) < 0.03
