"""Pins for the oracle's closed-loop gradient stand-in (Section 3 step (1): each worker evaluates
its gradient at its own, possibly stale, replica). CPU only."""
import numpy as np

from oracle.oracle import F32, SGD, Oracle

f32 = np.float32


def _mk(W, n, P, p, theta, lr, f64=True, seed=0):
    return Oracle(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=F32, replica_dtype=F32,
                  optimizer=SGD, theta0=theta, lr=lr, f64=f64)


def test_lossless_noise_free_run_contracts_geometrically():
    """p = 0, no noise: theta_t - x* = (1 - lr a)^t (theta_0 - x*), element by element."""
    rng = np.random.default_rng(0)
    W, n, P, lr, T = 3, 96, 8, 0.25, 12
    theta0 = rng.standard_normal(n).astype(f32)
    a = rng.uniform(0.5, 1.5, n).astype(f32)
    xs = rng.standard_normal(n).astype(f32)
    o = _mk(W, n, P, 0.0, theta0, lr)
    zero = [np.zeros(n, f32) for _ in range(W)]
    for t in range(1, T + 1):
        o.step(t, o.closed_loop_grads(a, xs, zero))
    want = xs.astype(np.float64) + (1 - lr * a.astype(np.float64)) ** T * (theta0.astype(np.float64) - xs)
    # gradients are rounded to fp32 each step; the trajectory itself is in double
    assert np.max(np.abs(o.master - want)) <= 5e-7 * np.max(np.abs(want))


def test_gradient_is_evaluated_at_each_workers_own_replica():
    rng = np.random.default_rng(1)
    W, n, P = 4, 64, 8
    o = _mk(W, n, P, 0.5, rng.standard_normal(n).astype(f32), 0.1, f64=False, seed=3)   # the fp32 contract build
    a = rng.uniform(0.5, 1.5, n).astype(f32)
    xs = rng.standard_normal(n).astype(f32)
    for t in range(1, 6):                          # lossy steps make the replicas differ
        noise = [rng.standard_normal(n).astype(f32) * 0.1 for _ in range(W)]
        g = o.closed_loop_grads(a, xs, noise)
        for i in range(W):
            want = (a * (o.replicas[i] - xs)).astype(f32) + noise[i]
            assert np.array_equal(g[i], want.astype(f32))
        o.step(t, g)
    assert any(not np.array_equal(o.replicas[0], r) for r in o.replicas[1:])


def test_loss_floor_rises_with_the_drop_rate():
    """The trend of the paper's Table 1 in miniature: more loss, worse final objective."""
    rng = np.random.default_rng(2)
    W, n, P, lr, T = 8, 4096, 16, 0.1, 150
    theta0 = rng.standard_normal(n).astype(f32)
    a = rng.uniform(0.5, 1.5, n).astype(f32)
    xs = rng.standard_normal(n).astype(f32)
    floors = []
    for p in (0.0, 0.2, 0.4):
        o = _mk(W, n, P, p, theta0, lr, seed=7)
        nrng = np.random.default_rng(11)
        tail = []
        for t in range(1, T + 1):
            noise = [nrng.standard_normal(n).astype(f32) for _ in range(W)]
            o.step(t, o.closed_loop_grads(a, xs, noise))
            if t > 100:
                tail.append(0.5 * np.mean(a * (o.master - xs) ** 2))
        floors.append(np.mean(tail))
    assert floors[0] < floors[1] < floors[2]
    # lossless floor of SGD on a quadratic: 1/2 a * lr sigma^2 / (W (2 - lr a)) averaged over a
    a64 = a.astype(np.float64)
    want = np.mean(0.5 * a64 * lr * 1.0 / (W * (2 - lr * a64)))
    assert abs(floors[0] / want - 1) < 0.05
