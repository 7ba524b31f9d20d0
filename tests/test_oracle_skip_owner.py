"""Pins of the oracle's owner-elided replica layout.

Section 3 step (4) broadcasts a shard's new values "to all other workers": the owner of a shard needs no
replica of it. In the elided layout worker i's array holds the bucket without the packets worker i owns.
What fixes it: it is the default layout with those packets deleted — every element a worker does not own is
bit-identical to the default run, the owner's own packets never add to its drift (they are exactly fresh in
the default run), and masks, counts, parameters and moments do not depend on the layout at all.
"""
import numpy as np
import pytest

from oracle import oracle as O


def _grads(rng, W, n, dtype):
    g = (rng.standard_normal((W, n)) * 1e-2).astype(np.float32)
    if dtype == O.BF16:
        return [O.cast_wire(x, O.BF16) for x in g]
    return [x.copy() for x in g]


def _pair(W, n, P, p, opt, gd, rd, *, k0=0, n_slab=None, n_total=None, flags=0, seed=5):
    rng = np.random.default_rng(seed)
    n_total = n if n_total is None else n_total
    n_slab = n if n_slab is None else n_slab
    th = (rng.standard_normal(n_slab) * 0.02).astype(np.float32)
    kw = dict(W=W, n=n_total, packet_elems=P, p_grad=p, p_param=p, seed=seed, grad_dtype=gd, replica_dtype=rd,
              optimizer=opt, theta0=th, lr=1e-2, k0=k0, n_slab=n_slab)
    return O.Oracle(flags=flags, **kw), O.Oracle(flags=flags | O.REPLICA_SKIP_OWNER, **kw), rng


CASES = [
    # W, n, P, p, optimizer, grad dtype, replica dtype
    (4, 64 * 13 + 5, 64, 0.3, O.ADAM, O.BF16, O.BF16),      # ragged last packet, last shard shorter
    (8, 16 * 5, 16, 0.4, O.SGD, O.F32, O.F32),              # fewer packets than workers: empty shards
    (1, 100, 8, 0.5, O.SGD, O.F32, O.BF16),                 # one worker: its array is empty
    (3, 8 * 300, 8, 0.6, O.ADAM, O.BF16, O.F32),
    (64, 8 * 64 * 3, 8, 0.2, O.SGD, O.BF16, O.BF16),
]


@pytest.mark.parametrize("W,n,P,p,opt,gd,rd", CASES)
def test_elided_layout_is_the_default_layout_with_the_owners_packets_deleted(W, n, P, p, opt, gd, rd):
    full, elided, rng = _pair(W, n, P, p, opt, gd, rd)
    K = (n + P - 1) // P
    pps = (K + W - 1) // W
    for i in range(W):
        # the array's length, from the shard map written out here on its own
        lo, hi = min(K, i * pps), min(K, (i + 1) * pps)
        own = min(n, hi * P) - min(n, lo * P)
        assert elided.replicas[i].shape == (n - own,)
    for t in range(1, 9):
        g = _grads(rng, W, n, gd)
        a, b = full.step(t, g), elided.step(t, g)
        for key in ("count", "recv_bits", "stale_bits", "ghat"):
            assert np.array_equal(a[key], b[key]), key
        assert np.array_equal(full.master, elided.master)
        assert np.array_equal(full.m, elided.m) and np.array_equal(full.v, elided.v)
        # drift sums are identical: in the default run the owner's own packets are fresh, term exactly 0
        assert np.array_equal(a["sumsq"], b["sumsq"])
        assert np.array_equal(full.drift_sumsq(), elided.drift_sumsq())
        for i in range(W):
            lo, hi = min(n, min(K, i * pps) * P), min(n, min(K, (i + 1) * pps) * P)
            want = np.concatenate([full.replicas[i][:lo], full.replicas[i][hi:]])
            assert np.array_equal(elided.replicas[i], want), f"replica {i} step {t}"
            # and in the default run the owner's own range is always the wire value of the master
            assert np.array_equal(full.replicas[i][lo:hi], O.cast_wire(full.master[lo:hi].astype(np.float32), rd))
    if p > 0 and W > 1:
        assert a["sumsq"].max() > 0


def test_elided_slab_of_a_bucket_equals_the_same_packets_of_the_whole_bucket():
    """A slab in the middle of a bucket (packet ranges, slab-by-slab checks): the arrays hold the slab's
    packets minus the owner's, whatever the slab's position relative to the shard boundaries."""
    W, P, K, p = 5, 16, 23, 0.35
    n = K * P - 3
    whole_f, whole_e, rng = _pair(W, n, P, p, O.ADAM, O.BF16, O.BF16)
    k0, k1 = 3, 17                                  # crosses shard boundaries at packets 5, 10, 15
    e0, e1 = k0 * P, k1 * P
    th = whole_f.master[e0:e1].astype(np.float32).copy()
    slab = O.Oracle(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=5, grad_dtype=O.BF16, replica_dtype=O.BF16,
                    optimizer=O.ADAM, theta0=th, lr=1e-2, k0=k0, n_slab=e1 - e0, flags=O.REPLICA_SKIP_OWNER)
    pps = (K + W - 1) // W
    for t in range(1, 7):
        g = _grads(rng, W, n, O.BF16)
        whole_f.step(t, g)
        r = slab.step(t, [x[e0:e1] for x in g])
        for i in range(W):
            keep = (np.arange(e0, e1) // P) // pps != i
            assert np.array_equal(slab.replicas[i], whole_f.replicas[i][e0:e1][keep])
        assert np.array_equal(slab.master, whole_f.master[e0:e1])
    assert r["sumsq"].max() > 0


def test_elided_pairwise_sums_leave_out_the_owner_on_its_own_packets():
    W, n, P, p = 4, 32 * 12, 32, 0.4
    full, elided, rng = _pair(W, n, P, p, O.SGD, O.F32, O.F32)
    for t in range(1, 6):
        g = _grads(rng, W, n, O.F32)
        full.step(t, g)
        elided.step(t, g)
    K = n // P
    pps = (K + W - 1) // W
    owner = (np.arange(n) // P) // pps
    want = np.zeros((W, W))
    for i in range(W):
        for k in range(W):
            both = (owner != i) & (owner != k)          # elements of which neither of the two is the owner
            d = full.replicas[i][both].astype(np.float64) - full.replicas[k][both].astype(np.float64)
            want[i, k] = np.sum(d * d)
    got = elided.pairwise_sumsq()
    assert np.allclose(got, want, rtol=1e-12, atol=0) and got.max() > 0


def test_closed_loop_gradients_need_the_full_layout():
    _, elided, rng = _pair(2, 64, 8, 0.1, O.SGD, O.F32, O.F32)
    with pytest.raises(ValueError):
        elided.closed_loop_grads(np.ones(64, np.float32), np.zeros(64, np.float32), _grads(rng, 2, 64, O.F32))
