"""Shared driver of the GPU parity tests: runs the CUDA path (through the C ABI binding) and the
CPU oracle on the same seeded inputs and compares them element by element.

Bar (written here once): masks, received counts and stale sets bit-exact; every float within
max relative error 1e-5 of the oracle (fp32 accumulation in fixed worker order on both sides).
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2507_07114_b200 as L
import workload
from oracle import oracle as O

REL_TOL = 1e-5
TINY = 1e-30


def tdtype(name):
    return torch.bfloat16 if name == "bf16" else torch.float32


def odtype(name):
    return O.BF16 if name == "bf16" else O.F32


def to_np(t: torch.Tensor) -> np.ndarray:
    """Tensor -> numpy (bf16 as uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def as_f64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:
        return O.bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def assert_rel(got, want, what, tol=REL_TOL):
    got, want = as_f64(np.asarray(got)), as_f64(np.asarray(want))
    assert got.shape == want.shape, what
    if got.size == 0:
        return
    got, want = got.ravel(), want.ravel()
    err = np.abs(got - want) / np.maximum(np.abs(want), TINY)
    bad = int(np.argmax(err))
    assert err[bad] <= tol, f"{what}: rel err {err[bad]:.3e} at {bad} (got {got[bad]!r}, want {want[bad]!r})"


def assert_same(got, want, what):
    got, want = np.asarray(got), np.asarray(want)
    assert got.shape == want.shape, what
    if not np.array_equal(got, want):
        bad = int(np.flatnonzero(got != want)[0])
        raise AssertionError(f"{what}: first mismatch at {bad} (got {got[bad]!r}, want {want[bad]!r}); "
                             f"{int((got != want).sum())} of {got.size} differ")


class GpuRun:
    """State of one simulated run on the GPU, advanced through the C ABI."""

    def __init__(self, w: workload.Workload, *, flags=0, p_grad=None, p_param=None, theta0=None, device="cuda",
                 alg1=False, burst=None, shard_packet0=0, bucket_packets=0):
        self.w, self.dev, self.alg1, self.burst = w, device, alg1, burst
        rng_kw = {"shard_packet0": shard_packet0, "bucket_packets": bucket_packets} if bucket_packets else {}
        self.ctx = L.lossy_init(W=w.W, n=w.n, packet_elems=w.packet_elems,
                                p_grad=w.p if p_grad is None else p_grad,
                                p_param=w.p if p_param is None else p_param, seed=w.seed,
                                grad_dtype=tdtype(w.grad_dtype), replica_dtype=tdtype(w.replica_dtype),
                                optimizer=w.optimizer, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                                flags=flags, packet_base=w.packet_base, **rng_kw)
        n, W, K = w.n, w.W, w.K
        th = workload.theta0_slab(w, 0, n, device) if theta0 is None else theta0.to(device)
        self.master = th.clone()
        self.m = torch.zeros(n, dtype=torch.float32, device=device)
        self.v = torch.zeros(n, dtype=torch.float32, device=device)
        self.elided = bool(flags & L.LOSSY_REPLICA_SKIP_OWNER)
        wire = self.master.to(tdtype(w.replica_dtype))
        if self.elided:
            # owner-elided layout: replica i is the bucket without the packets worker i owns
            Kb = bucket_packets if bucket_packets else K
            pps = (Kb + W - 1) // W
            owner = (shard_packet0 + torch.arange(n, device=device) // w.packet_elems) // pps
            self.replicas = [wire[owner != i].clone() for i in range(W)]
            for i in range(W):
                assert self.replicas[i].numel() == L.lossy_replica_elems(self.ctx, i)
        else:
            self.replicas = [wire.clone() for _ in range(W)]
        self.ghat = torch.zeros(n, dtype=torch.float32, device=device)
        self.ghat_prev = torch.zeros(n, dtype=torch.float32, device=device) if alg1 else None
        self.count = torch.zeros(K, dtype=torch.uint8, device=device)
        self.recv = torch.zeros(K, dtype=torch.int64, device=device)
        self.stale = torch.zeros(K, dtype=torch.int64, device=device)
        self.norms = torch.zeros(W, dtype=torch.float32, device=device)
        self.sumsq = torch.zeros(W, dtype=torch.float64, device=device)
        self.burst_state = None
        if burst is not None:
            self.burst_state = torch.zeros(4 * K, dtype=torch.int64, device=device)   # [2 buffers][2 rows][K]
            L.lossy_set_bursty(self.ctx, burst[0], burst[1], self.burst_state)

    def burst_rows(self, t):
        """Link states after step t as numpy [2][K] (row 0 gradient links, row 1 broadcast links)."""
        K = self.w.K
        buf = self.burst_state.view(2, 2, K)[t & 1]
        return to_np(buf).view(np.uint64)

    def close(self):
        if self.ctx is not None:
            L.lossy_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step_fused(self, t, grads, outputs=True):
        adam = self.w.optimizer == "adam"
        self.sumsq.zero_()
        if self.alg1:
            L.lossy_fused_step_alg1(self.ctx, t, grads, self.ghat_prev, self.master, self.m if adam else None,
                                    self.v if adam else None, self.replicas, self.ghat, self.count, self.recv,
                                    self.stale, self.norms, self.sumsq)
        elif outputs:
            L.lossy_fused_step(self.ctx, t, grads, self.master, self.m if adam else None, self.v if adam else None,
                               self.replicas, self.ghat, self.count, self.recv, self.stale, self.norms, self.sumsq)
        else:
            L.lossy_fused_step(self.ctx, t, grads, self.master, self.m if adam else None, self.v if adam else None,
                               self.replicas, norms=self.norms)

    def step_unfused(self, t, grads):
        adam = self.w.optimizer == "adam"
        self.sumsq.zero_()
        if self.alg1:
            L.lossy_aggregate_alg1(self.ctx, t, grads, self.ghat_prev, self.ghat, self.count, self.recv)
        else:
            L.lossy_aggregate(self.ctx, t, grads, self.ghat, self.count, self.recv)
        L.lossy_step(self.ctx, t, self.ghat, self.count, self.master, self.m if adam else None,
                     self.v if adam else None)
        L.lossy_broadcast(self.ctx, t, self.master, self.replicas, self.stale)
        L.drift_norms(self.ctx, self.master, self.replicas, self.norms, self.sumsq)

    def outputs(self):
        torch.cuda.synchronize()
        return {"ghat": to_np(self.ghat), "count": to_np(self.count),
                "recv_bits": to_np(self.recv).view(np.uint64), "stale_bits": to_np(self.stale).view(np.uint64),
                "norms": to_np(self.norms).astype(np.float64), "sumsq": to_np(self.sumsq)}


def make_oracle(w: workload.Workload, *, flags=0, p_grad=None, p_param=None, theta0=None, k0=0, n_slab=None,
                e0=0, alg1=False, burst=None):
    n_slab = w.n - e0 if n_slab is None else n_slab
    th = workload.theta0_slab(w, e0, e0 + n_slab) if theta0 is None else theta0
    return O.Oracle(W=w.W, n=w.n, packet_elems=w.packet_elems, p_grad=w.p if p_grad is None else p_grad,
                    p_param=w.p if p_param is None else p_param, seed=w.seed, grad_dtype=odtype(w.grad_dtype),
                    replica_dtype=odtype(w.replica_dtype), optimizer=O.ADAM if w.optimizer == "adam" else O.SGD,
                    theta0=to_np(th), lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, flags=flags,
                    packet_base=w.packet_base, k0=k0, n_slab=n_slab, alg1=alg1, burst=burst)


def compare_state(gpu: GpuRun, orc, what, e0=0, e1=None):
    whole = e0 == 0 and e1 is None
    e1 = gpu.w.n if e1 is None else e1
    assert_rel(to_np(gpu.master[e0:e1]), orc.master, f"{what} master")
    if gpu.w.optimizer == "adam":
        assert_rel(to_np(gpu.m[e0:e1]), orc.m, f"{what} m")
        assert_rel(to_np(gpu.v[e0:e1]), orc.v, f"{what} v")
    for i in range(gpu.w.W):
        if gpu.elided and not whole:
            # a slab [e0, e1) of an owner-elided replica: the slab's elements that worker i does not own, which
            # start where the elements in front of the slab that it does not own end
            P, K = gpu.w.packet_elems, gpu.w.K
            pps = (K + gpu.w.W - 1) // gpu.w.W
            lo, hi = min(gpu.w.n, i * pps * P), min(gpu.w.n, (i + 1) * pps * P)      # worker i's own elements
            own_before = max(0, min(hi, e0) - lo)
            own_inside = max(0, min(hi, e1) - max(lo, e0))
            a = e0 - own_before
            got = gpu.replicas[i][a:a + (e1 - e0) - own_inside]
        else:
            got = gpu.replicas[i] if gpu.elided else gpu.replicas[i][e0:e1]
        assert_rel(to_np(got), orc.replicas[i], f"{what} replica {i}")


def compare_outputs(out, ref, what, with_ghat=True):
    assert_same(out["count"], ref["count"], f"{what} count")
    assert_same(out["recv_bits"], ref["recv_bits"], f"{what} recv_bits")
    assert_same(out["stale_bits"], ref["stale_bits"], f"{what} stale_bits")
    if with_ghat:
        assert_rel(out["ghat"], ref["ghat"], f"{what} ghat")
    assert_rel(out["norms"], ref["norms"], f"{what} norms")
    assert_rel(out["sumsq"], ref["sumsq"], f"{what} sumsq", tol=2 * REL_TOL)


def run_parity(w: workload.Workload, steps, *, fused=True, flags=0, p_grad=None, p_param=None, exact=True,
               alg1=False, burst=None):
    """Element-by-element parity of a whole (small) run. Returns the GpuRun for further checks."""
    gpu = GpuRun(w, flags=flags, p_grad=p_grad, p_param=p_param, alg1=alg1, burst=burst)
    orc = make_oracle(w, flags=flags & ~(L.LOSSY_REGISTER_PATH | L.LOSSY_PACKED_BULK | L.LOSSY_GATHER_PATH), p_grad=p_grad, p_param=p_param, alg1=alg1,
                      burst=burst)                                                  # those bits only pick the kernel
    for t in range(1, steps + 1):
        gs = [workload.grad_slab(w, t, i, 0, w.n) for i in range(w.W)]
        gd = [g.cuda() for g in gs]
        (gpu.step_fused if fused else gpu.step_unfused)(t, gd)
        ref = orc.step(t, [to_np(g) for g in gs])
        compare_outputs(gpu.outputs(), ref, f"{w.name} step {t}")
        compare_state(gpu, orc, f"{w.name} step {t}")
        if alg1:
            assert_same(to_np(gpu.ghat_prev), orc.ghat_prev, f"{w.name} step {t} ghat_prev")
        if burst is not None:
            assert_same(gpu.burst_rows(t), orc.burst_state, f"{w.name} step {t} link states")
    L.lossy_device_status(gpu.ctx)      # raises if a bounded wait inside a kernel gave up
    if exact:
        # fixed order + separately rounded operations on both sides: the state is in fact bit-identical
        assert_same(to_np(gpu.master), orc.master, f"{w.name} master bits")
        for i in range(w.W):
            assert_same(to_np(gpu.replicas[i]), orc.replicas[i], f"{w.name} replica {i} bits")
    return gpu, orc
