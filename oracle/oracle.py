"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module. It compiles ``lossy_oracle.c`` with gcc (twice: the fp32 contract build
and the fp64 build) and exposes the functions on numpy arrays. bf16 data is
carried as ``uint16`` bit patterns.

The class mirrors one simulated run of the paper's Section 3 iteration:
state = (master, m, v, W replicas, per-replica packet ages), advanced by
``step(t, grads)``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "lossy_oracle.c")
_LIB32 = os.path.join(_DIR, "liblossy_oracle.so")
_LIB64 = os.path.join(_DIR, "liblossy_oracle64.so")
_lock = threading.Lock()
_libs: dict = {}

F32, BF16 = 0, 1
SGD, ADAM = 0, 1
SELF_LOSSLESS, ZERO_SKIP, REPLICA_SKIP_OWNER = 1, 2, 8


class OracleConfig(C.Structure):
    _fields_ = [
        ("W", C.c_uint32), ("packet_elems", C.c_uint32), ("n", C.c_uint64),
        ("packet_base", C.c_uint64), ("p_grad", C.c_double), ("p_param", C.c_double),
        ("seed", C.c_uint64), ("grad_dtype", C.c_uint32), ("replica_dtype", C.c_uint32),
        ("optimizer", C.c_uint32), ("flags", C.c_uint32),
        ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
    ]


def build(force: bool = False) -> None:
    """Compile both oracle libraries next to the source (no-op when up to date)."""
    with _lock:
        for out, extra in ((_LIB32, []), (_LIB64, ["-DORACLE_F64"])):
            if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
                continue
            cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-fPIC", "-shared",
                   *extra, "-o", out + ".tmp", _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(out + ".tmp", out)


def _lib(f64: bool):
    key = "f64" if f64 else "f32"
    if key not in _libs:
        build()
        lib = C.CDLL(_LIB64 if f64 else _LIB32)
        pre = "oracle64_" if f64 else "oracle_"
        h = getattr(lib, pre + "hash_u32")
        h.restype = C.c_uint32
        h.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
        mx = getattr(lib, pre + "mix64")
        mx.restype = C.c_uint64
        mx.argtypes = [C.c_uint64]
        t = getattr(lib, pre + "threshold")
        t.restype = C.c_uint32
        t.argtypes = [C.c_double]
        d = getattr(lib, pre + "delivered")
        d.restype = C.c_int
        d.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_double]
        b = getattr(lib, pre + "f32_to_bf16")
        b.restype = C.c_uint16
        b.argtypes = [C.c_float]
        o = getattr(lib, pre + "owner")
        o.restype = C.c_uint32
        o.argtypes = [C.POINTER(OracleConfig), C.c_uint64]
        s = getattr(lib, pre + "step")
        s.restype = C.c_int
        s.argtypes = [C.POINTER(OracleConfig), C.c_uint64, C.c_uint64, C.c_uint64] + [C.c_void_p] * 18
        ds = getattr(lib, pre + "drift_sumsq")
        ds.restype = C.c_int
        ds.argtypes = [C.POINTER(OracleConfig), C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p]
        mk = getattr(lib, pre + "masks")
        mk.restype = C.c_int
        mk.argtypes = [C.POINTER(OracleConfig), C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p]
        sq = getattr(lib, pre + "packet_sqnorms")
        sq.restype = C.c_int
        sq.argtypes = [C.POINTER(OracleConfig), C.c_uint64, C.c_void_p, C.c_void_p]
        pw = getattr(lib, pre + "pairwise_sumsq")
        pw.restype = C.c_int
        pw.argtypes = [C.POINTER(OracleConfig), C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        cl = getattr(lib, pre + "closed_loop_grads")
        cl.restype = C.c_int
        cl.argtypes = [C.POINTER(OracleConfig), C.c_uint64] + [C.c_void_p] * 5
        _libs[key] = (lib, pre)
    return _libs[key]


def hash_u32(seed: int, step: int, src: int, dst: int, packet: int) -> int:
    lib, pre = _lib(False)
    return getattr(lib, pre + "hash_u32")(seed, step, src, dst, packet)


def mix64(z: int) -> int:
    lib, pre = _lib(False)
    return getattr(lib, pre + "mix64")(z)


def threshold(p: float) -> int:
    lib, pre = _lib(False)
    return getattr(lib, pre + "threshold")(p)


def delivered(seed: int, step: int, src: int, dst: int, packet: int, p: float) -> int:
    lib, pre = _lib(False)
    return getattr(lib, pre + "delivered")(seed, step, src, dst, packet, p)


def f32_to_bf16(x: float) -> int:
    lib, pre = _lib(False)
    return getattr(lib, pre + "f32_to_bf16")(x)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _ptr_table(arrs):
    tab = (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    return tab


class Oracle:
    """State of one simulated run over a slab of a bucket.

    ``n`` is the size of the whole bucket (it fixes the packet count K and the
    shard map); the slab starts at packet ``k0`` and holds ``n_slab`` elements
    (default: the whole bucket). ``theta0`` is the fp32 initial master slab; every
    replica starts as cast(theta0) (synchronised start, zero drift).
    """

    def __init__(self, *, W, n, packet_elems, p_grad, p_param, seed, grad_dtype, replica_dtype,
                 optimizer, theta0, lr, beta1=0.9, beta2=0.95, eps=1e-8, flags=0, packet_base=0,
                 k0=0, n_slab=None, f64=False, track_age=False, alg1=False, burst=None):
        self.cfg = OracleConfig(W, packet_elems, n, packet_base, p_grad, p_param, seed, grad_dtype,
                                replica_dtype, optimizer, flags, lr, beta1, beta2, eps)
        self.W, self.P, self.n, self.k0 = W, packet_elems, n, k0
        self.n_slab = n if n_slab is None else n_slab
        self.packets = (self.n_slab + packet_elems - 1) // packet_elems
        self.f64 = f64
        self.real = np.float64 if f64 else np.float32
        self.lib, self.pre = _lib(f64)
        theta0 = np.ascontiguousarray(theta0, dtype=np.float32)
        assert theta0.shape == (self.n_slab,)
        self.master = theta0.astype(self.real)
        self.m = np.zeros(self.n_slab, self.real)
        self.v = np.zeros(self.n_slab, self.real)
        wire = cast_wire(theta0, replica_dtype)
        self.elided = bool(flags & REPLICA_SKIP_OWNER)
        # owner-elided layout: worker i's array holds the slab without the packets it owns, back to back
        self.replicas = [wire[self.kept(i)].copy() if self.elided else wire.copy() for i in range(W)]
        self.age = [np.zeros(self.packets, np.uint32) for _ in range(W)] if track_age else None
        # Algorithm 1's gradient half keeps the last surviving aggregate per element ("g_prev"), zero at start
        self.ghat_prev = np.zeros(self.n_slab, self.real) if alg1 else None
        # bursty loss: (P(good->bad), P(bad->good)) and the link states [2][packets], all good at start
        self.burst = None if burst is None else np.array(burst, dtype=np.float64)
        self.burst_state = np.zeros((2, self.packets), np.uint64) if burst is not None else None
        self.grad_dtype, self.replica_dtype = grad_dtype, replica_dtype

    def owner(self, k: int) -> int:
        return getattr(self.lib, self.pre + "owner")(C.byref(self.cfg), k)

    def kept(self, i: int) -> np.ndarray:
        """Boolean mask over the slab's elements: True where worker i is NOT the owner (what its array
        holds in the owner-elided layout)."""
        K = (self.n + self.P - 1) // self.P
        pps = (K + self.W - 1) // self.W
        owner_of_elem = (self.k0 + np.arange(self.n_slab, dtype=np.int64) // self.P) // pps
        return owner_of_elem != i

    def set_lr(self, lr: float) -> None:
        self.cfg.lr = lr

    def masks(self, t, k0=0, packets=None):
        """(recv_bits, stale_bits, count) of `packets` packets from bucket packet k0 at step t (independent loss)."""
        K = (self.n + self.P - 1) // self.P
        packets = K - k0 if packets is None else packets
        recv = np.zeros(packets, np.uint64)
        stale = np.zeros(packets, np.uint64)
        count = np.zeros(packets, np.uint8)
        rc = getattr(self.lib, self.pre + "masks")(C.byref(self.cfg), t, k0, packets, _ptr(recv), _ptr(stale),
                                                   _ptr(count))
        if rc != 0:
            raise ValueError("oracle_masks rejected its arguments")
        return recv, stale, count

    def packet_sqnorms(self, grads):
        """[W][packets] squared norms of the gradient pieces, in double."""
        gd = np.uint16 if self.grad_dtype == BF16 else np.float32
        grads = [np.ascontiguousarray(g, dtype=gd) for g in grads]
        out = np.zeros((self.W, self.packets), np.float64)
        gt = _ptr_table(grads)
        rc = getattr(self.lib, self.pre + "packet_sqnorms")(C.byref(self.cfg), self.n_slab, C.cast(gt, C.c_void_p),
                                                            _ptr(out))
        if rc != 0:
            raise ValueError("oracle_packet_sqnorms rejected its arguments")
        return out

    def step(self, t, grads, *, recv_force=None, stale_force=None, want_ghat=True, reliable=None):
        """Advance one iteration; returns a dict of ghat, count, recv_bits, stale_bits, sumsq, norms."""
        gd = np.uint16 if self.grad_dtype == BF16 else np.float32
        grads = [np.ascontiguousarray(g, dtype=gd) for g in grads]
        assert len(grads) == self.W and all(g.shape == (self.n_slab,) for g in grads)
        ghat = np.zeros(self.n_slab, self.real) if want_ghat else None
        count = np.zeros(self.packets, np.uint8)
        recv = np.zeros(self.packets, np.uint64)
        stale = np.zeros(self.packets, np.uint64)
        sumsq = np.zeros(self.W, np.float64)
        gt, rt = _ptr_table(grads), _ptr_table(self.replicas)
        at = _ptr_table(self.age) if self.age is not None else None
        if recv_force is not None:
            recv_force = np.ascontiguousarray(recv_force, dtype=np.uint64)
        if stale_force is not None:
            stale_force = np.ascontiguousarray(stale_force, dtype=np.uint64)
        burst_out = np.zeros_like(self.burst_state) if self.burst is not None else None
        if reliable is not None:        # [2][packets]: reliable gradient links, reliable broadcast links
            reliable = np.ascontiguousarray(reliable, dtype=np.uint64)
            assert reliable.shape == (2, self.packets)
        rc = getattr(self.lib, self.pre + "step")(
            C.byref(self.cfg), t, self.k0, self.n_slab, C.cast(gt, C.c_void_p), _ptr(self.master),
            _ptr(self.m), _ptr(self.v), C.cast(rt, C.c_void_p), _ptr(self.ghat_prev), _ptr(self.burst),
            _ptr(self.burst_state), _ptr(burst_out), _ptr(reliable), _ptr(recv_force), _ptr(stale_force),
            _ptr(ghat), _ptr(count), _ptr(recv), _ptr(stale),
            C.cast(at, C.c_void_p) if at is not None else None, _ptr(sumsq))
        if rc != 0:
            raise ValueError("oracle_step rejected its arguments")
        if self.burst is not None:
            self.burst_state = burst_out
        return {"ghat": ghat, "count": count, "recv_bits": recv, "stale_bits": stale,
                "sumsq": sumsq, "norms": np.sqrt(sumsq)}

    def closed_loop_grads(self, curv, target, noise):
        """Gradients of the diagonal quadratic evaluated at each worker's own replica, plus its noise."""
        gd = np.uint16 if self.grad_dtype == BF16 else np.float32
        curv = np.ascontiguousarray(curv, dtype=np.float32)
        target = np.ascontiguousarray(target, dtype=np.float32)
        noise = [np.ascontiguousarray(x, dtype=gd) for x in noise]
        out = [np.zeros(self.n_slab, gd) for _ in range(self.W)]
        nt, rt, ot = _ptr_table(noise), _ptr_table(self.replicas), _ptr_table(out)
        rc = getattr(self.lib, self.pre + "closed_loop_grads")(
            C.byref(self.cfg), self.n_slab, _ptr(curv), _ptr(target), C.cast(nt, C.c_void_p),
            C.cast(rt, C.c_void_p), C.cast(ot, C.c_void_p))
        if rc != 0:
            raise ValueError("oracle_closed_loop_grads rejected its arguments")
        return out

    def pairwise_sumsq(self):
        """W x W matrix of sum_e (replica_i[e] - replica_k[e])^2, in double (the theorem's pairwise drift)."""
        d2 = np.zeros((self.W, self.W), np.float64)
        rt = _ptr_table(self.replicas)
        rc = getattr(self.lib, self.pre + "pairwise_sumsq")(C.byref(self.cfg), self.k0, self.n_slab,
                                                            C.cast(rt, C.c_void_p), _ptr(d2))
        if rc != 0:
            raise ValueError("oracle_pairwise_sumsq rejected its arguments")
        return d2

    def drift_sumsq(self):
        """Standalone drift: sum_e (replica_i[e] - cast(master[e]))^2 per replica, in double."""
        sumsq = np.zeros(self.W, np.float64)
        rt = _ptr_table(self.replicas)
        rc = getattr(self.lib, self.pre + "drift_sumsq")(
            C.byref(self.cfg), self.k0, self.n_slab, _ptr(self.master), C.cast(rt, C.c_void_p), _ptr(sumsq))
        if rc != 0:
            raise ValueError("oracle_drift_sumsq rejected its arguments")
        return sumsq


def cast_wire(theta_f32: np.ndarray, replica_dtype: int) -> np.ndarray:
    """The value a broadcast puts on the wire: fp32 itself, or its RNE bf16 bit pattern."""
    theta_f32 = np.ascontiguousarray(theta_f32, dtype=np.float32)
    if replica_dtype == F32:
        return theta_f32.copy()
    lib, pre = _lib(False)
    f = getattr(lib, pre + "f32_to_bf16")
    if theta_f32.size <= 4096:
        return np.array([f(float(x)) for x in theta_f32], dtype=np.uint16)
    # same rounding written on integers (checked against the scalar routine in the tests)
    u = theta_f32.view(np.uint32).astype(np.uint64)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    r[nan] = ((u[nan] >> 16) | 0x40).astype(np.uint16)
    return r


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)
