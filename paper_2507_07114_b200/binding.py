"""Thin ctypes binding of the C ABI in include/lossy.h (argument marshalling only).

Every function has the name of the C entry point it calls; tensors are passed as
raw device pointers and the current torch CUDA stream as the stream argument. All
arithmetic runs in the CUDA library. There is no fallback: if the shared library
is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

LOSSY_OK, LOSSY_EINVAL, LOSSY_ENOMEM, LOSSY_ECUDA, LOSSY_EDEVICE, LOSSY_ELIMIT, LOSSY_EDEVCHECK = 0, 1, 2, 3, 4, 5, 6
LOSSY_F32, LOSSY_BF16 = 0, 1
LOSSY_SGD, LOSSY_ADAM = 0, 1
LOSSY_SELF_LOSSLESS, LOSSY_ZERO_SKIP, LOSSY_REGISTER_PATH, LOSSY_REPLICA_SKIP_OWNER, LOSSY_PACKED_BULK = 1, 2, 4, 8, 16
LOSSY_GATHER_PATH = 32

EXPORTS = [
    "lossy_init", "lossy_destroy", "lossy_set_lr", "lossy_set_bursty", "lossy_set_reliable", "lossy_packet_sqnorms", "lossy_aggregate", "lossy_step", "lossy_broadcast",
    "drift_norms", "drift_pairwise", "drift_norms_static", "lossy_fused_step", "lossy_aggregate_alg1", "lossy_fused_step_alg1", "lossy_fused_step_host", "lossy_mask", "lossy_hash_u32",
    "lossy_mask_grid", "lossy_closed_loop_grads", "lossy_device_status", "lossy_last_error", "lossy_num_packets", "lossy_kernel_launches",
    "lossy_describe_plan", "lossy_replica_elems", "lossy_reset_status", "lossy_selftest_wait_expiry",
    "lossy_has_device_checks", "lossy_selftest_shrink_checks",
]


class lossy_config(C.Structure):
    _fields_ = [
        ("W", C.c_uint32), ("packet_elems", C.c_uint32), ("n", C.c_uint64), ("packet_base", C.c_uint64),
        ("p_grad", C.c_double), ("p_param", C.c_double), ("seed", C.c_uint64),
        ("grad_dtype", C.c_uint32), ("replica_dtype", C.c_uint32), ("optimizer", C.c_uint32),
        ("flags", C.c_uint32), ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
        ("eps", C.c_float), ("shard_packet0", C.c_uint64), ("bucket_packets", C.c_uint64),
    ]


class LossyError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"lossy error {code}: {msg}")
        self.code = code


_lib = None


def default_library_path() -> str:
    """The library this process binds to: the debug build (index checks in every kernel of the step path) when the
    environment says LOSSY_B200_CHECKED=1, else the normal one. Read once, at the first call."""
    return _build.CHECK_LIB_PATH if os.environ.get("LOSSY_B200_CHECKED") == "1" else _build.LIB_PATH


def load_library(path: str | None = None) -> C.CDLL:
    """dlopen liblossy_b200.so (built in-tree by paper_2507_07114_b200.build) and declare its signatures."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    default = default_library_path()
    path = path or default
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: run paper_2507_07114_b200.build.build() (needs nvcc); "
                                "there is no CPU fallback")
    lib = C.CDLL(path)
    vp, u64, u32 = C.c_void_p, C.c_uint64, C.c_uint32
    lib.lossy_init.restype = C.c_int
    lib.lossy_init.argtypes = [C.POINTER(lossy_config), C.POINTER(vp)]
    lib.lossy_destroy.restype = None
    lib.lossy_destroy.argtypes = [vp]
    lib.lossy_set_lr.restype = C.c_int
    lib.lossy_set_lr.argtypes = [vp, C.c_float]
    lib.lossy_set_bursty.restype = C.c_int
    lib.lossy_set_bursty.argtypes = [vp, C.c_double, C.c_double, vp]
    lib.lossy_set_reliable.restype = C.c_int
    lib.lossy_set_reliable.argtypes = [vp, vp]
    lib.lossy_packet_sqnorms.restype = C.c_int
    lib.lossy_packet_sqnorms.argtypes = [vp, vp, vp, vp]
    lib.lossy_aggregate.restype = C.c_int
    lib.lossy_aggregate.argtypes = [vp, u64, vp, vp, vp, vp, vp]
    lib.lossy_step.restype = C.c_int
    lib.lossy_step.argtypes = [vp, u64, vp, vp, vp, vp, vp, vp]
    lib.lossy_broadcast.restype = C.c_int
    lib.lossy_broadcast.argtypes = [vp, u64, vp, vp, vp, vp]
    lib.drift_norms.restype = C.c_int
    lib.drift_norms.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.drift_pairwise.restype = C.c_int
    lib.drift_pairwise.argtypes = [vp, vp, vp, vp]
    lib.drift_norms_static.restype = C.c_int
    lib.drift_norms_static.argtypes = [C.POINTER(lossy_config), vp, vp, vp, vp, vp]
    lib.lossy_fused_step.restype = C.c_int
    lib.lossy_fused_step.argtypes = [vp, u64] + [vp] * 12
    lib.lossy_aggregate_alg1.restype = C.c_int
    lib.lossy_aggregate_alg1.argtypes = [vp, u64, vp, vp, vp, vp, vp, vp]
    lib.lossy_fused_step_alg1.restype = C.c_int
    lib.lossy_fused_step_alg1.argtypes = [vp, u64] + [vp] * 13
    lib.lossy_fused_step_host.restype = C.c_int
    lib.lossy_fused_step_host.argtypes = [vp, u64] + [vp] * 9
    lib.lossy_mask.restype = C.c_int
    lib.lossy_mask.argtypes = [vp, u64, u32, u32, u64, C.c_int]
    lib.lossy_hash_u32.restype = u32
    lib.lossy_hash_u32.argtypes = [u64, u64, u32, u32, u64]
    lib.lossy_mask_grid.restype = C.c_int
    lib.lossy_mask_grid.argtypes = [vp, u64, vp, vp, vp, u64, C.c_int, vp, vp]
    lib.lossy_closed_loop_grads.restype = C.c_int
    lib.lossy_closed_loop_grads.argtypes = [vp] * 7
    lib.lossy_device_status.restype = C.c_int
    lib.lossy_device_status.argtypes = [vp, vp]
    lib.lossy_last_error.restype = C.c_char_p
    lib.lossy_last_error.argtypes = [vp]
    lib.lossy_num_packets.restype = u64
    lib.lossy_num_packets.argtypes = [vp]
    lib.lossy_kernel_launches.restype = u64
    lib.lossy_kernel_launches.argtypes = [vp]
    lib.lossy_replica_elems.restype = u64
    lib.lossy_replica_elems.argtypes = [vp, u32]
    lib.lossy_reset_status.restype = C.c_int
    lib.lossy_reset_status.argtypes = [vp, vp]
    lib.lossy_selftest_wait_expiry.restype = C.c_int
    lib.lossy_selftest_wait_expiry.argtypes = [vp, u32, vp]
    lib.lossy_has_device_checks.restype = C.c_int
    lib.lossy_has_device_checks.argtypes = []
    lib.lossy_selftest_shrink_checks.restype = C.c_int
    lib.lossy_selftest_shrink_checks.argtypes = [vp, u64]
    lib.lossy_describe_plan.restype = C.c_int
    lib.lossy_describe_plan.argtypes = [vp, C.c_int, C.c_char_p, C.c_size_t]
    if path == default:
        _lib = lib
    return lib


def _dt(t: torch.dtype) -> int:
    if t == torch.float32:
        return LOSSY_F32
    if t == torch.bfloat16:
        return LOSSY_BF16
    raise TypeError(f"unsupported element type {t}")


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _table(ts):
    return (C.c_void_p * len(ts))(*[None if t is None else t.data_ptr() for t in ts])


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(ctx, rc):
    if rc != LOSSY_OK:
        raise LossyError(rc, load_library().lossy_last_error(ctx).decode())


def lossy_init(*, W, n, packet_elems, p_grad, p_param, seed, grad_dtype, replica_dtype, optimizer, lr,
               beta1=0.9, beta2=0.95, eps=1e-8, flags=0, packet_base=0, shard_packet0=0, bucket_packets=0):
    """Create a context on the current CUDA device; returns an opaque handle (free with lossy_destroy)."""
    lib = load_library()
    torch.cuda.init()
    opt = {"sgd": LOSSY_SGD, "adam": LOSSY_ADAM}.get(optimizer, optimizer)
    cfg = lossy_config(W, packet_elems, n, packet_base, p_grad, p_param, seed, _dt(grad_dtype), _dt(replica_dtype),
                       opt, flags, lr, beta1, beta2, eps, shard_packet0, bucket_packets)
    ctx = C.c_void_p()
    with torch.cuda.device(torch.cuda.current_device()):
        rc = lib.lossy_init(C.byref(cfg), C.byref(ctx))
    if rc != LOSSY_OK:
        raise LossyError(rc, "lossy_init rejected the configuration" if rc == LOSSY_EINVAL else "lossy_init failed")
    return ctx


def lossy_destroy(ctx):
    load_library().lossy_destroy(ctx)


def lossy_set_lr(ctx, lr):
    _check(ctx, load_library().lossy_set_lr(ctx, lr))


def lossy_set_bursty(ctx, p_enter_bad, p_leave_bad, state):
    """state: int64/uint64 device tensor of 4*K elements, zeroed before step 1; None = independent loss."""
    _check(ctx, load_library().lossy_set_bursty(ctx, p_enter_bad, p_leave_bad, _p(state)))


def lossy_set_reliable(ctx, reliable):
    """reliable: int64/uint64 device tensor of 2*K elements (row 0 gradient links, row 1 broadcast links) or None."""
    _check(ctx, load_library().lossy_set_reliable(ctx, _p(reliable)))


def lossy_packet_sqnorms(ctx, grads, out):
    _check(ctx, load_library().lossy_packet_sqnorms(ctx, _table(grads), _p(out), _stream()))


def lossy_aggregate(ctx, step, grads, ghat, count=None, recv_bits=None):
    _check(ctx, load_library().lossy_aggregate(ctx, step, _table(grads), _p(ghat), _p(count), _p(recv_bits),
                                               _stream()))


def lossy_step(ctx, step, ghat, count, master, m=None, v=None):
    _check(ctx, load_library().lossy_step(ctx, step, _p(ghat), _p(count), _p(master), _p(m), _p(v), _stream()))


def lossy_broadcast(ctx, step, master, replicas, stale_bits=None):
    _check(ctx, load_library().lossy_broadcast(ctx, step, _p(master), _table(replicas), _p(stale_bits), _stream()))


def drift_norms(ctx, master, replicas, norms=None, sumsq=None):
    _check(ctx, load_library().drift_norms(ctx, _p(master), _table(replicas), _p(norms), _p(sumsq), _stream()))


def drift_pairwise(ctx, replicas, d2):
    """d2: fp64 device tensor of W*W elements, added to (zero it first)."""
    _check(ctx, load_library().drift_pairwise(ctx, _table(replicas), _p(d2), _stream()))


def drift_norms_static(*, W, n, packet_elems, replica_dtype, master, replicas, norms=None, sumsq=None, flags=0,
                       shard_packet0=0, bucket_packets=0):
    """drift_norms for callers that may not allocate device memory (no context; static scratch in the library).

    Raises LossyError with code LOSSY_ELIMIT when a size is beyond the static scratch's limits."""
    cfg = lossy_config(W, packet_elems, n, 0, 0.0, 0.0, 0, LOSSY_F32, _dt(replica_dtype), LOSSY_SGD, flags,
                       0.0, 0.0, 0.0, 0.0, shard_packet0, bucket_packets)
    rc = load_library().drift_norms_static(C.byref(cfg), _p(master), _table(replicas), _p(norms), _p(sumsq),
                                           _stream())
    if rc != LOSSY_OK:
        raise LossyError(rc, "drift_norms_static: " + {LOSSY_EINVAL: "bad argument", LOSSY_ELIMIT:
                         "size beyond the static scratch limits", LOSSY_ECUDA: "CUDA error",
                         LOSSY_ENOMEM: "no device memory left to load the library image"}.get(rc, "error"))


def lossy_fused_step(ctx, step, grads, master, m, v, replicas, ghat=None, count=None, recv_bits=None,
                     stale_bits=None, norms=None, sumsq=None):
    _check(ctx, load_library().lossy_fused_step(ctx, step, _table(grads), _p(master), _p(m), _p(v), _table(replicas),
                                                _p(ghat), _p(count), _p(recv_bits), _p(stale_bits), _p(norms),
                                                _p(sumsq), _stream()))


class lossy_fused_step_prepared:
    """lossy_fused_step (or, with ghat_prev, lossy_fused_step_alg1) with its arguments marshalled once: the pointer
    tables and handles are built here, a call `prepared(step)` is one foreign call. For buckets so small that a
    step is bound by launch overhead (a 40 MB bucket: 19 -> 12 us per step); the tensors are kept alive by this
    object and must not be reallocated while it is used. `stream`: a torch stream whose handle is read once, or
    None to read the current stream at every call."""

    def __init__(self, ctx, grads, master, m, v, replicas, ghat=None, count=None, recv_bits=None, stale_bits=None,
                 norms=None, sumsq=None, ghat_prev=None, stream=None):
        lib = load_library()
        self._ctx, self._keep = ctx, (grads, master, m, v, replicas, ghat, count, recv_bits, stale_bits, norms, sumsq, ghat_prev)
        self._fn = lib.lossy_fused_step if ghat_prev is None else lib.lossy_fused_step_alg1
        head = (_table(grads),) + (() if ghat_prev is None else (_p(ghat_prev),))
        self._args = head + (_p(master), _p(m), _p(v), _table(replicas), _p(ghat), _p(count), _p(recv_bits),
                             _p(stale_bits), _p(norms), _p(sumsq))
        self._stream = None if stream is None else C.c_void_p(stream.cuda_stream)

    def __call__(self, step):
        rc = self._fn(self._ctx, step, *self._args, self._stream if self._stream is not None else _stream())
        if rc != LOSSY_OK:
            _check(self._ctx, rc)


def lossy_aggregate_alg1(ctx, step, grads, ghat_prev, ghat, count=None, recv_bits=None):
    _check(ctx, load_library().lossy_aggregate_alg1(ctx, step, _table(grads), _p(ghat_prev), _p(ghat), _p(count),
                                                    _p(recv_bits), _stream()))


def lossy_fused_step_alg1(ctx, step, grads, ghat_prev, master, m, v, replicas, ghat=None, count=None,
                          recv_bits=None, stale_bits=None, norms=None, sumsq=None):
    _check(ctx, load_library().lossy_fused_step_alg1(ctx, step, _table(grads), _p(ghat_prev), _p(master), _p(m),
                                                     _p(v), _table(replicas), _p(ghat), _p(count), _p(recv_bits),
                                                     _p(stale_bits), _p(norms), _p(sumsq), _stream()))


def lossy_fused_step_host(ctx, step, host_grads, dev_grads, master, m, v, replicas, dev_norms, host_norms):
    """host_grads: W CPU tensors (pinned: read in place over PCIe; pageable: staged through dev_grads, which
    may be None otherwise); host_norms: a CPU fp32 tensor of W elements (valid on return)."""
    _check(ctx, load_library().lossy_fused_step_host(ctx, step, _table(host_grads),
                                                     None if dev_grads is None else _table(dev_grads), _p(master),
                                                     _p(m), _p(v), _table(replicas), _p(dev_norms), _p(host_norms),
                                                     _stream()))


def lossy_mask(ctx, step, src, dst, packet, is_param=False) -> int:
    return load_library().lossy_mask(ctx, step, src, dst, packet, int(is_param))


def lossy_hash_u32(seed, step, src, dst, packet) -> int:
    return load_library().lossy_hash_u32(seed, step, src, dst, packet)


def lossy_mask_grid(ctx, step, src, dst, packet, out, is_param=False):
    _check(ctx, load_library().lossy_mask_grid(ctx, step, _p(src), _p(dst), _p(packet), src.numel(), int(is_param),
                                               _p(out), _stream()))


def lossy_closed_loop_grads(ctx, curv, target, noise, replicas, grads_out):
    _check(ctx, load_library().lossy_closed_loop_grads(ctx, _p(curv), _p(target), _table(noise), _table(replicas),
                                                       _table(grads_out), _stream()))


def lossy_device_status(ctx):
    """Synchronise the current stream; raises LossyError(LOSSY_EDEVICE) if a kernel gave up a bounded wait."""
    _check(ctx, load_library().lossy_device_status(ctx, _stream()))


def lossy_reset_status(ctx):
    _check(ctx, load_library().lossy_reset_status(ctx, _stream()))


def lossy_selftest_wait_expiry(ctx, max_polls: int = 1024):
    _check(ctx, load_library().lossy_selftest_wait_expiry(ctx, max_polls, _stream()))


def lossy_has_device_checks() -> bool:
    return bool(load_library().lossy_has_device_checks())


def lossy_selftest_shrink_checks(ctx, elems: int):
    _check(ctx, load_library().lossy_selftest_shrink_checks(ctx, elems))


def lossy_replica_elems(ctx, worker: int) -> int:
    return load_library().lossy_replica_elems(ctx, worker)


def lossy_last_error(ctx) -> str:
    return load_library().lossy_last_error(ctx).decode()


def lossy_num_packets(ctx) -> int:
    return load_library().lossy_num_packets(ctx)


def lossy_kernel_launches(ctx) -> int:
    return load_library().lossy_kernel_launches(ctx)


def lossy_describe_plan(ctx, with_drift: bool = True) -> str:
    """Text naming the kernel build lossy_fused_step would launch for this context's complete packets."""
    buf = C.create_string_buffer(128)
    _check(ctx, load_library().lossy_describe_plan(ctx, int(with_drift), buf, len(buf)))
    return buf.value.decode()
