"""Counter-based synthetic gradients and initial parameters.

Every value is a pure function of (seed, stream, step, element index), built from
64-bit integer hashing and ONE fp32 multiply, so that CPU and CUDA tensors are
bit-identical and any slab [e0, e1) can be regenerated on its own.

Distribution: the sum of the four 16-bit fields of a hashed word, centred, times
sigma / 37837.227 — a symmetric bell (Irwin-Hall, n = 4) with standard deviation
sigma and excess kurtosis -0.3, standing in for N(0, sigma).
"""
from __future__ import annotations

import dataclasses
import math

import torch

_M64 = (1 << 64) - 1
# one LLaMA-2-7B decoder layer: q,k,v,o 4096x4096; gate,up 4096x11008; down 11008x4096; two RMSNorm 4096
LAYER_ELEMS = 4 * 4096 * 4096 + 2 * 4096 * 11008 + 11008 * 4096 + 2 * 4096
_IH4_STD = math.sqrt(4 * (65536.0 ** 2 - 1.0) / 12.0)  # std of the sum of four U{0..65535}

STREAM_SHARED = 1000   # the signal all workers share (config 3)
STREAM_BIAS = 2000     # + worker: per-worker bias, fixed over steps (config 3)
STREAM_THETA = 3000    # initial parameters


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same bit pattern."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _fmix_int(z: int) -> int:
    z &= _M64
    z ^= z >> 33
    z = (z * 0xFF51AFD7ED558CCD) & _M64
    z ^= z >> 33
    z = (z * 0xC4CEB9FE1A85EC53) & _M64
    z ^= z >> 33
    return z


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _fmix_tensor(z: torch.Tensor) -> torch.Tensor:
    z = z ^ _lsr(z, 33)
    z = z * _s64(0xFF51AFD7ED558CCD)
    z = z ^ _lsr(z, 33)
    z = z * _s64(0xC4CEB9FE1A85EC53)
    z = z ^ _lsr(z, 33)
    return z


def _key(seed: int, stream: int, step: int) -> int:
    return _fmix_int(_fmix_int(seed * 0x9E3779B97F4A7C15 + stream) ^ (step * 0xD1B54A32D192ED03))


def normal_f32(seed: int, stream: int, step: int, e0: int, e1: int, sigma: float,
               device="cpu") -> torch.Tensor:
    """fp32 tensor of elements [e0, e1) of the (seed, stream, step) sequence."""
    out = torch.empty(e1 - e0, dtype=torch.float32, device=device)
    key = _s64(_key(seed, stream, step))
    scale = torch.tensor(sigma / _IH4_STD, dtype=torch.float32).item()  # rounded once to fp32
    chunk = 1 << 24
    for c0 in range(e0, e1, chunk):
        c1 = min(e1, c0 + chunk)
        e = torch.arange(c0 + 1, c1 + 1, dtype=torch.int64, device=device)
        z = _fmix_tensor(e * _s64(0x9E3779B97F4A7C15) + key)
        s = (z & 0xFFFF) + (_lsr(z, 16) & 0xFFFF) + (_lsr(z, 32) & 0xFFFF) + _lsr(z, 48)
        out[c0 - e0:c1 - e0] = (s - 131070).to(torch.float32) * scale
    return out


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic configuration (shapes follow the LLaMA-2-7B training setup of the paper's
    Experiments section; drop rates and worker counts are the paper's)."""
    name: str
    W: int
    n: int
    packet_elems: int
    p: float
    optimizer: str          # "sgd" | "adam"
    lr: float
    grad_dtype: str         # "f32" | "bf16"
    replica_dtype: str
    steps: int
    grad_sigma: float = 1e-3
    bias_sigma: float = 0.0     # > 0: g_i = shared signal + fixed per-worker bias
    theta_sigma: float = 0.02
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    seed: int = 0
    packet_base: int = 0

    @property
    def K(self) -> int:
        return (self.n + self.packet_elems - 1) // self.packet_elems


def baseline_workloads() -> dict:
    """The benchmark configurations by name."""
    emb = 32000 * 4096
    return {
        "cfg1_w4_sgd_f32": Workload("cfg1_w4_sgd_f32", 4, 1 << 20, 1024, 0.1, "sgd", 1e-2, "f32", "f32", 10),
        "cfg2_w8_layer_adam": Workload("cfg2_w8_layer_adam", 8, LAYER_ELEMS, 2048, 0.1, "adam", 3e-4,
                                       "bf16", "bf16", 100),
        "cfg3_w64_layer_p01": Workload("cfg3_w64_layer_p01", 64, LAYER_ELEMS, 4096, 0.01, "adam", 3e-4,
                                       "bf16", "bf16", 50, bias_sigma=1e-4),
        "cfg3_w64_layer_p10": Workload("cfg3_w64_layer_p10", 64, LAYER_ELEMS, 4096, 0.1, "adam", 3e-4,
                                       "bf16", "bf16", 50, bias_sigma=1e-4),
        "cfg4_w8_full_model": Workload("cfg4_w8_full_model", 8, 32 * LAYER_ELEMS + 2 * emb, 2048, 0.1,
                                       "adam", 3e-4, "bf16", "bf16", 20),
        "cfg5_w16_layer_sweep": Workload("cfg5_w16_layer_sweep", 16, LAYER_ELEMS, 2048, 0.1, "adam", 3e-4,
                                         "bf16", "bf16", 20),
    }


def scaled(w: Workload, n: int, **kw) -> Workload:
    """The same recipe on a smaller (or ragged) bucket, for element-by-element parity tests."""
    return dataclasses.replace(w, n=n, **kw)


def _torch_dtype(name: str):
    return torch.bfloat16 if name == "bf16" else torch.float32


def grad_slab(w: Workload, step: int, worker: int, e0: int, e1: int, device="cpu") -> torch.Tensor:
    """Worker `worker`'s gradient elements [e0, e1) at `step`, in the workload's gradient dtype.
    Redrawn every step; with bias_sigma > 0 a shared signal plus a per-worker bias that is fixed
    over steps, added in fp32 and rounded once."""
    if w.bias_sigma > 0.0:
        g = normal_f32(w.seed, STREAM_SHARED, step, e0, e1, w.grad_sigma, device)
        g = g + normal_f32(w.seed, STREAM_BIAS + worker, 0, e0, e1, w.bias_sigma, device)
    else:
        g = normal_f32(w.seed, worker, step, e0, e1, w.grad_sigma, device)
    return g.to(_torch_dtype(w.grad_dtype))


def theta0_slab(w: Workload, e0: int, e1: int, device="cpu") -> torch.Tensor:
    """Initial fp32 master parameters, elements [e0, e1)."""
    return normal_f32(w.seed, STREAM_THETA, 0, e0, e1, w.theta_sigma, device)
