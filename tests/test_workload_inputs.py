"""The seeded input generator: reproducible, sliceable, with the stated distribution. CPU only."""
import math

import torch

import workload
from workload import synth


def test_slabs_regenerate_bit_identically():
    full = workload.normal_f32(0, 3, 5, 0, 50000, 1e-3)
    assert torch.equal(workload.normal_f32(0, 3, 5, 12345, 23456, 1e-3), full[12345:23456])
    assert not torch.equal(workload.normal_f32(0, 3, 6, 0, 1000, 1e-3), full[:1000])   # redrawn per step
    assert not torch.equal(workload.normal_f32(0, 4, 5, 0, 1000, 1e-3), full[:1000])   # per worker
    assert not torch.equal(workload.normal_f32(1, 3, 5, 0, 1000, 1e-3), full[:1000])   # per seed


def test_moments_match_the_stated_bell():
    x = workload.normal_f32(0, 0, 1, 0, 1 << 20, 1e-3).double()
    n = x.numel()
    assert abs(x.mean().item()) < 5e-3 / math.sqrt(n)
    assert abs(x.std().item() / 1e-3 - 1) < 5e-3
    kurt = ((x - x.mean()) ** 4).mean().item() / x.var().item() ** 2 - 3
    assert abs(kurt + 0.3) < 0.02                       # Irwin-Hall n=4: excess kurtosis -6/(5*4)
    assert x.abs().max().item() <= 1e-3 * 131070 / synth._IH4_STD * 1.0001


def test_workload_shapes():
    w = workload.baseline_workloads()
    assert workload.LAYER_ELEMS == 202383360
    c2 = w["cfg2_w8_layer_adam"]
    assert c2.K == 98820 and c2.W == 8
    assert w["cfg3_w64_layer_p10"].K == 49410
    assert w["cfg1_w4_sgd_f32"].K == 1024
    assert w["cfg4_w8_full_model"].n == 6738411520


def test_shared_signal_plus_fixed_bias():
    w = workload.scaled(workload.baseline_workloads()["cfg3_w64_layer_p10"], 4096)
    a1, b1 = workload.grad_slab(w, 1, 0, 0, 4096).float(), workload.grad_slab(w, 1, 1, 0, 4096).float()
    a2, b2 = workload.grad_slab(w, 2, 0, 0, 4096).float(), workload.grad_slab(w, 2, 1, 0, 4096).float()
    assert a1.dtype == torch.float32 and workload.grad_slab(w, 1, 0, 0, 8).dtype == torch.bfloat16
    # the difference between two workers is the (fixed) bias difference, up to bf16 rounding
    d1, d2 = (a1 - b1), (a2 - b2)
    assert (d1 - d2).abs().max() < 2e-5
    assert abs(d1.std().item() / (1e-4 * math.sqrt(2)) - 1) < 0.1
    assert abs(a1.std().item() / 1e-3 - 1) < 0.05
