"""Pairwise drift matrix on the GPU (the theorem's D between two workers' copies) against the oracle,
and the stationary pair constant at scale."""
from math import comb

import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, assert_rel, make_oracle, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("W,n,P,rd", [(8, 2048 * 21 + 1003, 2048, "bf16"), (5, 1000 * 13, 1000, "f32"),
                                      (64, 1024 * 20 + 8, 1024, "bf16"), (3, 45, 8, "f32"), (13, 256 * 50, 256, "bf16")])
def test_pairwise_matrix_matches_the_oracle(W, n, P, rd):
    w = workload.Workload("pairwise", W, n, P, 0.3, "sgd", 1e-2, "bf16", rd, 4, seed=9)
    gpu, orc = GpuRun(w), make_oracle(w)
    for t in range(1, 5):
        gs = [workload.grad_slab(w, t, i, 0, n) for i in range(W)]
        gpu.step_fused(t, [g.cuda() for g in gs])
        orc.step(t, [to_np(g) for g in gs])
    d2 = torch.zeros(W * W, dtype=torch.float64, device="cuda")
    L.drift_pairwise(gpu.ctx, gpu.replicas, d2)
    torch.cuda.synchronize()
    got, want = d2.cpu().numpy().reshape(W, W), orc.pairwise_sumsq()
    assert np.all(np.diag(got) == 0) and np.allclose(got, got.T, rtol=1e-12, atol=0)
    off = ~np.eye(W, dtype=bool)
    assert_rel(got[off], want[off], "pairwise squared drift", tol=2e-5)
    L.drift_pairwise(gpu.ctx, gpu.replicas, d2)               # the matrix is added to
    torch.cuda.synchronize()
    assert_rel(d2.cpu().numpy().reshape(W, W)[off], 2 * want[off], "accumulation", tol=2e-5)


def test_pair_constant_of_the_theorem_at_scale():
    """Between two receivers the stationary squared drift per element is 2p/(1-p^2) sigma^2 where neither
    owns the packet and p/(1-p) sigma^2 where one of them does; bounded in t."""
    W, p, lr, sg = 8, 0.3, 1e-2, 1e-3
    n = 1024 * 16000
    w = workload.Workload("pair_at_scale", W, n, 1024, p, "sgd", lr, "bf16", "f32", 60, grad_sigma=sg, seed=14)
    gpu = GpuRun(w)
    d2 = torch.zeros(W * W, dtype=torch.float64, device="cuda")
    samples = 0
    for t in range(1, 61):
        gpu.step_fused(t, [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)], outputs=False)
        if t > 35:
            L.drift_pairwise(gpu.ctx, gpu.replicas, d2)
            samples += 1
    L.lossy_device_status(gpu.ctx)
    got = d2.cpu().numpy().reshape(W, W) / samples
    inv_c = sum(comb(W, c) * (1 - p) ** c * p ** (W - c) / c for c in range(1, W + 1))
    sigma2 = (lr * sg) ** 2 * inv_c
    pps = (w.K + W - 1) // W
    own = np.array([min(w.K, (i + 1) * pps) - min(w.K, i * pps) for i in range(W)]) * 1024
    for i in range(W):
        for k in range(W):
            if i == k:
                continue
            want = sigma2 * ((n - own[i] - own[k]) * 2 * p / (1 - p * p) + (own[i] + own[k]) * p / (1 - p))
            assert abs(got[i, k] / want - 1) < 0.03, (i, k, got[i, k] / want)
