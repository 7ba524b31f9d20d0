"""Hybrid reliable/unreliable transport on the GPU (reliable-link bitmaps, per-packet gradient norms)
against the oracle."""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, assert_rel, assert_same, compare_outputs, compare_state, make_oracle, to_np

pytestmark = pytest.mark.gpu
REG = L.LOSSY_REGISTER_PATH

CASES = [
    ("cfg2_shape", 8, 2048 * 37 + 1003, 2048, 0.3, "adam", "bf16", "bf16", False),
    ("w64", 64, 4096 * 30, 4096, 0.2, "adam", "bf16", "bf16", False),
    ("small_packets", 6, 256 * 80 + 16, 256, 0.4, "sgd", "f32", "f32", False),
    ("alg1", 8, 2048 * 33, 2048, 0.5, "adam", "bf16", "bf16", True),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("mode", ["fused", "fused_reg", "unfused"])
def test_importance_classes_by_gradient_norm(case, mode):
    """Each step the pieces whose norm is in the top quarter travel reliably (the rule is the caller's: here
    a quantile of lossy_packet_sqnorms); broadcasts of even packets are reliable."""
    name, W, n, P, p, opt, gd, rd, alg1 = case
    w = workload.Workload("rel_" + name, W, n, P, p, opt, 1e-2 if opt == "sgd" else 3e-4, gd, rd, 5, seed=23)
    gpu = GpuRun(w, flags=REG if mode == "fused_reg" else 0, alg1=alg1)
    orc = make_oracle(w, alg1=alg1)
    K = w.K
    rel = torch.zeros(2 * K, dtype=torch.int64, device="cuda")
    L.lossy_set_reliable(gpu.ctx, rel)
    sq = torch.zeros(W * K, dtype=torch.float32, device="cuda")
    shifts = torch.arange(W, dtype=torch.int64, device="cuda")[:, None]
    for t in range(1, 6):
        gs = [workload.grad_slab(w, t, i, 0, n) for i in range(W)]
        gd_ = [g.cuda() for g in gs]
        L.lossy_packet_sqnorms(gpu.ctx, gd_, sq)
        want_sq = orc.packet_sqnorms([to_np(g) for g in gs])
        assert_rel(sq.cpu().numpy().reshape(W, K), want_sq, f"{name} step {t} packet norms", tol=2e-5)
        # the caller's importance rule, applied to the ORACLE's norms so both sides get the same bitmap
        thr = np.quantile(want_sq, 0.75)
        bits = torch.from_numpy((want_sq > thr)).cuda().to(torch.int64)
        rel[:K] = (bits << shifts).sum(dim=0)
        rel[K:] = torch.where(torch.arange(K, device="cuda") % 2 == 0, torch.tensor(-1, device="cuda"),
                              torch.tensor(0, device="cuda"))
        (gpu.step_fused if mode != "unfused" else gpu.step_unfused)(t, gd_)
        ref = orc.step(t, [to_np(g) for g in gs], reliable=to_np(rel).view(np.uint64).reshape(2, K))
        compare_outputs(gpu.outputs(), ref, f"{name} step {t}")
        compare_state(gpu, orc, f"{name} step {t}")
    assert int(gpu.stale[::2].abs().sum()) == 0 and int(gpu.stale[1::2].ne(0).sum()) > 0
    assert_same(to_np(gpu.master), orc.master, "master bits")
    L.lossy_set_reliable(gpu.ctx, None)
    L.lossy_device_status(gpu.ctx)
