"""GPU parity of the Algorithm 1 mode (reliable reduce, one drop draw per packet with reuse of the
previous aggregate, stale-retaining broadcast) against the oracle, on every kernel that serves it."""
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, run_parity

pytestmark = pytest.mark.gpu
CFG = workload.baseline_workloads()
REG, SKIP = L.LOSSY_REGISTER_PATH, L.LOSSY_ZERO_SKIP

CASES = [
    # name, W, n, P, p_grad, p_param, opt, gd, rd, flags
    ("cfg2_shape_wide", 8, 2048 * 37 + 1003, 2048, 0.1, 0.1, "adam", "bf16", "bf16", 0),
    ("cfg2_shape_heavy_loss", 8, 2048 * 41, 2048, 0.5, 0.3, "adam", "bf16", "bf16", 0),
    ("shard_granular_w8", 8, 8 * 10240, 10240, 0.3, 0.2, "adam", "bf16", "bf16", 0),
    ("shard_granular_w5_ragged", 5, 5 * 4104 - 16, 4104, 0.4, 0.4, "sgd", "f32", "f32", 0),
    ("w64_twin", 64, 4096 * 70 + 40, 4096, 0.2, 0.05, "adam", "bf16", "bf16", 0),
    ("w16_two_groups", 16, 2048 * 30, 2048, 0.25, 0.25, "adam", "bf16", "f32", 0),
    ("small_packets_register", 6, 256 * 90 + 24, 256, 0.3, 0.1, "adam", "bf16", "bf16", 0),
    ("zero_skip_on_drop", 4, 1024 * 33, 1024, 0.5, 0.2, "adam", "f32", "bf16", SKIP),
    ("tiny", 3, 45, 8, 0.5, 0.5, "sgd", "bf16", "bf16", 0),
    ("packed_small_packets_low_loss", 8, 256 * 70 + 24, 256, 0.1, 0.1, "adam", "bf16", "bf16", 0),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("mode", ["fused", "fused_reg", "unfused"])
def test_alg1_parity(case, mode):
    name, W, n, P, pg, pp, opt, gd, rd, flags = case
    w = workload.Workload("alg1_" + name, W, n, P, pg, opt, 1e-2 if opt == "sgd" else 3e-4, gd, rd, 6, seed=21)
    gpu, orc = run_parity(w, 6, fused=mode != "unfused", flags=flags | (REG if mode == "fused_reg" else 0),
                          p_grad=pg, p_param=pp, alg1=True)
    kept = (gpu.count == W).sum().item()
    assert 0 < kept < gpu.count.numel() or gpu.count.numel() < 4     # both branches were exercised


def test_alg1_without_loss_equals_the_default_path_bitwise():
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 25, p=0.0)
    a, b = GpuRun(w, alg1=True), GpuRun(w)
    for t in range(1, 5):
        gd = [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)]
        a.step_fused(t, gd)
        b.step_fused(t, gd)
    torch.cuda.synchronize()
    assert torch.equal(a.master, b.master) and torch.equal(a.ghat, b.ghat) and torch.equal(a.ghat_prev, a.ghat)
    for x, y in zip(a.replicas, b.replicas):
        assert torch.equal(x, y)


def test_alg1_rejects_self_lossless_and_missing_state():
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 4)
    run = GpuRun(w, flags=L.LOSSY_SELF_LOSSLESS, alg1=True)
    gd = [workload.grad_slab(w, 1, i, 0, w.n, "cuda") for i in range(w.W)]
    with pytest.raises(L.LossyError) as ei:
        run.step_fused(1, gd)
    assert ei.value.code == L.LOSSY_EINVAL
    run2 = GpuRun(w, alg1=True)
    run2.ghat_prev = None
    with pytest.raises((L.LossyError, AttributeError)):
        run2.step_fused(1, gd)
    assert L.lossy_kernel_launches(run.ctx) == 0
