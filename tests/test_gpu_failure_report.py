"""The library's failure report, exercised without a failure: a bounded wait that runs out sets the context's
status word; nothing faults, traps or hangs, and the context works again after a reset."""
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import run_parity

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_recovers():
    w = workload.scaled(workload.baseline_workloads()["cfg2_w8_layer_adam"], 2048 * 40 + 16)
    gpu, orc = run_parity(w, 2)                         # a healthy context: status is clean
    L.lossy_device_status(gpu.ctx)
    before = L.lossy_kernel_launches(gpu.ctx)
    L.lossy_selftest_wait_expiry(gpu.ctx, 1024)         # one small block waits on a barrier nothing completes
    with pytest.raises(L.LossyError) as ei:
        L.lossy_device_status(gpu.ctx)
    assert ei.value.code == L.LOSSY_EDEVICE
    assert L.lossy_kernel_launches(gpu.ctx) == before + 1
    with pytest.raises(L.LossyError) as ei:             # sticky until it is cleared
        L.lossy_device_status(gpu.ctx)
    assert ei.value.code == L.LOSSY_EDEVICE
    L.lossy_reset_status(gpu.ctx)
    L.lossy_device_status(gpu.ctx)
    # the CUDA context is intact and the same lossy context still computes what the oracle computes
    from parity_util import compare_outputs, compare_state, to_np
    for t in (3, 4):
        gs = [workload.grad_slab(w, t, i, 0, w.n) for i in range(w.W)]
        gpu.step_fused(t, [g.cuda() for g in gs])
        ref = orc.step(t, [to_np(g) for g in gs])
        compare_outputs(gpu.outputs(), ref, f"after reset, step {t}")
        compare_state(gpu, orc, f"after reset, step {t}")
    L.lossy_device_status(gpu.ctx)


def test_selftest_arguments_are_checked():
    ctx = L.lossy_init(W=2, n=64, packet_elems=64, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
                       replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
    for bad in (0, (1 << 20) + 1):
        with pytest.raises(L.LossyError) as ei:
            L.lossy_selftest_wait_expiry(ctx, bad)
        assert ei.value.code == L.LOSSY_EINVAL
    L.lossy_device_status(ctx)
    assert L.lossy_kernel_launches(ctx) == 0
    L.lossy_destroy(ctx)


def test_step_zero_is_rejected_by_every_entry_point_that_hashes_the_step():
    n = 1024 * 4
    ctx = L.lossy_init(W=2, n=n, packet_elems=1024, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
                       replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
    z = [torch.zeros(n, device="cuda") for _ in range(2)]
    count = torch.zeros(4, dtype=torch.uint8, device="cuda")
    for call in (lambda: L.lossy_aggregate(ctx, 0, z, z[0], count),
                 lambda: L.lossy_aggregate_alg1(ctx, 0, z, z[1], z[0], count),
                 lambda: L.lossy_step(ctx, 0, z[0], count, z[1]),
                 lambda: L.lossy_broadcast(ctx, 0, z[0], z),
                 lambda: L.lossy_fused_step(ctx, 0, z, z[0], None, None, z)):
        with pytest.raises(L.LossyError) as ei:
            call()
        assert ei.value.code == L.LOSSY_EINVAL
    assert L.lossy_kernel_launches(ctx) == 0
    L.lossy_destroy(ctx)
