"""The binding's prepared call (arguments of lossy_fused_step marshalled once) is the same call: same state, bit
for bit, as the plain binding call on the same inputs, in both modes."""
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, assert_same, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("alg1", [False, True])
def test_prepared_call_equals_the_plain_call(alg1):
    w = workload.Workload("prepared", 5, 1024 * 9 + 100, 1024, 0.25, "adam", 3e-4, "bf16", "bf16", 4, seed=9)
    a, b = GpuRun(w, alg1=alg1), GpuRun(w, alg1=alg1)
    sets = [[workload.grad_slab(w, s, i, 0, w.n, "cuda") for i in range(w.W)] for s in (1, 2)]
    calls = [L.lossy_fused_step_prepared(b.ctx, gs, b.master, b.m, b.v, b.replicas, b.ghat, b.count, b.recv, b.stale,
                                         b.norms, b.sumsq, ghat_prev=b.ghat_prev, stream=torch.cuda.current_stream())
             for gs in sets]
    for t in range(1, 5):
        a.step_fused(t, sets[t % 2])
        b.sumsq.zero_()
        calls[t % 2](t)
        oa, ob = a.outputs(), b.outputs()
        for k in oa:
            assert_same(ob[k], oa[k], f"step {t} {k}")
        assert_same(to_np(b.master), to_np(a.master), f"step {t} master")
        for i in range(w.W):
            assert_same(to_np(b.replicas[i]), to_np(a.replicas[i]), f"step {t} replica {i}")
    L.lossy_device_status(b.ctx)
