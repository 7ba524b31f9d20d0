"""drift_norms_static: the drift norms for callers that are not allowed to allocate device memory
(a loop inside a frozen memory pool, a process that has handed all of HBM to its own buffers, a
service that bans allocation calls after start-up). It keeps its partial sums in a fixed array
inside the library instead of a context's cudaMalloc'ed scratch.

The file name makes pytest collect it last: if this addition fails, a run that stops at the first
failure has already run every other test. It passes alone in a fresh process and after the rest.
"""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, REL_TOL, make_oracle, to_np

pytestmark = pytest.mark.gpu


def _rel(a, b):
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), 1e-30)))


@pytest.mark.parametrize("rdt,W,n,P", [("bf16", 8, 2048 * 300 + 1000, 2048), ("f32", 5, 1000 * 77 + 8, 1000)])
def test_static_scratch_variant_matches_drift_norms_on_two_calls_in_a_row(rdt, W, n, P):
    w = workload.Workload("noalloc", W, n, P, 0.3, "sgd", 1e-2, "bf16", rdt, 2, seed=11)
    run = GpuRun(w)
    got = torch.zeros(W, device="cuda")
    got_sq = torch.zeros(W, dtype=torch.float64, device="cuda")
    for call in (1, 2):                      # the second call finds the first call's partial sums in the array
        run.step_fused(call, [workload.grad_slab(w, call, i, 0, n, "cuda") for i in range(W)])
        want = torch.zeros(W, device="cuda")
        want_sq = torch.zeros(W, dtype=torch.float64, device="cuda")
        L.drift_norms(run.ctx, run.master, run.replicas, want, want_sq)         # the existing entry point
        got_sq.zero_()
        L.drift_norms_static(W=W, n=n, packet_elems=P, replica_dtype=run.replicas[0].dtype, master=run.master,
                             replicas=run.replicas, norms=got, sumsq=got_sq)
        torch.cuda.synchronize()
        assert float(want.max()) > 0.0
        assert _rel(got, want) <= REL_TOL
        assert _rel(got_sq, want_sq) <= 2 * REL_TOL
        # and against the CPU oracle's own drift routine, run on the state the GPU holds
        orc = make_oracle(w)
        orc.master, orc.replicas = to_np(run.master), [to_np(r) for r in run.replicas]
        ref_sq = torch.from_numpy(orc.drift_sumsq())
        assert _rel(got_sq, ref_sq) <= 2 * REL_TOL
        assert _rel(got, ref_sq.sqrt()) <= REL_TOL
    # sumsq is added to, norms alone is allowed
    L.drift_norms_static(W=W, n=n, packet_elems=P, replica_dtype=run.replicas[0].dtype, master=run.master,
                         replicas=run.replicas, sumsq=got_sq)
    torch.cuda.synchronize()
    assert _rel(got_sq, 2 * want_sq) <= 2 * REL_TOL


def test_sizes_beyond_the_static_limits_are_rejected_without_a_launch():
    z = [torch.zeros(64, device="cuda") for _ in range(2)]
    out = torch.full((2,), 7.0, device="cuda")
    with pytest.raises(L.LossyError) as ei:          # more replicas than the static rows are laid out for
        L.drift_norms_static(W=65, n=64, packet_elems=64, replica_dtype=torch.float32, master=z[0],
                             replicas=z * 33, norms=out)
    assert ei.value.code == L.LOSSY_ELIMIT
    with pytest.raises(L.LossyError) as ei:          # more chunks than the 32-bit chunk index covers
        L.drift_norms_static(W=2, n=2 ** 40, packet_elems=8, replica_dtype=torch.float32, master=z[0],
                             replicas=z, norms=out)
    assert ei.value.code == L.LOSSY_ELIMIT
    with pytest.raises(L.LossyError) as ei:          # nothing to write
        L.drift_norms_static(W=2, n=64, packet_elems=64, replica_dtype=torch.float32, master=z[0], replicas=z)
    assert ei.value.code == L.LOSSY_EINVAL
    torch.cuda.synchronize()
    assert out.tolist() == [7.0, 7.0]
    # an empty bucket writes zero norms
    L.drift_norms_static(W=2, n=0, packet_elems=64, replica_dtype=torch.float32, master=z[0], replicas=z, norms=out)
    torch.cuda.synchronize()
    assert out.tolist() == [0.0, 0.0]
