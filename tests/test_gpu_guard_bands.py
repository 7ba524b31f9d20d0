"""Out-of-bounds check without a sanitizer: every buffer sits between two poisoned 4 KB bands that must
come back untouched, on ragged sizes and on every kernel (bulk-copy wide / twin / packed, gather wide / twin,
register path, unfused calls)."""
import pytest
import torch

import paper_2507_07114_b200 as L
import workload

pytestmark = pytest.mark.gpu
BAND = 4096          # bytes on each side
POISON = 0x5A


class Guarded:
    """A tensor view with poisoned bands before and after it inside one allocation."""

    def __init__(self, n, dtype, fill=None):
        esz = torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((2 * BAND + n * esz + 16,), POISON, dtype=torch.uint8, device="cuda")
        self.nbytes = n * esz
        self.t = self.raw[BAND:BAND + self.nbytes].view(dtype)
        if fill is None:
            self.t.zero_()
        else:
            self.t.copy_(fill)

    def intact(self):
        return bool((self.raw[:BAND] == POISON).all()) and bool((self.raw[BAND + self.nbytes:] == POISON).all())


CASES = [
    # name, W, n, P, p, opt, gd, rd, flags
    ("wide_ragged", 8, 2048 * 19 + 1003, 2048, 0.2, "adam", "bf16", "bf16", 0),
    ("twin_w40_short_last_tile", 40, 1032 * 23 + 512, 1032, 0.2, "adam", "bf16", "f32", 0),
    ("twin_w64_split_staged", 64, 1024 * 30 + 16, 1024, 0.3, "adam", "bf16", "bf16", 0),
    ("packed_1024_two_per_wide_tile", 16, 1024 * 21 + 8, 1024, 0.05, "adam", "bf16", "bf16", 0),
    ("packed_256", 16, 256 * 45 + 40, 256, 0.1, "adam", "bf16", "bf16", L.LOSSY_PACKED_BULK),
    ("packed_128_twin", 30, 128 * 77 + 8, 128, 0.1, "sgd", "f32", "bf16", L.LOSSY_PACKED_BULK),
    ("gather_wide_256", 16, 256 * 45 + 40, 256, 0.1, "adam", "bf16", "bf16", 0),
    ("gather_wide_drift_warps_256", 16, 256 * 45 + 40, 256, 0.3, "adam", "bf16", "bf16", 0),
    ("gather_wide_drift_warps_quarters_512_f32_replicas", 5, 512 * 27 + 24, 512, 0.3, "adam", "bf16", "f32", L.LOSSY_GATHER_PATH),
    ("gather_wide_drift_warps_scratch_overflow", 24, 256 * 83 + 8, 256, 0.3, "sgd", "bf16", "bf16", 0),
    ("gather_twin_128", 20, 128 * 77 + 8, 128, 0.1, "sgd", "f32", "bf16", 0),
    ("gather_twin_few_workers_512", 3, 512 * 23 + 16, 512, 0.4, "adam", "bf16", "f32", 0),
    ("register_path", 8, 2048 * 7 + 5, 2048, 0.3, "adam", "bf16", "bf16", L.LOSSY_REGISTER_PATH),
    ("tiny_unaligned_tail", 3, 1029, 1000, 0.3, "sgd", "f32", "f32", 0),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("fused", [True, False])
def test_no_kernel_writes_outside_its_buffers(case, fused):
    name, W, n, P, p, opt, gd, rd, flags = case
    w = workload.Workload("guard_" + name, W, n, P, p, opt, 1e-2, gd, rd, 3, seed=3)
    gdt = torch.bfloat16 if gd == "bf16" else torch.float32
    rdt = torch.bfloat16 if rd == "bf16" else torch.float32
    K = w.K
    ctx = L.lossy_init(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=3, grad_dtype=gdt, replica_dtype=rdt,
                       optimizer=opt, lr=1e-2, flags=flags)
    th0 = workload.theta0_slab(w, 0, n, "cuda")
    master, m, v = Guarded(n, torch.float32, th0), Guarded(n, torch.float32), Guarded(n, torch.float32)
    reps = [Guarded(n, rdt, th0.to(rdt)) for _ in range(W)]
    ghat, prev = Guarded(n, torch.float32), Guarded(n, torch.float32)
    count, recv, stale = Guarded(K, torch.uint8), Guarded(K, torch.int64), Guarded(K, torch.int64)
    norms, sumsq = Guarded(W, torch.float32), Guarded(W, torch.float64)
    burst = Guarded(4 * K, torch.int64)
    adam = opt == "adam"
    everything = [master, m, v, ghat, prev, count, recv, stale, norms, sumsq, burst] + reps
    for t in range(1, 4):
        grads = [Guarded(n, gdt, workload.grad_slab(w, t, i, 0, n, "cuda")) for i in range(W)]
        if t == 3:
            L.lossy_set_bursty(ctx, 0.1, 0.4, burst.t)
        if fused:
            L.lossy_fused_step(ctx, t, [g.t for g in grads], master.t, m.t if adam else None, v.t if adam else None,
                               [r.t for r in reps], ghat.t, count.t, recv.t, stale.t, norms.t, sumsq.t)
            L.lossy_fused_step_alg1(ctx, t, [g.t for g in grads], prev.t, master.t, m.t if adam else None,
                                    v.t if adam else None, [r.t for r in reps], norms=norms.t)
        else:
            L.lossy_aggregate(ctx, t, [g.t for g in grads], ghat.t, count.t, recv.t)
            L.lossy_step(ctx, t, ghat.t, count.t, master.t, m.t if adam else None, v.t if adam else None)
            L.lossy_broadcast(ctx, t, master.t, [r.t for r in reps], stale.t)
            L.drift_norms(ctx, master.t, [r.t for r in reps], norms.t, sumsq.t)
            L.drift_norms_static(W=W, n=n, packet_elems=P, replica_dtype=rdt, master=master.t,
                                 replicas=[r.t for r in reps], norms=norms.t)
        L.lossy_device_status(ctx)
        for i, g in enumerate(everything + grads):
            assert g.intact(), f"{name}: band of buffer {i} was written at step {t}"
    L.lossy_destroy(ctx)
