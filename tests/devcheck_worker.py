"""Runs in a child process whose environment selects the debug library (LOSSY_B200_CHECKED=1): parity of every kernel
family with the index checks compiled in, then the checks' failure report, made to fire without any access out of
bounds (the checks are told a smaller element count than the arrays really have)."""
import sys

import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun, run_parity

SKIP = L.LOSSY_REPLICA_SKIP_OWNER
CASES = [
    # name, W, n, P, p, optimizer, gradient type, replica type, flags, fused, kernel named in a failed check
    ("register", 8, 2048 * 9 + 77, 2048, 0.2, "adam", "bf16", "bf16", L.LOSSY_REGISTER_PATH, True, "register kernel"),
    ("register_elided", 5, 512 * 23 + 9, 512, 0.3, "sgd", "f32", "bf16", L.LOSSY_REGISTER_PATH | SKIP, True, "register kernel"),
    ("register_packets_shorter_than_a_chunk_elided", 17, 128 * 60, 128, 0.3, "adam", "bf16", "bf16", L.LOSSY_REGISTER_PATH | SKIP, True, "register kernel"),
    ("fused_bulk", 8, 2048 * 11, 2048, 0.1, "adam", "bf16", "bf16", 0, True, "fused bulk-copy pipeline"),
    ("fused_bulk_elided_w17", 17, 4096 * 40, 4096, 0.3, "adam", "bf16", "f32", SKIP, True, "fused bulk-copy pipeline"),
    ("fused_packed", 16, 256 * 64, 256, 0.1, "adam", "bf16", "bf16", L.LOSSY_PACKED_BULK, True, "fused bulk-copy pipeline (packed)"),
    ("gather_drift_warps", 12, 256 * 67, 256, 0.3, "adam", "bf16", "bf16", 0, True, "gather pipeline"),
    ("gather_twin_elided", 3, 512 * 21, 512, 0.4, "adam", "f32", "f32", SKIP, True, "gather pipeline"),
    ("single_phase", 8, 2048 * 11, 2048, 0.1, "adam", "bf16", "bf16", 0, False, "single-phase bulk-copy pipeline"),
]


def main():
    assert L.lossy_has_device_checks(), "the child process did not bind to the debug library"
    for name, W, n, P, p, opt, gd, rd, flags, fused, where in CASES:
        w = workload.Workload(name, W, n, P, p, opt, 1e-2 if opt == "sgd" else 3e-4, gd, rd, 3, seed=11)
        run_parity(w, 3, fused=fused, flags=flags)              # identical results, and a clean status, with the checks in
        gpu = GpuRun(w, flags=flags)
        grads = [workload.grad_slab(w, 1, i, 0, w.n, "cuda") for i in range(W)]
        L.lossy_selftest_shrink_checks(gpu.ctx, 2 * P + 5)      # the last packets now fail their range check
        (gpu.step_fused if fused else gpu.step_unfused)(1, grads)
        try:
            L.lossy_device_status(gpu.ctx)
        except L.LossyError as e:
            assert e.code == L.LOSSY_EDEVCHECK, e
            assert where + ":" in str(e), (where, str(e))
        else:
            raise AssertionError(f"{name}: the shrunk range check did not fire")
        torch.cuda.synchronize()                                # the device context is intact
        L.lossy_reset_status(gpu.ctx)
        L.lossy_selftest_shrink_checks(gpu.ctx, 0)
        (gpu.step_fused if fused else gpu.step_unfused)(2, grads)
        L.lossy_device_status(gpu.ctx)                          # clean again
        gpu.close()
        print("ok", name, flush=True)
    print("DEVCHECK-WORKER-PASSED")


if __name__ == "__main__":
    sys.exit(main())
