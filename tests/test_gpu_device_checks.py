"""The debug build (the same sources with -DLOSSY_DEVCHECK): every kernel of the step path checks its index ranges
before touching memory. In a child process bound to that library: parity with the oracle is unchanged, and a
check that fails (made to fail by telling the checks a smaller element count than the arrays have, so nothing is
out of bounds) is reported as LOSSY_EDEVCHECK, naming the kernel, and leaves the context usable."""
import os
import subprocess
import sys

import pytest

import paper_2507_07114_b200 as L
import workload
from parity_util import GpuRun

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_debug_build_same_results_and_its_failure_report():
    env = dict(os.environ, LOSSY_B200_CHECKED="1", PYTHONPATH=os.pathsep.join([os.path.dirname(HERE), HERE, os.environ.get("PYTHONPATH", "")]))
    res = subprocess.run([sys.executable, os.path.join(HERE, "devcheck_worker.py")], env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "DEVCHECK-WORKER-PASSED" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


def test_normal_build_has_no_checks_and_says_so():
    assert not L.lossy_has_device_checks()
    w = workload.Workload("plain", 4, 2048 * 4, 2048, 0.1, "sgd", 1e-2, "bf16", "bf16", 1, seed=3)
    gpu = GpuRun(w)
    with pytest.raises(L.LossyError) as e:
        L.lossy_selftest_shrink_checks(gpu.ctx, 100)
    assert e.value.code == L.LOSSY_EINVAL
    L.lossy_device_status(gpu.ctx)
