"""The tcgen05 projection kernel (opt-in, Q4D_GEMM_KERNEL=tcgen05) against the same oracle checks as the default
kernels: the GEMM tests of test_gpu_ops.py and the toy decode steps of test_gpu_step.py, re-run in a child process
whose library reads the switch when it initialises."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("selection", [
    ["test_gpu_ops.py", "-k", "gemm"],
    ["test_gpu_step.py", "-k", "toy and chain and not moe"],
])
def test_same_checks_with_the_tcgen05_kernel(selection):
    env = dict(os.environ, Q4D_GEMM_KERNEL="tcgen05")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(HERE, selection[0])] + selection[1:]
    r = subprocess.run(cmd, env=env, cwd=os.path.dirname(HERE), capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
