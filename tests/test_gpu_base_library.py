"""The library without cluster-multicast operand loads is the one every multi-GPU run uses; on one GPU
the binding prefers the optional single-GPU build when it exists.  This test runs the einsum and
feed-forward parity tests once more in a child process that is told to load the base library, so
both builds stay covered whichever one the other tests happened to load."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_suite_on_the_base_library():
    import paper_1811_02084_b200 as mtf
    from paper_1811_02084_b200 import binding
    if os.path.basename(binding.LIB_PATH) == "libmtf_b200.so":
        pytest.skip("this process already runs the base library")
    env = dict(os.environ, MTF_NO_MULTICAST="1")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_einsum.py"), os.path.join(ROOT, "tests", "test_gpu_ffn.py")]
    proc = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert proc.returncode == 0, proc.stdout[-3000:] + proc.stderr[-2000:]
