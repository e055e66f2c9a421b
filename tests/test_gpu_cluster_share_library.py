"""Which library a process loads.  The default everywhere is libmtf_b200.so; the optional single-GPU
build (CTA clusters that share operand tiles) is loaded only on an explicit request, and only by a
process that drives one GPU and was not started by a multi-rank launcher.  The rest of the suite runs
on the default library; one child process covers the optional build with the einsum and feed-forward
parity tests."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _chosen(env_extra):
    code = "from paper_1811_02084_b200 import binding; import os; print(os.path.basename(binding.LIB_PATH))"
    env = {k: v for k, v in os.environ.items() if k not in ("MTF_CLUSTER_SHARE", "WORLD_SIZE", "LOCAL_WORLD_SIZE")}
    env.update(env_extra)
    proc = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert proc.returncode == 0, proc.stderr[-2000:]
    return proc.stdout.strip().splitlines()[-1]


def test_default_library_is_the_base_one():
    assert _chosen({}) == "libmtf_b200.so"


def test_opt_in_is_refused_under_a_multi_rank_launcher_or_without_exactly_one_gpu():
    # two ranks: refused whatever the machine has; here (or on any box) without exactly one visible GPU: refused too
    assert _chosen({"MTF_CLUSTER_SHARE": "1", "WORLD_SIZE": "2"}) == "libmtf_b200.so"
    assert _chosen({"MTF_CLUSTER_SHARE": "1", "CUDA_VISIBLE_DEVICES": ""}) == "libmtf_b200.so"


@pytest.mark.gpu
def test_this_process_runs_the_base_library():
    from paper_1811_02084_b200 import binding
    assert os.path.basename(binding.LIB_PATH) == "libmtf_b200.so"


@pytest.mark.gpu
def test_parity_suite_on_the_opt_in_library():
    import torch
    share = os.path.join(ROOT, "paper_1811_02084_b200", "libmtf_b200_mc.so")
    if not os.path.exists(share) or torch.cuda.device_count() != 1:
        pytest.skip("the optional single-GPU library is not built, or this process sees more than one GPU")
    env = dict(os.environ, MTF_CLUSTER_SHARE="1")
    env.pop("WORLD_SIZE", None)
    assert _chosen({"MTF_CLUSTER_SHARE": "1"}) == "libmtf_b200_mc.so"
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_einsum.py"), os.path.join(ROOT, "tests", "test_gpu_ffn.py")]
    proc = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert proc.returncode == 0, proc.stdout[-3000:] + proc.stderr[-2000:]
