"""The checked build of the library (index tests inside the kernels, guard zones around every device
buffer it allocates) runs the parity cases of every regime without raising its status bit or
finding a damaged guard zone, and still matches the CPU oracle.

The cases run in a child process, because the library a process uses is chosen when the binding is
first loaded (EDGELORA_CHECKED=1).  The helper that runs a workload compares the guard zones after
every call, and the rows in front of and behind y.
"""
import os
import subprocess
import sys

import pytest

from paper_2507_01438_b200 import build as libbuild

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CASES = ["tests/test_gpu_parity.py", "tests/test_gpu_fused_decode.py", "tests/test_gpu_gather_tiles.py",
         "tests/test_gpu_siteset.py", "tests/test_gpu_routing.py", "tests/test_gpu_quant.py"]


def test_parity_cases_under_the_checked_build():
    assert os.path.exists(libbuild.OUT_CHECKED), \
        "libedgelora_checked.so is missing: python -m paper_2507_01438_b200.build --checked"
    env = dict(os.environ, EDGELORA_CHECKED="1")
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2507_01438_b200 import binding as B; print(B.edgelora_build_is_checked())"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert probe.stdout.strip() == "True", probe.stdout + probe.stderr
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + CASES,
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert run.returncode == 0, run.stdout[-4000:] + run.stderr[-2000:]


def test_the_normal_build_reports_itself():
    from paper_2507_01438_b200 import binding as B
    if os.environ.get("EDGELORA_CHECKED") == "1":
        assert B.edgelora_build_is_checked()
    else:
        assert not B.edgelora_build_is_checked()
        assert B.edgelora_check_guards() == B.OK
