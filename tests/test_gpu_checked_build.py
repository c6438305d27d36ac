"""The parity and random-case tests once more against the checked build of the library (-DSAGEKV_CHECKS): every
global-memory index of the kernels is compared with the extent the call was given, a violation is recorded in
the context's status word (and the access skipped) instead of being executed.  The tests themselves assert a
clean status word after every case, so a green run means no kernel stepped outside its buffers on any of them.
This is the stand-in for a memory checker, which cannot be run on every machine."""

import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FILES = ["tests/test_gpu_score_fuzz.py", "tests/test_gpu_select_fuzz.py", "tests/test_gpu_decode_fuzz.py",
         "tests/test_gpu_select_and_errors.py", "tests/test_gpu_refresh.py"]
PARITY = "tests/test_gpu_parity.py"
PARITY_CASES = "c1_full or scaled or strided or group_sizes or degenerate or softmax_scale or dependent or prefetch"


def test_parity_and_random_cases_on_the_checked_build():
    from paper_2503_08879_b200 import build
    lib = build.build(checks=True)
    env = dict(os.environ, SAGEKV_LIB=lib)
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2503_08879_b200 import binding as B; print(B.lib.sagekv_checked_build())"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr[-2000:]
    for args in (FILES, [PARITY, "-k", PARITY_CASES]):
        res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu"] + args, cwd=ROOT, env=env,
                             capture_output=True, text=True)
        assert res.returncode == 0, (res.stdout[-3000:], res.stderr[-2000:])
