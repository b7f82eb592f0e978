"""The small-case parity files once more, against the bounds-checked build of the library.

``libdq_checked.so`` is the same source compiled with ``-DDQ_CHECKED``: every store of a kernel to
global memory first checks that it lies inside the buffer it belongs to (the extents are in the
kernel's arguments) and raises ``DQ_STAT_INTERNAL`` instead of storing if it does not.  The parity
tests assert a clean status word after every call, so an out-of-bounds store anywhere in the cases
they cover fails them here -- the stand-in for a memory checker, which cannot be run on this
hardware pool.  (Stores of the average kernel leave through a TMA tensor store, which the
hardware clips to the tensor map's extents.)
"""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FILES = ["tests/test_gpu_parity.py", "tests/test_gpu_fuzz.py", "tests/test_gpu_norm_range.py",
         "tests/test_gpu_norm_family.py", "tests/test_gpu_team_route.py"]


def test_small_case_parity_files_pass_on_the_checked_build():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2107_14575_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, DQ_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", *FILES],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
