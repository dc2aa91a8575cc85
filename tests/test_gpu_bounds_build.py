"""The parity cases against the checked build (-DH2O_BOUNDS): the stand-in for a memory checker.

Every slot, unit and prompt-row index of the kernels is verified before use in that build; a violation would show as
H2O_ERR_STATE in the status word, which every case checks.  The binding loads one library per process, so the
cases run as a script in a child process with H2O_B200_LIB pointing at the checked library.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_parity_cases_pass_on_the_checked_build(oracle):
    import torch

    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU fallback"
    import __graft_entry__

    __graft_entry__.build()
    import paper_2306_14048_b200 as pkg

    assert pkg.lib.h2o_debug_bounds_checked() == 0  # this process runs the normal build
    lib = os.path.join(ROOT, "paper_2306_14048_b200", "libh2o_b200_bounds.so")
    assert os.path.exists(lib)
    env = dict(os.environ, H2O_B200_LIB=lib)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "bounds_cases.py")], env=env, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0 and "BOUNDS_CASES_PASSED" in res.stdout, res.stdout[-3000:] + res.stderr[-3000:]


def test_checked_build_exists_and_exports_the_same_symbols():
    import ctypes

    import __graft_entry__

    __graft_entry__.build()
    import paper_2306_14048_b200 as pkg

    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2306_14048_b200", "libh2o_b200_bounds.so"))
    for name in pkg.EXPORTED:
        assert hasattr(lib, name), name
    lib.h2o_debug_bounds_checked.restype = ctypes.c_int
    assert lib.h2o_debug_bounds_checked() == 1
