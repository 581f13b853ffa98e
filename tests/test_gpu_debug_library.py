"""The debug library (libpsa_debug.so: the product sources built with -DPSA_DEBUG_BOUNDS, every index a
thread forms itself checked against its tensor) on small packs: results as the product library's, and no
check fires.  It runs in a process of its own because a process loads one of the two libraries.  The
product library's side of the self test (the check compiles to nothing there) runs here."""
import os
import subprocess
import sys

import pytest
import torch

from paper_2410_20305_b200 import binding as B

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_debug_library_runs_the_small_packs_without_an_index_out_of_bounds():
    env = dict(os.environ, PSA_DEBUG_LIB="1")
    res = subprocess.run([sys.executable, os.path.join(HERE, "debug_library_cases.py")], env=env, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0 and "DEBUG_LIBRARY_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


def test_the_product_library_carries_no_index_checks():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.psa_selftest_bounds(status, result)
    torch.cuda.synchronize()
    assert int(result.item()) == 3 and int(status.item()) == 0
