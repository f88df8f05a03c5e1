"""The bounds-checked build of the library (-DPEARL_CHECKED) under the parity tests.

In that build every index into a tree level, the Data Storage, a batch or a staging area is compared
with its extent before use; an index out of range raises PEARL_ST_INTERNAL instead of touching memory,
and the cross-CTA tickets carry release/acquire semantics.  The parity tests compare status bits with the
oracle's after every call, so a check that fires anywhere fails a test.  A representative part of the
suite is run in a child process with PEARL_PRB_LIB pointing at the checked library.
"""
import os
import subprocess
import sys

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu

SUBSET = ("small_buffers or random_call or step or captured or fused or large_batch_sample or many_cta_update or delta or "
          "falls_off or ragged or reduced_capacity or normalised_over or streamed or uniform or default_insert or "
          "after_insert or (sweep_cells and 65536-) or (sweep_cells and 1048576-16) or min_tree")


def test_parity_suite_against_the_checked_library():
    from paper_2311_09445_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, PEARL_PRB_LIB=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join("tests", "test_gpu_parity.py"), os.path.join("tests", "test_zz_no_alloc.py"),
                        os.path.join("tests", "test_gpu_min_tree.py"),
                        "-x", "-q", "-m", "gpu", "-k", SUBSET], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1800)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail
