"""The checked build (libflashloop_debug.so, -DFL_DEBUG_BOUNDS): same results as the normal build on valid inputs, and
every damaged index array is refused with FL_ERR_INVALID_ARG (return value and status word) before anything is
launched that would follow it.  Runs in child processes because the library is chosen when the binding is imported."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
PKG = os.path.join(ROOT, "paper_2609_29812_b200")


def child(mode, lib):
    env = dict(os.environ, FLASHLOOP_LIB=os.path.join(PKG, lib), PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, os.path.join(HERE, "debug_bounds_child.py"), mode], env=env, capture_output=True,
                       text=True, timeout=600)
    assert r.returncode == 0, r.stdout + r.stderr
    return r.stdout.strip().splitlines()


def test_checked_build_agrees_and_refuses_damaged_indices():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import build
    build.build()                      # no-op when the three libraries are there and current
    normal = child("run", "libflashloop.so")
    checked = child("run", "libflashloop_debug.so")
    assert len(normal) == 2 and normal == checked
    report = child("corrupt", "libflashloop_debug.so")
    assert report == ["c1 refused every damaged input", "bf16 refused every damaged input"]
