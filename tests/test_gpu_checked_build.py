"""The bounds-check build of the library (liboasis_checked.so, -DOASIS_BOUNDS_CHECK): tiny configurations match the
oracle with every check armed, and each kind of index is flagged -- and its access skipped -- when it lies between
a declared extent and the larger size really allocated.  Runs in a process of its own because a process loads one
build of the library."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_build_parity_and_flags():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_08097_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, OASIS_LIB=lib)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "checked_worker.py")], env=env, capture_output=True,
                       text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    out = json.loads(r.stdout.strip().splitlines()[-1])
    assert out["ok"] and out["tiny_configs"] == 4 and len(out["flagged"]) == 8
