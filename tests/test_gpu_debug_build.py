"""The -DMONA_DEBUG build (libmona_debug.so): the kernels check their own indices - tile coordinates, slab positions,
staging offsets, the addresses of the axpy operand, slab ranges of the elementwise passes - and latch MONA_ERR_BOUNDS
in the status word instead of trapping.  It stands in for a memory checker where none is available.  The parity cases
with ragged tiles, padded batches, tall / wide / tiny shapes and both state formats run under it in a child process
(the library is chosen when the binding first loads it) and must come back clean and within tolerance."""
import os
import subprocess
import sys

import pytest

from paper_2605_26842_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import torch
import paper_2605_26842_b200 as pkg
from paper_2605_26842_b200 import binding
from tests.parity_util import TOL_O_BF16, TOL_STATE, TOL_W, run_case
assert binding._LIB_PATH.endswith("libmona_debug.so"), binding._LIB_PATH
cases = [dict(shapes=[(1, 72, 200), (1, 1000, 136), (3, 192, 320), (2, 320, 192)], steps=2, seed=3),
         dict(shapes=[(5, 256, 768), (2, 768, 256), (1, 1024, 1536), (1, 32, 512), (1, 33, 17)], steps=2, seed=4),
         dict(shapes=[(3, 128, 384)], steps=3, seed=9, grad_dtype=torch.bfloat16, pad=64),
         dict(shapes=[(2, 512, 256), (1, 264, 520)], steps=3, seed=21, lite=True),
         dict(shapes=[(2, 2048, 768), (1, 1536, 2048)], steps=1, seed=5),
         dict(shapes=[(4, 256, 512)], steps=2, seed=6, options=pkg.default_options(fuse_update=1, ns_delay=1, macro_tile_min_k=64))]
for kw in cases:
    errs = run_case(**kw)       # run_case polls the status word after every step and fails on anything but MONA_OK
    assert errs["M"] <= (3e-4 if kw.get("lite") else TOL_STATE), errs
    assert errs["O"] <= TOL_O_BF16 and errs["dW"] <= TOL_W, errs
print("debug build clean")
"""


@pytest.mark.gpu
def test_parity_cases_run_clean_under_the_index_checking_build():
    lib = build_mod.build(debug=True)
    env = dict(os.environ, MONA_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "debug build clean" in res.stdout


def test_debug_build_exports_the_same_entry_points():
    import ctypes as C
    import re
    lib = C.CDLL(build_mod.build(debug=True))
    text = open(os.path.join(ROOT, "include", "mona.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for name in sorted(set(re.findall(r"\b(mona_[a-z_0-9]+)\s*\(", text))):
        assert hasattr(lib, name), name
