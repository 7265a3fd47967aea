"""The debug build of the library (-DFF_DEBUG: every computed band rank, row offset and tile coordinate is
range-checked on the device and a value out of range raises FF_ERR_INVALID_ARG in the status word instead of
being used) runs a layer that reaches every tensor-core kernel; no check may fire and the result must match
the fp64 oracle like the release build's.  Run in a child process, because the binding loads one variant of
the library per process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import numpy as np
from paper_2604_22808_b200 import binding as B, configs as C, inputs as I
import harness as Hn
assert B._LIB_PATH.endswith("libfreqformer_debug.so")
for cfg, alloc in ((C.R64K, [1, 2, 4, 7, 2, 4]), (C.R_PAPER_REF, [1, 2, 4, 7]), (C.GEOM, [7, 2, 4])):
    Q, K, V = Hn.host_inputs(cfg)
    weights = I.router_weights(cfg)
    ts = [cfg.timesteps[0]] * cfg.batch
    res = Hn.oracle_forward(cfg, Q, K, V, weights, I.summary_projection(cfg), ts, alloc=alloc)
    out, plan = Hn.gpu_forward(cfg, Q, K, V, weights, None, timesteps=ts, alloc=alloc)     # asserts device status 0
    Hn.assert_close(out[0], res[0]["out"], cfg.dtype, cfg.name)
    plan.destroy()
print("DEBUG_BUILD_OK")
"""


def test_debug_build_runs_clean_and_matches():
    from paper_2604_22808_b200 import build as ffbuild
    ffbuild.build(debug=True)
    env = dict(os.environ, FF_LIBRARY_VARIANT="debug")
    child = CHILD % (ROOT, os.path.join(ROOT, "tests"))
    child = child.replace("C.GEOM", 'C._make("geom_16x16x128", 1, (16, 16, 128), 3, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 22, (500,))')
    r = subprocess.run([sys.executable, "-c", child], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "DEBUG_BUILD_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
