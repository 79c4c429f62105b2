"""The checked build (libcovspec_debug.so, -DCOVSPEC_DEBUG_BOUNDS) run in a child process: the small
parity cases must pass with a clean device status (no index test fires on valid input), and a kept
index that lies outside its request must be reported as COVSPEC_ERR_BOUNDS with the row skipped
instead of gathered."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
import numpy as np
import torch
from paper_2605_02218_b200 import api, workloads
from tests import parity

lib = api.load_library()
assert lib.covspec_build_has_bounds_checks() == 1, "the checked library was not the one loaded"
for seed, kw in [(51, dict(batch=3, n_vis=(150, 700), n_txt=(3, 20), d=256, n_heads=2, rank=16, keep_ratio=0.25)),
                 (52, dict(batch=2, n_vis=(1300, 2100), n_txt=(8, 40), d=384, n_heads=3, rank=24, keep_ratio=0.3))]:
    wl = workloads.make_workload("checked%d" % seed, seed=seed, dtype=torch.bfloat16, **kw)
    st = parity.run_gpu(wl)
    print("parity", wl.name, st["keep_exact"], "of", st["requests"])
wl = workloads.make_config("c2")
parity.run_gpu(wl)

# a kept index outside its request (but inside X, so that no build could fault on it)
wl = workloads.make_workload("bad-index", seed=53, dtype=torch.bfloat16, batch=2, n_vis=(200, 300),
                             n_txt=(4, 8), d=256, n_heads=2, rank=16, keep_ratio=0.25).to("cuda:0")
pr = api.Pruner.for_workload(wl)
m = pr.marshal(wl)
out, keep_idx, ko = pr.prune(m)
assert pr.device_status() == 0
bad = keep_idx.clone()
n0 = int(wl.vis_offsets[1] - wl.vis_offsets[0])
bad[0] = n0 + 3                                   # request 0 has n0 tokens
sentinel = torch.full_like(out, 7.0)
ko_arr = np.asarray(ko, dtype=np.int32)
import ctypes as C
st = pr.lib.covspec_compact(pr._ctx, C.byref(m.problem), api._ptr(bad), ko_arr.ctypes.data_as(C.POINTER(C.c_int)),
                            api._ptr(sentinel), None, api._stream())
assert st == 0, st
status = pr.device_status()
assert status == -10, status
torch.cuda.synchronize()
assert torch.all(sentinel[0] == 7.0), "the row with the bad index must not be written"
assert torch.equal(sentinel[1:], out[1:])
assert pr.device_status() == 0                    # cleared, context still usable
out2, keep2, _ = pr.prune(m)
assert torch.equal(out2, out) and torch.equal(keep2, keep_idx)
print("checked build ok")
"""


def test_checked_build_passes_parity_and_reports_a_bad_index():
    from paper_2605_02218_b200 import build
    path = build.build(debug_bounds=True)
    env = dict(os.environ, COVSPEC_LIBRARY=path, PYTHONPATH=ROOT)
    res = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True,
                         timeout=900)
    sys.stdout.write(res.stdout[-2000:])
    assert res.returncode == 0, res.stderr[-3000:]
    assert "checked build ok" in res.stdout
