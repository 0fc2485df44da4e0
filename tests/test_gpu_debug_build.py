"""The debug build of the library (-DFB_DEBUG): its kernels check every index they are about to
write - chosen expert ids inside [0, E) and distinct, rows inside [0, T), dispatch positions
inside [0, T k), slots inside [0, E) - and raise FB_ERR_INTERNAL in the device status word.
compute-sanitizer is not available to these tests; the checks, together with the guard regions
around every output buffer (tests/parity_util.py), stand in for it.  The test runs in a process
of its own because a process loads one build of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
sys.path.insert(0, sys.argv[1])
from paper_2608_14205_b200 import build as fb_build
fb_build.use_library(fb_build.build_variant("debug", ["-DFB_DEBUG"]))
import torch
from paper_2608_14205_b200 import binding as B, inputs as I
from tests import parity_util as P
cases = [("tiny", 500, 0), ("mixtral", 300, 0), ("qwen3", 1000, 0), ("dsv3", 777, 0), ("dsv3", 1500, 1),
         ("sweep32k", 900, 2)]
for name, T, pair_limit in cases:
    wl = I.WORKLOADS[name]
    li = I.make_layer(wl, 0, 0, T=T)
    ctx = P.make_context(wl, T)
    bkw = P.budget_kwargs(wl, T)
    gpu = P.run_gpu_layer(ctx, wl, li, bkw, pair_limit=pair_limit)     # guard regions are checked inside
    assert gpu["status"] == 0, (name, gpu["status"])
    P.compare_layer(wl, li, bkw, gpu)
    ctx.close()
# the checks do fire: a dispatch index asked for ids that are out of range
wl = I.WORKLOADS["tiny"]
ctx = P.make_context(wl, 256)
dev = torch.device("cuda")
li = I.make_layer(wl, 0, 0, T=256)
router = B.make_router(li.W.to(dev))
i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
ids, w = i32(256 * wl.k), torch.zeros(256 * wl.k, device=dev)
so, ro, perm, inv, rl = i32(wl.E + 1), i32(wl.R + 1), i32(256 * wl.k), i32(256 * wl.k), i32(wl.R)
bad_pi = torch.tensor([0, 1, 2, 3, 4, 5, 6, 99], dtype=torch.int32, device=dev)   # a slot outside [0, E)
ctx.fb_route_dispatch(router, li.H.to(dev), 256, bad_pi, ids, w, so, ro, perm, inv, rl)
st = ctx.fb_device_status()
assert st in (B.FB_ERR_BAD_PLACEMENT, B.FB_ERR_INTERNAL), st
assert ctx.fb_device_status() == 0
ctx.close()
print("debug build ok")
'''


def test_debug_build_checks_stay_silent_on_valid_runs_and_fire_on_bad_input():
    proc = subprocess.run([sys.executable, "-c", CHILD, ROOT], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert proc.returncode == 0, proc.stdout[-2000:] + proc.stderr[-4000:]
    assert "debug build ok" in proc.stdout
