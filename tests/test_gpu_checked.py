"""The small parity cases once more under the CHECKED build of the library (libgptq2d_checked.so,
-DGPTQ2D_CHECKED): every index that feeds a shared- or global-memory access of the tiled sweep, of its
DMMA tile loop and of the blocked sweep is range-checked on the device, and a violation comes back through
the status words as GPTQ2D_ERR_CHECK (nothing traps).  compute-sanitizer is not available where this library
is developed; this is its stand-in.  Runs in a process of its own so that the two builds never share one."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import sys
sys.path.insert(0, %r)
sys.path.insert(0, %r)
import numpy as np, torch
import oracle as O
from oracle import cref
from certify import certified_case
from paper_2607_27042_b200 import gptq2d as g, workloads as W
assert g.library_path().endswith("libgptq2d_checked.so")
# the check itself: a deliberately bad index must be recorded (status 10, site, index, limit) and redirected to 0
probe = torch.full((5,), -1, dtype=torch.int32, device="cuda")
g.gptq2d_internal_test_hook(5, probe.data_ptr())
torch.cuda.synchronize()
assert probe.cpu().tolist() == [10, 999, 7, 3, 0], probe.cpu().tolist()

def draw(m, n):
    def d(seed):
        X, A, B = W.general_bases(m, n, seed)
        L, U, _, _ = O.feedback_factors(A, B)
        return X, L, U
    return d

cases = []
for k, (m, n) in enumerate([(1, 1), (17, 5), (65, 63), (129, 257), (200, 75), (257, 130), (300, 515), (3, 700)]):
    (X, L, U), ref, _ = certified_case(draw(m, n), cref.nested, 50 + k)
    dX, dL, dU = (torch.from_numpy(a).cuda() for a in (X, L, U))
    Z, E, mm, info = g.gptq2d_round(dX, dL, dU, want_E=True, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)                                   # raises on GPTQ2D_ERR_CHECK (status 10)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"]), (m, n)
    for w in (17, 64):
        Zb, _, _, ib = g.gptq2d_round_blocked(dX, dL, dU, w)
        torch.cuda.synchronize()
        g.check_info(ib)
        assert np.array_equal(Zb.cpu().numpy().astype(np.int64), ref["Z"]), (m, n, w)
    cases.append((dX, dL, dU, ref["Z"]))
Zs, _, _, info = g.gptq2d_round_batched([c[0] for c in cases], [c[1] for c in cases], [c[2] for c in cases])
torch.cuda.synchronize()
g.check_info(info)
for z, c in zip(Zs, cases):
    assert np.array_equal(z.cpu().numpy().astype(np.int64), c[3])
hX, hL, hU = (c.cpu().pin_memory() for c in cases[6][:3])
hZ, hinfo = g.gptq2d_round_host(hX, hL, hU)
assert np.array_equal(hZ.numpy().astype(np.int64), cases[6][3])
print("checked build: %%d cases clean" %% len(cases))
"""


def test_small_parity_cases_under_the_checked_build():
    from paper_2607_27042_b200 import build
    build.build(checked=True)                                # no-op when the library is already there
    env = dict(os.environ, GPTQ2D_LIBRARY="libgptq2d_checked.so")
    r = subprocess.run([sys.executable, "-c", SCRIPT % (ROOT, os.path.join(ROOT, "tests"))], env=env, capture_output=True,
                       text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "cases clean" in r.stdout
