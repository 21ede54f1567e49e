"""The checked build of the library (the same sources compiled with -DKIMAD_CHECKED): index tests that set a status
word instead of trapping, and canary words between the workspace regions.  A selection of the parity tests runs
against it in a child process (the library is chosen when the binding loads it); every comparison with the oracle
there also asks kimad_debug_check for a clean status word and intact canaries."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2312_08053_b200 import build as kbuild

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run_checked(code_or_args, is_code):
    kbuild.build(checked=True)
    env = dict(os.environ, KIMAD_CHECKED="1")
    cmd = [sys.executable, "-c", code_or_args] if is_code else [sys.executable, "-m", "pytest", "-x", "-q"] + code_or_args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_parity_selection_under_the_checked_build():
    sel = ("cfg1 or cfg2 or cfg3 or cfg4 or adversarial or unaligned or concentrated or interface_limits or "
           "randomized_configurations or huge_dynamic or fitted_ratio_matches or dense_fallback_matches or "
           "exact_radix_everywhere or paper_grid or row_sparse or loose_candidates or thresholds_among_zeros or "
           "window_wider")
    res = _run_checked(["tests/test_gpu_parity.py", "tests/test_gpu_policies.py", "tests/test_gpu_tables.py", "-k", sel],
                       is_code=False)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout and "failed" not in res.stdout


def test_a_damaged_canary_is_reported():
    """The failure is made on the host: one byte of a canary is overwritten through the workspace tensor."""
    code = r'''
import numpy as np, torch
from paper_2312_08053_b200 import binding as kb
ctx = kb.new_context([5000, 17, 70000], 2, [0.01, 0.1, 1.0])
out = kb.Packed(ctx)
g = torch.randn((2, 75017), device="cuda")
kb.kimad_step(ctx, g, torch.zeros_like(g), [1e5, 2e5], 1.0, out)
assert kb.kimad_debug_check(ctx) == (True, 0, 0)
ws = ctx._keep[0]
host = ws.cpu().numpy()
blocks = host[: host.size // 256 * 256].reshape(-1, 256)
guards = np.nonzero((blocks == 0xA5).all(axis=1))[0]
assert guards.size > 20
ws[int(guards[7]) * 256 + 3] = 0
torch.cuda.synchronize()
checked, failed, damaged = kb.kimad_debug_check(ctx)
assert (checked, failed, damaged) == (True, 0, 1), (checked, failed, damaged)
print("canary ok")
'''
    res = _run_checked(code, is_code=True)
    assert res.returncode == 0 and "canary ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_ordinary_build_reports_that_it_is_not_checked():
    from paper_2312_08053_b200 import binding as kb

    if os.environ.get("KIMAD_CHECKED") == "1":
        pytest.skip("this process runs the checked build")
    ctx = kb.new_context([100], 1, [1.0])
    assert kb.kimad_debug_check(ctx) == (False, 0, 0)
