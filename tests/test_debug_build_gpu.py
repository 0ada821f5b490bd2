"""The bounds-checking build of the library (-DLORY_DEBUG, liblory_debug.so): its kernels check every tile
coordinate, shared-memory stage and TMEM column range before use.  The small tensor-core parity cases must pass
under it with no check firing, and its self-test must make the checks fire without a fault.

A process can hold only one build of the library behind the binding, so the debug build runs in child
processes that select it with LORY_LIBRARY."""
import os
import subprocess
import sys

import pytest
import torch

import paper_2405_03133_b200 as lory
from paper_2405_03133_b200 import build as lory_build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def debug_env():
    if not os.path.exists(lory_build.LIB_DEBUG):
        lory_build.build(debug=True)
    env = dict(os.environ)
    env["LORY_LIBRARY"] = lory_build.LIB_DEBUG
    return env


def test_small_tensor_core_cases_pass_under_the_debug_build():
    code = ("import paper_2405_03133_b200 as lory, pytest, sys; assert lory.binding.lory_debug_build() == 1; "
            "sys.exit(pytest.main(['tests/test_parity_gpu.py', '-q', '-x', '-m', 'gpu', '-k', "
            "'small_cases_tensor_core or tensor_core_matches_plain_fma or one_hot', '-p', 'no:cacheprovider']))")
    res = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=debug_env(), capture_output=True, text=True,
                         timeout=1500)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-3000:]
    assert " passed" in res.stdout


SELFTEST = r"""
import torch, paper_2405_03133_b200 as lory
assert lory.binding.lory_debug_build() == 1
dims = lory.make_dims(2, 256, 128, 64, 136, 3, "bf16")
fwd, _ = lory.lory_moe_workspace_bytes(dims)
ws = torch.empty(fwd, dtype=torch.uint8, device="cuda")
lory.binding.lory_selftest_debug_bounds(dims, ws)
try:
    lory.lory_check_status(dims, ws)
    raise SystemExit("the bounds checks did not fire")
except lory.LoryError as e:
    assert e.status == -9, e.status
# the device is still usable and a real call clears the word again
x = torch.randn(2, 256, 64, device="cuda").bfloat16()
w_r = torch.randn(3, 64, device="cuda").bfloat16()
W1 = (0.02 * torch.randn(3, 136, 64, device="cuda")).bfloat16()
W3 = (0.02 * torch.randn(3, 136, 64, device="cuda")).bfloat16()
W2 = (0.02 * torch.randn(3, 64, 136, device="cuda")).bfloat16()
y = torch.empty_like(x)
rw = torch.empty(4, 3, device="cuda")
lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, rw, None, ws)
lory.lory_check_status(dims, ws)
assert torch.isfinite(y.float()).all()
print("selftest ok")
"""


def test_debug_checks_fire_in_the_self_test_without_a_fault():
    res = subprocess.run([sys.executable, "-c", SELFTEST], cwd=ROOT, env=debug_env(), capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "selftest ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_release_build_compiles_the_checks_out():
    assert lory.binding.lory_debug_build() == 0
    dims = lory.make_dims(2, 256, 128, 64, 136, 3, "bf16")
    fwd, _ = lory.lory_moe_workspace_bytes(dims)
    ws = torch.empty(fwd, dtype=torch.uint8, device="cuda")
    lory.binding.lory_selftest_debug_bounds(dims, ws)
    lory.lory_check_status(dims, ws)          # nothing fired: the predicates are constant-true in this build
