"""lory_route_noalloc: the routing step for callers that cannot allocate device memory (serving
plug-ins and control loops whose memory was handed out at start-up, hosts that pass only input and
output pointers).  Its scratch is a fixed array inside the library, shared by every call, so the
test runs two different problems back to back.  Each is checked twice: against the routing tables
of the ordinary workspace-based forward (the same kernels on other scratch memory, so the tables
must be bit-identical) and against the CPU oracle's routing step."""
import numpy as np
import pytest
import torch

import paper_2405_03133_b200 as lory
from oracle import lory_oracle as O
from paper_2405_03133_b200.workloads import Workload, make_inputs

from gpu_util import max_rel, to_dev

pytestmark = pytest.mark.gpu

ROUTE_TOL = 1e-5   # the routing tables are fp32 in either mode


def routing_both_ways(wl, flags=0):
    inp = make_inputs(wl)
    dims = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype, flags)
    x, w_r, W1, W2, W3 = (to_dev(inp[k], wl) for k in ("x", "w_r", "W1", "W2", "W3"))
    S = wl.S
    # existing entry point
    fwd_b, _ = lory.lory_moe_workspace_bytes(dims)
    ws = torch.empty(fwd_b, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    rw_ref = torch.empty((S, wl.E), dtype=torch.float32, device="cuda")
    rp_ref = torch.empty_like(rw_ref)
    lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, rw_ref, rp_ref, ws)
    # entry point under test: outputs pre-filled with NaN so that an unwritten element shows
    rw = torch.full((S, wl.E), float("nan"), dtype=torch.float32, device="cuda")
    rp = torch.full_like(rw, float("nan"))
    lory.lory_route_noalloc(dims, x, w_r, rw, rp)
    torch.cuda.synchronize()
    _, p_o, w_o = O.route(inp["x"], inp["w_r"], wl.T)
    return (rw.cpu().numpy(), rp.cpu().numpy()), (rw_ref.cpu().numpy(), rp_ref.cpu().numpy()), (w_o, p_o)


def check(wl, flags=0):
    (rw, rp), (rw_ref, rp_ref), (w_o, p_o) = routing_both_ways(wl, flags)
    assert np.array_equal(rw, rw_ref) and np.array_equal(rp, rp_ref), "differs from the workspace path"
    assert max_rel(rw, w_o) <= ROUTE_TOL
    assert max_rel(rp, p_o) <= ROUTE_TOL
    np.testing.assert_allclose(rw.sum(1), 1.0, atol=1e-5)


def test_two_calls_in_a_row_match_the_workspace_path_and_the_oracle():
    first = Workload("noalloc_a", B=3, L=256, T=32, d=64, f=64, E=5, dtype="bf16", w_r_std=2.0, seed=3)
    second = Workload("noalloc_b", B=2, L=64, T=16, d=40, f=16, E=3, dtype="fp32", w_r_std=1.0, seed=4)
    for wl in (first, second):          # the second call finds the first call's leftovers in the scratch
        check(wl)


def test_problem_that_fills_the_scratch_exactly():
    # S * (d + E) * 4 bytes = 1024 * (1016 + 8) * 4 = 4 MiB: the last float of the array is in use
    wl = Workload("noalloc_full", B=4, L=512, T=2, d=1016, f=8, E=8, dtype="bf16", w_r_std=1.0, seed=5)
    assert (wl.S * wl.d + wl.S * wl.E) * 4 == lory.binding.LORY_NOALLOC_SCRATCH_BYTES
    # (the reference forward runs its FFN part on the plain-FMA pipeline: only the routing step is compared)
    check(wl, lory.binding.LORY_FLAG_SIMT)


def test_one_element_more_is_refused():
    # 1025 segments: one segment (1024 floats) beyond the array; refused before anything is launched
    dims = lory.make_dims(1025, 2, 2, 1016, 8, 8, "bf16")
    dummy = torch.zeros(16, device="cuda")
    with pytest.raises(lory.LoryError) as err:
        lory.lory_route_noalloc(dims, dummy, dummy, dummy, None)
    assert err.value.status == -8
    # the same width with one expert more: S * (d + E) * 4 exceeds the array by 4 KiB
    dims = lory.make_dims(4, 512, 2, 1016, 8, 9, "bf16")
    with pytest.raises(lory.LoryError) as err:
        lory.lory_route_noalloc(dims, dummy, dummy, dummy, None)
    assert err.value.status == -8


def test_rejects_problems_beyond_the_fixed_scratch():
    # S*d floats alone exceed the 4 MiB array: must be refused before anything is launched
    dims = lory.make_dims(64, 4096, 64, 2048, 64, 8, "bf16")
    dummy = torch.zeros(16, device="cuda")
    with pytest.raises(lory.LoryError) as err:
        lory.lory_route_noalloc(dims, dummy, dummy, dummy, None)
    assert err.value.status == -8
    assert "scratch" in str(err.value)
