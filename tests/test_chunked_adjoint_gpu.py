"""LORY_FLAG_CHUNKED_ADJOINT: the backward that forms the per-segment weight gradients one parameter rectangle at a
time in an L2-sized buffer.  It must give what the default backward gives: the expert gradients bit for bit (the same
products over the same operands), the routing gradient and what follows from it up to fp32 summation order; and it
is held to the oracle like every other path."""
import numpy as np
import pytest
import torch

import paper_2405_03133_b200 as lory
from oracle import lory_oracle as O
from paper_2405_03133_b200.workloads import CONFIGS, Workload, make_inputs

from gpu_util import max_rel, run_layer

pytestmark = pytest.mark.gpu
TOL = 2e-2

CASES = [
    # three row rectangles of W1/W3 (f = 688), two column rectangles of W2 under the 1 MB budget
    Workload("chunk_rows_and_cols", B=2, L=512, T=256, d=256, f=688, E=8, w_r_std=1.0),
    # matrices smaller than one rectangle, ragged widths, single-CTA tiles
    Workload("chunk_small", B=2, L=192, T=64, d=72, f=200, E=5, w_r_std=2.0),
    # more than 32 experts, more than 256 segments (two adjoint launches per rectangle)
    Workload("chunk_520_segments_40_experts", B=13, L=640, T=16, d=64, f=328, E=40, w_r_std=1.0),
]


def oracle_all(wl, inp):
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y, w, p = O.forward(*a)
    return dict(y=y, route_w=w, route_p=p, **O.backward(*a, inp["dy"]))


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_chunked_adjoint_small(wl, monkeypatch):
    monkeypatch.setenv("LORY_ADJOINT_CHUNK_MB", "1")
    inp = make_inputs(wl)
    ref = oracle_all(wl, inp)
    plain = run_layer(wl, inp)
    got = run_layer(wl, inp, flags=lory.LORY_FLAG_CHUNKED_ADJOINT)
    assert got["launches_bwd"] > plain["launches_bwd"]          # it really took the rectangle-by-rectangle route
    for k in ("dW1", "dW2", "dW3"):
        assert np.array_equal(got[k], plain[k]), k
    # the routing gradient is summed in another order: fp32 noise there, at most one bf16 rounding step (2^-7 of the value) in
    # what is stored in bf16 behind it
    assert max_rel(got["d_route_w"], plain["d_route_w"]) <= 1e-4
    for k in ("dx", "dw_r"):
        assert max_rel(got[k], plain[k]) <= 2.0 ** -7, k
    errs = {k: max_rel(got[k], ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= (1e-5 if k.startswith("route_") else TOL)}
    assert not bad, f"{wl.name}: {bad}"


def test_chunked_adjoint_workspace_is_smaller():
    wl = CONFIGS["C3"]
    d0 = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype, 0)
    d1 = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype, lory.LORY_FLAG_CHUNKED_ADJOINT)
    f0, b0 = lory.lory_moe_workspace_bytes(d0)
    f1, b1 = lory.lory_moe_workspace_bytes(d1)
    assert f0 == f1
    # the three per-segment gradient matrices (3 * S * f * d bf16 = 2.16 GB) give way to one L2-sized buffer
    assert b0 - b1 > 2.0e9


def test_chunked_adjoint_accumulates():
    wl = Workload("chunk_accumulate", B=2, L=256, T=64, d=64, f=328, E=6, w_r_std=1.0, seed=5)
    inp = make_inputs(wl)
    base = run_layer(wl, inp, flags=lory.LORY_FLAG_CHUNKED_ADJOINT)
    # second pass adds to gradients that start at the first pass's values
    dims = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype,
                          lory.LORY_FLAG_CHUNKED_ADJOINT | lory.LORY_FLAG_ACCUMULATE_GRADS)
    dev = {k: torch.from_numpy(np.ascontiguousarray(inp[k])).to("cuda", torch.bfloat16) for k in ("x", "w_r", "W1", "W2", "W3", "dy")}
    _, bwd = lory.lory_moe_workspace_bytes(dims)
    ws = torch.empty(bwd, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(dev["x"])
    rw = torch.empty((wl.S, wl.E), dtype=torch.float32, device="cuda")
    lory.lory_moe_forward(dims, dev["x"], dev["w_r"], dev["W1"], dev["W2"], dev["W3"], y, rw, None, ws)
    g = {k: torch.from_numpy(base[k]).to("cuda", torch.bfloat16) for k in ("dw_r", "dW1", "dW2", "dW3")}
    dx = torch.empty_like(dev["x"])
    lory.lory_moe_backward(dims, dev["x"], dev["w_r"], dev["W1"], dev["W2"], dev["W3"], dev["dy"], dx, g["dw_r"],
                           g["dW1"], g["dW2"], g["dW3"], None, ws)
    lory.lory_check_status(dims, ws)
    for k in g:
        assert max_rel(g[k].double().cpu().numpy(), 2.0 * base[k]) <= 1e-2, k


def test_chunked_adjoint_full_size_matches_default():
    """C3 in the launch configuration bench.py times: expert gradients bit for bit, the rest to summation order."""
    wl = CONFIGS["C3"]
    inp = make_inputs(wl)
    plain = run_layer(wl, inp, keep_device=True)
    keep = {k: plain[k].clone() for k in ("dW1", "dW2", "dW3", "dx", "dw_r", "d_route_w")}
    del plain
    got = run_layer(wl, inp, flags=lory.LORY_FLAG_CHUNKED_ADJOINT, keep_device=True)
    for k in ("dW1", "dW2", "dW3"):
        assert torch.equal(got[k], keep[k]), k
    for k, tol in (("dx", 2.0 ** -7), ("dw_r", 2.0 ** -7), ("d_route_w", 1e-4)):
        ref = keep[k].double()
        assert float((got[k].double() - ref).abs().max() / ref.abs().max()) <= tol, k
