"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.
The CPU oracle cannot keep whole layers of this size in memory, so it works segment by segment.
At configurations 2, 3 and 4 and at both ends of the segment-length sweep it visits EVERY segment: dx, the routing gradient d_route_w and the router gradient dW_r are compared in full, the
expert gradients on slices through both of their dimensions, y on segments drawn over the whole batch.
The other configurations compare sampled segments and slices.  Routing tables are always compared in full.
bf16 tolerance: max|diff|/max|ref| <= 2e-2 per compared block; routing tables (fp32): 1e-5."""
import numpy as np
import pytest

from oracle import lory_oracle as O
from paper_2405_03133_b200.workloads import CONFIGS, make_inputs

from gpu_util import max_rel, run_layer

pytestmark = pytest.mark.gpu
TOL = 2e-2
ROUTE_TOL = 1e-5

_cache = {}


def inputs_for(wl):
    """The C5 sweep shares one set of tensors: only the segment length changes."""
    key = (wl.B, wl.L, wl.d, wl.f, wl.E, wl.seed, wl.dtype)
    if key not in _cache:
        _cache.clear()
        _cache[key] = make_inputs(wl)
    return _cache[key]


def sample_segments(wl, n_random, seed):
    """First and last segment of the batch, the first shifted one, and n_random more drawn over all of them
    (late tile-scheduler groups included)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    segs = {0, 1, wl.S - 1}
    segs.update(int(s) for s in rng.integers(0, wl.S, size=n_random))
    return sorted(segs)


def check_routing(wl, inp, got, errs):
    h_bar, p, w = O.route(inp["x"], inp["w_r"], wl.T)
    errs["route_w"] = max_rel(got["route_w"], w)
    errs["route_p"] = max_rel(got["route_p"], p)
    np.testing.assert_allclose(got["route_w"].sum(1), 1.0, atol=1e-5)
    return h_bar, p


def check_frows(wl, inp, got, a, errs):
    # expert weight gradients: a few FFN-hidden indices (rows of dW1/dW3, columns of dW2), all experts
    rows = [0, wl.f // 2 + 3, wl.f - 1]
    dW1r, dW2c, dW3r = O.backward_frows(*a, inp["dy"], rows)
    errs["dW1[rows]"] = max_rel(got["dW1"][:, rows, :], dW1r)
    errs["dW3[rows]"] = max_rel(got["dW3"][:, rows, :], dW3r)
    errs["dW2[cols]"] = max_rel(got["dW2"][:, :, rows], dW2c)


def finish(wl, errs):
    bad = {k: v for k, v in errs.items() if not v <= (ROUTE_TOL if k.startswith("route_") else TOL)}
    print(wl.name, {k: f"{v:.2e}" for k, v in errs.items()})
    assert not bad, f"{wl.name}: over tolerance: {bad}"


def check_sampled(wl):
    inp = inputs_for(wl)
    got = run_layer(wl, inp)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    N, S, T, d = wl.N, wl.S, wl.T, wl.d
    errs = {}
    h_bar, p = check_routing(wl, inp, got, errs)
    segs = sample_segments(wl, 2, seed=wl.T)
    y_gpu = got["y"].reshape(S, T, d)
    for s, y_s in O.forward_segments(*a, segs).items():
        errs[f"y[{s}]"] = max_rel(y_gpu[s], y_s)
    # backward: dx of segment s needs dw of segment s+1 for its router term; one early and one late segment
    for s0 in (1, S - 2 if (S - 2) % N < N - 1 else S - 3):
        bs = O.backward_segments(*a, inp["dy"], [s0, s0 + 1])
        dw = np.zeros((S, wl.E))
        dw[s0 + 1] = bs[s0 + 1][1]
        dx_router, _ = O.router_backward(inp["x"].shape, T, h_bar, p, inp["w_r"], dw)
        dx_ref = bs[s0][0] + dx_router.reshape(S, T, d)[s0]
        errs[f"dx[{s0}]"] = max_rel(got["dx"].reshape(S, T, d)[s0], dx_ref)
        for s in (s0, s0 + 1):
            errs[f"d_route_w[{s}]"] = max_rel(got["d_route_w"][s], bs[s][1])
    check_frows(wl, inp, got, a, errs)
    # a property that holds at any size: the softmax backward makes the router gradient sum to zero over experts
    assert np.abs(got["dw_r"].sum(0)).max() <= 2e-2 * max(np.abs(got["dw_r"]).max(), 1e-30)
    finish(wl, errs)


def check_every_segment(wl):
    inp = inputs_for(wl)
    got = run_layer(wl, inp)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    S, T, d = wl.S, wl.T, wl.d
    errs = {}
    h_bar, p = check_routing(wl, inp, got, errs)
    y_gpu = got["y"].reshape(S, T, d)
    for s, y_s in O.forward_segments(*a, sample_segments(wl, 6, seed=7)).items():
        errs[f"y[{s}]"] = max_rel(y_gpu[s], y_s)
    d_rows = [0, d // 2 + 5, d - 1]
    dx_ffn, dw, dW2r, dW1c, dW3c = O.backward_every_segment(*a, inp["dy"], d_rows)
    dx_router, dW_r = O.router_backward(inp["x"].shape, T, h_bar, p, inp["w_r"], dw)
    errs["d_route_w"] = max_rel(got["d_route_w"], dw)
    errs["dw_r"] = max_rel(got["dw_r"], dW_r)
    errs["dx"] = max_rel(got["dx"], dx_ffn.reshape(wl.B, wl.L, d) + dx_router)
    dx_gpu, dx_ref = got["dx"].reshape(S, T, d), dx_ffn + dx_router.reshape(S, T, d)
    errs["dx[worst segment]"] = max(max_rel(dx_gpu[s], dx_ref[s]) for s in range(S))
    errs["dW2[d rows]"] = max_rel(got["dW2"][:, d_rows, :], dW2r)
    errs["dW1[d cols]"] = max_rel(got["dW1"][:, :, d_rows], dW1c)
    errs["dW3[d cols]"] = max_rel(got["dW3"][:, :, d_rows], dW3c)
    check_frows(wl, inp, got, a, errs)
    finish(wl, errs)


@pytest.mark.parametrize("name", ["C2", "C3", "C4"])
def test_full_size_every_segment(name):
    check_every_segment(CONFIGS[name])


@pytest.mark.parametrize("T", [64, 128, 256, 512, 1024])
def test_full_size_segment_length_sweep(T):
    # the two ends of the sweep (most segments, longest segments) visit every segment, the rest are sampled
    (check_every_segment if T in (64, 1024) else check_sampled)(CONFIGS[f"C5_T{T}"])
