"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element,
on the same seeded inputs.  Tolerances: fp32 mode max|diff|/max|ref| <= 1e-4 per tensor,
bf16 mode <= 2e-2 per tensor; the routing tables are fp32 in either mode and are held to 1e-5."""
import numpy as np
import pytest

from oracle import lory_oracle as O
from paper_2405_03133_b200 import LORY_FLAG_SIMT
from paper_2405_03133_b200.workloads import CONFIGS, Workload, make_inputs

from gpu_util import max_rel, run_layer

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "bf16": 2e-2}
ALL_KEYS = ["y", "route_w", "route_p", "dx", "dw_r", "dW1", "dW2", "dW3", "d_route_w"]


def oracle_all(wl, inp):
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y, w, p = O.forward(*a)
    g = O.backward(*a, inp["dy"])
    return dict(y=y, route_w=w, route_p=p, **g)


ROUTE_TOL = 1e-5   # route_w, route_p: fp32 sums and an fp32 softmax whatever the storage type


def compare(wl, got, ref, tol, keys=None):
    errs = {k: max_rel(got[k], ref[k]) for k in (keys or ALL_KEYS)}
    bad = {k: v for k, v in errs.items() if not v <= (min(tol, ROUTE_TOL) if k in ("route_w", "route_p") else tol)}
    assert not bad, f"{wl.name}: over tolerance {tol}: {bad} (all: {errs})"
    return errs


SMALL = [
    Workload("tiny_fp32", B=2, L=64, T=16, d=32, f=48, E=3, dtype="fp32", w_r_std=1.0),
    Workload("ragged_fp32", B=3, L=40, T=8, d=24, f=52, E=5, dtype="fp32", w_r_std=3.0),
    Workload("one_expert_fp32", B=1, L=32, T=16, d=16, f=16, E=1, dtype="fp32"),
    Workload("one_segment_fp32", B=2, L=16, T=16, d=16, f=24, E=4, dtype="fp32", w_r_std=2.0),
    Workload("tiny_bf16_simt", B=2, L=64, T=16, d=32, f=48, E=3, dtype="bf16", w_r_std=1.0),
]


@pytest.mark.parametrize("wl", SMALL, ids=lambda w: w.name)
def test_small_cases_simt(wl):
    inp = make_inputs(wl)
    ref = oracle_all(wl, inp)
    got = run_layer(wl, inp, flags=LORY_FLAG_SIMT if wl.dtype == "bf16" else 0)
    compare(wl, got, ref, TOL[wl.dtype])


def test_config1_fp32():
    wl = CONFIGS["C1"]
    inp = make_inputs(wl)
    ref = oracle_all(wl, inp)
    got = run_layer(wl, inp)
    errs = compare(wl, got, ref, TOL["fp32"])
    print("C1 errors", errs)


def test_config1_sharp_router_fp32():
    wl = CONFIGS["C1"].with_(name="C1_sharp", w_r_std=2.0, seed=1)
    inp = make_inputs(wl)
    ref = oracle_all(wl, inp)
    assert ref["route_w"].max() > 0.9          # far from uniform
    got = run_layer(wl, inp)
    compare(wl, got, ref, TOL["fp32"])


# ---- bf16 tensor-core path ---------------------------------------------------------------------
TC_SMALL = [
    # several N tiles with a ragged tail (f = 136), one K block
    Workload("tc_tails", B=2, L=256, T=128, d=64, f=136, E=3, w_r_std=1.0),
    # segment shorter than the 128-row tile, K tail (d = 72), E not a multiple of 8
    Workload("tc_short_segment", B=2, L=192, T=64, d=72, f=200, E=5, w_r_std=2.0),
    # two M tiles per segment, several K blocks, E = 8
    Workload("tc_two_m_tiles", B=2, L=512, T=256, d=256, f=688, E=8, w_r_std=1.0),
    # one expert, one segment per sequence
    Workload("tc_one_expert", B=2, L=128, T=128, d=64, f=64, E=1),
    # more than 128 segments (two M tiles in the merge), T = 32
    Workload("tc_many_segments", B=5, L=1024, T=32, d=64, f=72, E=4, w_r_std=1.0),
    # more than 32 experts (hi and lo sums in separate accumulator halves), E not a multiple of 16
    Workload("tc_40_experts", B=2, L=256, T=64, d=64, f=136, E=40, w_r_std=1.0),
    # the largest expert count of the tensor-core path
    Workload("tc_64_experts", B=3, L=192, T=64, d=128, f=72, E=64, w_r_std=2.0),
    # 17..32 experts, between 64 and 128 segments
    Workload("tc_24_experts_80_segments", B=5, L=512, T=32, d=64, f=72, E=24, w_r_std=1.0),
    # exactly 64 and 65 segments: either side of the merge's small-S arrangement
    Workload("tc_64_segments", B=4, L=512, T=32, d=64, f=72, E=7, w_r_std=1.0),
    Workload("tc_65_segments", B=5, L=416, T=32, d=64, f=72, E=33, w_r_std=1.0),
    # more than 256 segments: the merge and its adjoint take one launch per 256 segments, later launches of the
    # adjoint adding to the expert gradients of the earlier ones (288 = 256 + 32; 520 = 2 * 256 + 8, > 32 experts)
    # segment lengths that are no multiple of 16, 32 or 64 (the contraction length of the weight-gradient GEMMs)
    Workload("tc_T100", B=2, L=300, T=100, d=64, f=72, E=4, w_r_std=1.0),
    Workload("tc_T24_T_smaller_than_a_k_block", B=3, L=96, T=24, d=136, f=64, E=6, w_r_std=1.0),
    Workload("tc_T1", B=2, L=6, T=1, d=64, f=64, E=3, w_r_std=1.0),
    # weight-gradient kernel with a resident operand (CTA-pair tiles, T <= 128): contraction tails (T = 100: two token
    # blocks, the second ragged; T = 24: one), a second row tile that is almost empty (d = 264), and enough segments
    # that every CTA pair takes several strips and both resident buffers change phase (400 segments, 74 pairs)
    Workload("tc_wgrad_resident_T100", B=2, L=300, T=100, d=256, f=328, E=4, w_r_std=1.0),
    Workload("tc_wgrad_resident_T24", B=3, L=96, T=24, d=264, f=256, E=6, w_r_std=1.0),
    Workload("tc_wgrad_resident_400_segments", B=25, L=512, T=32, d=256, f=328, E=4, w_r_std=1.0),
    Workload("tc_288_segments", B=9, L=1024, T=32, d=64, f=72, E=4, w_r_std=1.0),
    Workload("tc_520_segments_40_experts", B=13, L=640, T=16, d=64, f=72, E=40, w_r_std=1.0),
]


@pytest.mark.parametrize("wl", TC_SMALL, ids=lambda w: w.name)
def test_small_cases_tensor_core(wl):
    inp = make_inputs(wl)
    ref = oracle_all(wl, inp)
    got = run_layer(wl, inp)
    errs = compare(wl, got, ref, TOL["bf16"])
    print(wl.name, errs)


def test_tensor_core_matches_plain_fma_path():
    """Same bf16 inputs through both pipelines: they round the same intermediates to bf16,
    so they must agree much more tightly than either agrees with the oracle."""
    wl = Workload("tc_vs_simt", B=2, L=512, T=128, d=128, f=328, E=6, w_r_std=1.0)
    inp = make_inputs(wl)
    a = run_layer(wl, inp)
    b = run_layer(wl, inp, flags=LORY_FLAG_SIMT)
    for k in ALL_KEYS:
        assert max_rel(a[k], b[k]) < 1e-2, k


def test_injected_one_hot_weights_select_expert_tensor_core():
    wl = Workload("tc_one_hot", B=2, L=256, T=128, d=64, f=136, E=4)
    inp = make_inputs(wl)
    pick = np.arange(wl.S) % wl.E
    w = np.eye(wl.E)[pick]
    seg_x = inp["x"].reshape(wl.S, wl.T, wl.d)
    ref = O.moe_ffn(seg_x, w, inp["W1"], inp["W2"], inp["W3"]).reshape(wl.B, wl.L, wl.d)
    got = run_layer(wl, inp, injected_w=w)
    assert max_rel(got["y"], ref) <= TOL["bf16"]


def test_step_host_matches_separate_calls():
    """lory_moe_step_host (host activations, copies overlapped with compute) must return exactly what
    lory_moe_forward + lory_moe_backward return for the same inputs."""
    import torch
    import paper_2405_03133_b200 as lory
    from gpu_util import to_dev
    wl = Workload("step_host", B=2, L=512, T=256, d=128, f=328, E=6, w_r_std=1.0)
    inp = make_inputs(wl)
    ref = run_layer(wl, inp, keep_device=True)
    dims = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype)
    w_r, W1, W2, W3 = (to_dev(inp[k], wl) for k in ("w_r", "W1", "W2", "W3"))
    xh = torch.from_numpy(inp["x"]).to(torch.bfloat16).pin_memory()
    dyh = torch.from_numpy(inp["dy"]).to(torch.bfloat16).pin_memory()
    yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
    rwh = torch.empty((wl.S, wl.E), dtype=torch.float32).pin_memory()
    dw_r, dW1, dW2, dW3 = (torch.empty_like(t) for t in (w_r, W1, W2, W3))
    arena = torch.empty(lory.lory_moe_step_host_bytes(dims), dtype=torch.uint8, device="cuda")
    for _ in range(2):      # the second call reuses the arena and the internal copy stream
        yh.zero_(); dxh.zero_()
        lory.lory_moe_step_host(dims, xh, dyh, w_r, W1, W2, W3, yh, dxh, rwh, dw_r, dW1, dW2, dW3, arena)
        assert torch.equal(yh, ref["y"].cpu())
        assert torch.equal(dxh, ref["dx"].cpu())
        assert torch.equal(rwh, ref["route_w"].cpu())
        assert torch.equal(dW2.cpu(), ref["dW2"].cpu())
        assert torch.equal(dw_r.cpu(), ref["dw_r"].cpu())


def test_step_host_pipeline_matches_separate_calls():
    """The two-slot pipeline (copies of neighbouring steps overlapping the kernels) over five steps with
    different inputs: every step must return exactly what forward + backward return for its inputs."""
    import torch
    import paper_2405_03133_b200 as lory
    from gpu_util import to_dev
    base = Workload("step_pipe", B=2, L=512, T=256, d=128, f=328, E=6, w_r_std=1.0)
    dims = lory.make_dims(base.B, base.L, base.T, base.d, base.f, base.E, base.dtype)
    inp0 = make_inputs(base)
    w_r, W1, W2, W3 = (to_dev(inp0[k], base) for k in ("w_r", "W1", "W2", "W3"))
    steps = 5
    refs, xs, dys = [], [], []
    for i in range(steps):
        inp = dict(inp0)
        other = make_inputs(base.with_(seed=100 + i))
        inp["x"], inp["dy"] = other["x"], other["dy"]
        refs.append(run_layer(base, inp, keep_device=True))
        xs.append(torch.from_numpy(inp["x"]).to(torch.bfloat16).pin_memory())
        dys.append(torch.from_numpy(inp["dy"]).to(torch.bfloat16).pin_memory())
    yh = [torch.zeros_like(xs[0]).pin_memory() for _ in range(2)]
    dxh = [torch.zeros_like(xs[0]).pin_memory() for _ in range(2)]
    rwh = [torch.zeros((base.S, base.E), dtype=torch.float32).pin_memory() for _ in range(2)]
    dw_r, dW1, dW2, dW3 = (torch.empty_like(t) for t in (w_r, W1, W2, W3))
    arena = torch.empty(lory.lory_moe_step_host_pipeline_bytes(dims), dtype=torch.uint8, device="cuda")

    def check(i):
        slot = i & 1
        lory.lory_moe_step_host_wait(slot)
        assert torch.equal(yh[slot], refs[i]["y"].cpu()), i
        assert torch.equal(dxh[slot], refs[i]["dx"].cpu()), i
        assert torch.equal(rwh[slot], refs[i]["route_w"].cpu()), i

    for i in range(steps):
        slot = i & 1
        if i >= 2:
            check(i - 2)            # the slot is free again only after its outputs were awaited
        lory.lory_moe_step_host_enqueue(dims, slot, xs[i], dys[i], w_r, W1, W2, W3, yh[slot], dxh[slot], rwh[slot],
                                        dw_r, dW1, dW2, dW3, arena)
    check(steps - 2)
    check(steps - 1)
    torch.cuda.synchronize()
    assert torch.equal(dW2.cpu(), refs[-1]["dW2"].cpu())   # parameter gradients are those of the last step
    with pytest.raises(lory.LoryError):
        lory.lory_moe_step_host_enqueue(dims, 2, xs[0], dys[0], w_r, W1, W2, W3, yh[0], dxh[0], rwh[0],
                                        dw_r, dW1, dW2, dW3, arena)
