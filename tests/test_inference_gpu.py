"""GPU parity for the inference modes: prompt-only routing with a cached merged FFN (Section 3.1,
"Prompt-only routing during inference") and the expert-utilisation count (appendix "Expert Utilization")."""
import numpy as np
import pytest
import torch

import paper_2405_03133_b200 as lory
from oracle import lory_oracle as O
from paper_2405_03133_b200.workloads import Workload, make_inputs, round_to_bf16

from gpu_util import max_rel, tdtype, to_dev

pytestmark = pytest.mark.gpu
TOL = {"fp32": 1e-4, "bf16": 2e-2}


@pytest.mark.parametrize("wl", [
    Workload("prompt_bf16", B=3, L=384, T=384, d=128, f=200, E=6, dtype="bf16", w_r_std=2.0, seed=5),
    Workload("prompt_fp32", B=2, L=40, T=40, d=32, f=48, E=3, dtype="fp32", w_r_std=2.0, seed=6),
    Workload("prompt_bf16_fma", B=2, L=64, T=64, d=32, f=48, E=3, dtype="bf16", w_r_std=2.0, seed=7),
], ids=lambda w: w.name)
def test_prompt_only_routing_then_decode_with_cached_merged_ffn(wl):
    flags = lory.LORY_FLAG_SIMT if wl.name.endswith("fma") else 0
    inp = make_inputs(wl)
    rng = np.random.default_rng(wl.seed + 100)
    news = [rng.standard_normal((wl.B, n, wl.d)).astype(np.float32) for n in (1, 5)]
    if wl.dtype == "bf16":
        news = [round_to_bf16(a) for a in news]
    x, w_r, W1, W2, W3 = (to_dev(inp[k], wl) for k in ("x", "w_r", "W1", "W2", "W3"))
    # prompt pass: one segment per sequence
    dims = lory.make_dims(wl.B, wl.L, wl.L, wl.d, wl.f, wl.E, wl.dtype, flags)
    fwd_b, _ = lory.lory_moe_workspace_bytes(dims)
    ws = torch.empty(fwd_b, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    rw = torch.empty((wl.B, wl.E), dtype=torch.float32, device="cuda")
    lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, rw, None, ws)
    for x_new in news:
        y_ref_prompt, y_ref_new, w_ref = O.prompt_only_inference(inp["x"], x_new, inp["w_r"], inp["W1"], inp["W2"], inp["W3"])
        n = x_new.shape[1]
        xd = to_dev(x_new, wl)
        yd = torch.full_like(xd, float("nan"))
        ddims = lory.make_dims(wl.B, n, n, wl.d, wl.f, wl.E, wl.dtype, flags | lory.LORY_FLAG_REUSE_MERGED)
        lory.lory_moe_ffn(ddims, xd, None, W1, W2, W3, yd, ws)      # no routing weights: the merged FFN is cached
        lory.lory_check_status(dims, ws)
        assert max_rel(yd.double().cpu().numpy(), y_ref_new) <= TOL[wl.dtype]
    assert max_rel(rw.double().cpu().numpy(), w_ref) <= 1e-5
    assert max_rel(y.double().cpu().numpy(), y_ref_prompt) <= TOL[wl.dtype]


def test_forward_rejects_the_reuse_flag():
    dims = lory.make_dims(1, 8, 8, 8, 8, 2, "fp32", lory.LORY_FLAG_REUSE_MERGED)
    t = torch.zeros(64, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(lory.LoryError) as e:
        lory.lory_moe_forward(dims, t, t, t, t, t, t, t, None, ws)
    assert e.value.status == -2


def test_expert_utilization_matches_oracle():
    rng = np.random.default_rng(11)
    for S, E in ((128, 32), (7, 5), (300, 8)):
        z = rng.standard_normal((S, E)) * 2.0
        w = np.exp(z) / np.exp(z).sum(1, keepdims=True)
        wd = torch.from_numpy(w.astype(np.float32)).cuda()
        counts = torch.full((E,), -1, dtype=torch.int32, device="cuda")
        lory.lory_expert_utilization(wd, counts)
        np.testing.assert_array_equal(counts.cpu().numpy(), O.expert_utilization(wd.cpu().numpy()))


@pytest.mark.parametrize("wl", [
    Workload("prefix_bf16", B=2, L=512, T=128, d=64, f=136, E=5, dtype="bf16", w_r_std=2.0, seed=8),
    Workload("prefix_fp32", B=3, L=48, T=8, d=24, f=40, E=4, dtype="fp32", w_r_std=2.0, seed=9),
], ids=lambda w: w.name)
def test_prefix_routing_forward_and_backward(wl):
    """The prefix-routing ablation (Section 5.1) as a flag on the routing step."""
    from gpu_util import run_layer
    inp = make_inputs(wl)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y, w, p = O.forward(*a, prefix=True)
    ref = dict(y=y, route_w=w, route_p=p, **O.backward(*a, inp["dy"], prefix=True))
    got = run_layer(wl, inp, flags=lory.LORY_FLAG_PREFIX_ROUTING)
    w3 = got["route_w"].reshape(wl.B, wl.N, wl.E)
    assert np.all(w3 == w3[:, :1])
    errs = {k: max_rel(got[k], ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= TOL[wl.dtype]}
    assert not bad, (bad, errs)


@pytest.mark.parametrize("wl,prefix", [
    # whole-sequence routing (Section 2.2): one segment per sequence, the router learns from it
    (Workload("sequence_routing_bf16", B=4, L=128, T=128, d=64, f=136, E=5, dtype="bf16", w_r_std=2.0, seed=12), False),
    (Workload("sequence_routing_fp32", B=3, L=16, T=16, d=24, f=40, E=4, dtype="fp32", w_r_std=2.0, seed=13), False),
    # causal routing with several segments, and prefix routing, without the stop-gradient
    (Workload("first_grad_bf16", B=2, L=512, T=128, d=64, f=136, E=5, dtype="bf16", w_r_std=2.0, seed=14), False),
    (Workload("first_grad_prefix_fp32", B=2, L=48, T=8, d=24, f=40, E=4, dtype="fp32", w_r_std=2.0, seed=15), True),
], ids=lambda v: v.name if isinstance(v, Workload) else str(v))
def test_first_segment_gradient_flag(wl, prefix):
    from gpu_util import run_layer
    inp = make_inputs(wl)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y, w, p = O.forward(*a, prefix=prefix)
    ref = dict(y=y, route_w=w, route_p=p, **O.backward(*a, inp["dy"], prefix=prefix, first_grad=True))
    assert np.abs(ref["dw_r"]).max() > 0
    flags = lory.LORY_FLAG_FIRST_SEGMENT_GRAD | (lory.LORY_FLAG_PREFIX_ROUTING if prefix else 0)
    got = run_layer(wl, inp, flags=flags)
    errs = {k: max_rel(got[k], ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= TOL[wl.dtype]}
    assert not bad, (bad, errs)
    if wl.N == 1:
        # with the stop-gradient the router of a one-segment problem receives nothing
        got0 = run_layer(wl, inp)
        assert np.all(got0["dw_r"] == 0.0)


def test_bounded_wait_expires_and_is_reported():
    """Failure detection without a GPU fault: a wait that nothing satisfies runs out of polls, the kernel
    returns normally, the status word reports it, and the device keeps working."""
    dims = lory.make_dims(1, 32, 16, 16, 16, 2, "bf16")
    fwd_b, _ = lory.lory_moe_workspace_bytes(dims)
    ws = torch.zeros(fwd_b, dtype=torch.uint8, device="cuda")
    lory.lory_check_status(dims, ws)                      # clean
    lory.lory_selftest_bounded_wait(dims, ws)
    with pytest.raises(lory.LoryError) as e:
        lory.lory_check_status(dims, ws)
    assert e.value.status == -7
    # the context is intact: a normal forward clears the word and succeeds
    wl = Workload("after_timeout", B=1, L=32, T=16, d=16, f=16, E=2, dtype="bf16")
    inp = make_inputs(wl)
    x, w_r, W1, W2, W3 = (to_dev(inp[k], wl) for k in ("x", "w_r", "W1", "W2", "W3"))
    y = torch.empty_like(x)
    rw = torch.empty((wl.S, wl.E), dtype=torch.float32, device="cuda")
    lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, rw, None, ws)
    lory.lory_check_status(dims, ws)
    assert torch.isfinite(y.float()).all()


@pytest.mark.parametrize("wl,extra_flags", [
    (Workload("accumulate_bf16", B=2, L=512, T=128, d=72, f=200, E=5, dtype="bf16", w_r_std=1.0, seed=21), 0),
    (Workload("accumulate_bf16_40_experts", B=2, L=256, T=64, d=64, f=136, E=40, dtype="bf16", w_r_std=1.0, seed=22), 0),
    (Workload("accumulate_fp32", B=2, L=48, T=8, d=24, f=40, E=4, dtype="fp32", w_r_std=1.0, seed=23), 0),
    (Workload("accumulate_bf16_fma", B=2, L=64, T=16, d=32, f=48, E=3, dtype="bf16", w_r_std=1.0, seed=24), lory.LORY_FLAG_SIMT),
], ids=lambda v: v.name if isinstance(v, Workload) else str(v))
def test_gradient_accumulation_flag(wl, extra_flags):
    """Two micro-batches: the second backward adds its parameter gradients to those the first one left."""
    from gpu_util import to_dev
    inps = [make_inputs(wl), make_inputs(wl.with_(seed=wl.seed + 100))]
    params = {k: to_dev(inps[0][k], wl) for k in ("w_r", "W1", "W2", "W3")}
    fwd_b, bwd_b = lory.lory_moe_workspace_bytes(lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype, extra_flags))
    ws = torch.empty(bwd_b, dtype=torch.uint8, device="cuda")
    grads = {k: torch.full_like(params[k], float("nan")) for k in params}
    ref_sum, ref_each = None, []
    for i, inp in enumerate(inps):
        flags = extra_flags | (lory.LORY_FLAG_ACCUMULATE_GRADS if i > 0 else 0)
        dims = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, wl.dtype, flags)
        x, dy = to_dev(inp["x"], wl), to_dev(inp["dy"], wl)
        y, dx = torch.empty_like(x), torch.empty_like(x)
        rw = torch.empty((wl.S, wl.E), dtype=torch.float32, device="cuda")
        lory.lory_moe_forward(dims, x, params["w_r"], params["W1"], params["W2"], params["W3"], y, rw, None, ws)
        lory.lory_moe_backward(dims, x, params["w_r"], params["W1"], params["W2"], params["W3"], dy, dx,
                               grads["w_r"], grads["W1"], grads["W2"], grads["W3"], None, ws)
        lory.lory_check_status(dims, ws)
        g = O.backward(inp["x"], inps[0]["w_r"], inps[0]["W1"], inps[0]["W2"], inps[0]["W3"], wl.T, inp["dy"])
        ref_each.append(g)
        # dx stays per call
        assert max_rel(dx.double().cpu().numpy(), g["dx"]) <= TOL[wl.dtype]
    names = {"w_r": "dw_r", "W1": "dW1", "W2": "dW2", "W3": "dW3"}
    for k, gk in names.items():
        ref = ref_each[0][gk] + ref_each[1][gk]
        err = max_rel(grads[k].double().cpu().numpy(), ref)
        assert err <= TOL[wl.dtype], (k, err)
        # and it really is the sum, not the second gradient alone
        assert max_rel(grads[k].double().cpu().numpy(), ref_each[1][gk]) > 0.1


@pytest.mark.parametrize("wl,world", [
    (Workload("sharded_bf16", B=2, L=512, T=128, d=72, f=200, E=5, dtype="bf16", w_r_std=2.0, seed=41), 3),
    (Workload("sharded_fp32", B=2, L=48, T=8, d=24, f=40, E=4, dtype="fp32", w_r_std=2.0, seed=42), 2),
], ids=lambda v: v.name if isinstance(v, Workload) else str(v))
def test_expert_sharded_slices_sum_to_the_full_layer(wl, world):
    """Expert-wise model parallelism (Section 6) with the CUDA kernels, the ranks run one after the other on this
    GPU.  The all-reduce is stood in for by what `parallel.torch_all_reduce` does on the wire: every rank's partial
    tensor (in the storage type, bf16 here) is widened to fp32, the fp32 copies are added, and the sum is rounded
    to the storage type once.  The slices' partial y, dx, dW_r must add up to the full layer's (the router path
    included), and the weight-gradient slices must be the matching parts of the full ones."""
    from gpu_util import to_dev
    from paper_2405_03133_b200 import parallel
    inp = make_inputs(wl)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y_ref, w_ref, _ = O.forward(*a)
    g_ref = O.backward(*a, inp["dy"])
    x, w_r, W1, W2, W3, dy = (to_dev(inp[k], wl) for k in ("x", "w_r", "W1", "W2", "W3", "dy"))
    sums = {}

    def collect(name):
        def all_reduce(t):
            sums[name] = sums.get(name, 0) + t.float()          # fp32 accumulation of the ranks' tensors
        return all_reduce

    def landed(name, like):
        return sums[name].to(like.dtype).double().cpu().numpy()   # one rounding to the storage type

    mult = 8 if wl.dtype == "bf16" else 1
    for rank in range(world):
        fwd, bwd = parallel.cuda_layer_fns(wl.B, wl.L, wl.T, wl.dtype)
        W1s, W2s, W3s = parallel.shard_experts(W1, W2, W3, rank, world, mult)
        f0, f1 = parallel.shard_range(wl.f, rank, world, mult)
        y, rw = parallel.sharded_forward(fwd, collect("y"), x, w_r, W1s, W2s, W3s)
        assert max_rel(rw.double().cpu().numpy(), w_ref) <= TOL[wl.dtype]        # routing is replicated
        names = iter(("dx", "dw_r", "d_route_w"))
        g = parallel.sharded_backward(bwd, lambda t: collect(next(names))(t), x, w_r, W1s, W2s, W3s, dy)
        assert max_rel(g["dW1"].double().cpu().numpy(), g_ref["dW1"][:, f0:f1, :]) <= TOL[wl.dtype]
        assert max_rel(g["dW3"].double().cpu().numpy(), g_ref["dW3"][:, f0:f1, :]) <= TOL[wl.dtype]
        assert max_rel(g["dW2"].double().cpu().numpy(), g_ref["dW2"][:, :, f0:f1]) <= TOL[wl.dtype]
    assert max_rel(landed("y", x), y_ref) <= TOL[wl.dtype]
    for k, like in (("dx", x), ("dw_r", w_r), ("d_route_w", sums["d_route_w"])):
        assert max_rel(landed(k, like), g_ref[k]) <= TOL[wl.dtype], k
