"""The torch.nn.Module wrapper (autograd glue over the C ABI) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import lory_oracle as O
from paper_2405_03133_b200.layer import LoryMoE
from paper_2405_03133_b200.workloads import Workload, make_inputs

from gpu_util import max_rel, to_dev

pytestmark = pytest.mark.gpu
TOL = {"fp32": 1e-4, "bf16": 2e-2}


def module_for(wl, inp):
    dtype = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    m = LoryMoE(wl.d, wl.f, wl.E, wl.T, dtype=dtype, device="cuda")
    with torch.no_grad():
        for name, key in (("w_r", "w_r"), ("W1", "W1"), ("W2", "W2"), ("W3", "W3")):
            getattr(m, name).copy_(to_dev(inp[key], wl))
    return m


@pytest.mark.parametrize("wl", [
    Workload("module_bf16", B=2, L=512, T=128, d=72, f=200, E=5, dtype="bf16", w_r_std=2.0, seed=61),
    Workload("module_fp32", B=3, L=40, T=8, d=24, f=52, E=5, dtype="fp32", w_r_std=2.0, seed=62),
], ids=lambda w: w.name)
def test_module_forward_and_autograd(wl):
    inp = make_inputs(wl)
    m = module_for(wl, inp)
    x = to_dev(inp["x"], wl).requires_grad_(True)
    y = m(x)
    y.backward(to_dev(inp["dy"], wl))
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y_ref, w_ref, _ = O.forward(*a)
    g = O.backward(*a, inp["dy"])
    got = dict(y=y, route_w=m.last_route_w, dx=x.grad, dw_r=m.w_r.grad, dW1=m.W1.grad, dW2=m.W2.grad, dW3=m.W3.grad)
    ref = dict(y=y_ref, route_w=w_ref, dx=g["dx"], dw_r=g["dw_r"], dW1=g["dW1"], dW2=g["dW2"], dW3=g["dW3"])
    errs = {k: max_rel(got[k].detach().double().cpu().numpy(), ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= TOL[wl.dtype]}
    assert not bad, (bad, errs)


def test_two_calls_in_flight_and_no_grad():
    """Two forwards before either backward (each keeps its own workspace), backward in reverse order; parameter
    gradients add up as autograd adds them; a forward without gradients leaves nothing behind."""
    wl = Workload("module_two", B=2, L=256, T=64, d=64, f=136, E=4, dtype="bf16", w_r_std=1.0, seed=63)
    inps = [make_inputs(wl), make_inputs(wl.with_(seed=64))]
    m = module_for(wl, inps[0])
    xs = [to_dev(i["x"], wl).requires_grad_(True) for i in inps]
    ys = [m(x) for x in xs]
    ys[1].backward(to_dev(inps[1]["dy"], wl))
    ys[0].backward(to_dev(inps[0]["dy"], wl))
    gs = [O.backward(i["x"], inps[0]["w_r"], inps[0]["W1"], inps[0]["W2"], inps[0]["W3"], wl.T, i["dy"]) for i in inps]
    for k in range(2):
        assert max_rel(xs[k].grad.double().cpu().numpy(), gs[k]["dx"]) <= TOL["bf16"]
    assert max_rel(m.W2.grad.double().cpu().numpy(), gs[0]["dW2"] + gs[1]["dW2"]) <= TOL["bf16"]
    assert max_rel(m.w_r.grad.double().cpu().numpy(), gs[0]["dw_r"] + gs[1]["dw_r"]) <= TOL["bf16"]
    with torch.no_grad():
        y = m(xs[0].detach())
    assert not y.requires_grad
    assert torch.equal(y, ys[0].detach())
    with pytest.raises(RuntimeError):
        m(torch.zeros(1, wl.L, wl.d))          # CPU tensor: there is no CPU path


def test_block_module_autograd():
    from paper_2405_03133_b200.layer import LoryBlock
    from paper_2405_03133_b200.workloads import round_to_bf16
    wl = Workload("module_block", B=2, L=512, T=128, d=72, f=200, E=5, dtype="bf16", w_r_std=1.0, seed=65)
    inp = dict(make_inputs(wl))
    for k in ("W1", "W2", "W3"):
        inp[k] = round_to_bf16(inp[k] * 10.0)            # layer output of the size of the residual
    gamma = round_to_bf16(1.0 + 0.2 * np.random.default_rng(66).standard_normal(wl.d))
    m = LoryBlock(wl.d, wl.f, wl.E, wl.T, eps=1e-5)
    with torch.no_grad():
        for name in ("w_r", "W1", "W2", "W3"):
            getattr(m, name).copy_(to_dev(inp[name], wl))
        m.gamma.copy_(to_dev(gamma, wl))
    x = to_dev(inp["x"], wl).requires_grad_(True)
    y = m(x)
    y.backward(to_dev(inp["dy"], wl))
    a = (inp["x"], gamma, 1e-5, inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y_ref, _, _ = O.block_forward(*a)
    g = O.block_backward(*a, inp["dy"])
    got = dict(y=y, dx=x.grad, dgamma=m.gamma.grad, dw_r=m.w_r.grad, dW1=m.W1.grad, dW2=m.W2.grad)
    ref = dict(y=y_ref, dx=g["dx"], dgamma=g["dgamma"], dw_r=g["dw_r"], dW1=g["dW1"], dW2=g["dW2"])
    errs = {k: max_rel(got[k].detach().double().cpu().numpy(), ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= TOL["bf16"]}
    assert not bad, (bad, errs)


def test_prompt_routed_ffn_helper():
    from paper_2405_03133_b200.layer import LoryPromptRoutedFFN
    from paper_2405_03133_b200.workloads import round_to_bf16
    wl = Workload("module_prompt", B=3, L=384, T=384, d=128, f=200, E=6, dtype="bf16", w_r_std=2.0, seed=67)
    inp = make_inputs(wl)
    m = module_for(wl, inp)
    ffn = LoryPromptRoutedFFN(m)
    with pytest.raises(RuntimeError):
        ffn.decode(torch.zeros(wl.B, 1, wl.d, device="cuda", dtype=torch.bfloat16))
    y_prompt = ffn.prefill(to_dev(inp["x"], wl))
    x_new = round_to_bf16(np.random.default_rng(68).standard_normal((wl.B, 4, wl.d)).astype(np.float32))
    y_new = ffn.decode(to_dev(x_new, wl))
    ref_prompt, ref_new, w_ref = O.prompt_only_inference(inp["x"], x_new, inp["w_r"], inp["W1"], inp["W2"], inp["W3"])
    assert max_rel(y_prompt.double().cpu().numpy(), ref_prompt) <= TOL["bf16"]
    assert max_rel(y_new.double().cpu().numpy(), ref_new) <= TOL["bf16"]
    assert max_rel(ffn.route_w.double().cpu().numpy(), w_ref) <= 1e-5


def test_prompt_routed_ffn_on_a_side_stream():
    """prefill and decode issued inside `with torch.cuda.stream(s)`: inputs are produced and outputs consumed on
    that stream only, so the library calls must run there too."""
    from paper_2405_03133_b200.layer import LoryPromptRoutedFFN
    from paper_2405_03133_b200.workloads import round_to_bf16
    wl = Workload("module_prompt_stream", B=2, L=256, T=256, d=128, f=200, E=5, dtype="bf16", w_r_std=2.0, seed=69)
    inp = make_inputs(wl)
    m = module_for(wl, inp)
    ffn = LoryPromptRoutedFFN(m)
    x_new = round_to_bf16(np.random.default_rng(70).standard_normal((wl.B, 3, wl.d)).astype(np.float32))
    xp_host = torch.from_numpy(inp["x"]).to(torch.bfloat16).pin_memory()
    xn_host = torch.from_numpy(x_new).to(torch.bfloat16).pin_memory()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        # the inputs reach the device on the side stream, right in front of the calls that read them
        xp = xp_host.to("cuda", non_blocking=True)
        xn = xn_host.to("cuda", non_blocking=True)
        y_prompt = ffn.prefill(xp)
        y_new = ffn.decode(xn)
        yp_host = y_prompt.to("cpu", non_blocking=True)
        yn_host = y_new.to("cpu", non_blocking=True)
    side.synchronize()
    ref_prompt, ref_new, _ = O.prompt_only_inference(inp["x"], x_new, inp["w_r"], inp["W1"], inp["W2"], inp["W3"])
    assert max_rel(yp_host.double().numpy(), ref_prompt) <= TOL["bf16"]
    assert max_rel(yn_host.double().numpy(), ref_new) <= TOL["bf16"]
