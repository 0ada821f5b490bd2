"""Pins for the CPU oracle: each test ties it to something other than itself
(a dense SwiGLU FFN written with torch ops, torch autograd on an independent
transcription of Algorithm 1, finite differences, invariants of the method,
the figures Appendix B prints)."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import lory_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_problem(B=2, L=12, T=4, d=6, f=10, E=3, seed=1, w_r_std=1.0, w_std=0.5):
    rng = np.random.default_rng(seed)
    return dict(
        x=rng.standard_normal((B, L, d)),
        w_r=rng.standard_normal((E, d)) * w_r_std,
        W1=rng.standard_normal((E, f, d)) * w_std,
        W2=rng.standard_normal((E, d, f)) * w_std,
        W3=rng.standard_normal((E, f, d)) * w_std,
        dy=rng.standard_normal((B, L, d)),
        T=T,
    )


def fwd(p):
    return O.forward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"])


def bwd(p):
    return O.backward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"])


def dense_ffn_torch(x, W1, W2, W3):
    """Textbook LLaMA SwiGLU FFN with library ops: W2 (silu(W1 x) * W3 x)."""
    return F.linear(F.silu(F.linear(x, W1)) * F.linear(x, W3), W2)


def t64(a, grad=False):
    return torch.tensor(np.asarray(a), dtype=torch.float64, requires_grad=grad)


# ---- I1 ------------------------------------------------------------------
@pytest.mark.parametrize("std", [0.02, 1.0, 5.0])
def test_routing_weights_are_a_distribution(std):
    p = rand_problem(w_r_std=std)
    _, w, pr = fwd(p)
    assert np.all(w > 0) and np.all(pr > 0)
    np.testing.assert_allclose(w.sum(1), 1.0, rtol=0, atol=1e-14)
    np.testing.assert_allclose(pr.sum(1), 1.0, rtol=0, atol=1e-14)


def test_softmax_matches_library_and_is_shift_invariant():
    rng = np.random.default_rng(0)
    h = rng.standard_normal((5, 7))
    wr = rng.standard_normal((4, 7)) * 3
    p = O.router_probs(h, wr)
    ref = torch.softmax(t64(h) @ t64(wr).T, dim=-1).numpy()
    np.testing.assert_allclose(p, ref, rtol=1e-13, atol=0)
    # huge logits must not overflow
    p_big = O.router_probs(h * 1e4, wr)
    assert np.all(np.isfinite(p_big))


# ---- the shift (Algorithm 1) -----------------------------------------------
def test_causal_shift_layout():
    B, N, E = 3, 4, 2
    p = np.arange(B * N * E, dtype=float).reshape(B * N, E)
    w = O.causal_shift(p, B, N).reshape(B, N, E)
    p3 = p.reshape(B, N, E)
    for b in range(B):
        np.testing.assert_array_equal(w[b, 0], p3[b, 0])       # first segment routes itself
        for n in range(1, N):
            np.testing.assert_array_equal(w[b, n], p3[b, n - 1])


def test_shift_equals_roll_then_overwrite():
    """Algorithm 1 rolls the flat [B*N, E] table by one row and then overwrites
    row 0 of every sequence; the per-sequence shift must be the same thing."""
    B, N, E = 3, 5, 4
    rng = np.random.default_rng(3)
    p = rng.random((B * N, E))
    e = torch.roll(torch.tensor(p), 1, dims=0).view(B, N, E).clone()
    e[:, 0] = torch.tensor(p).view(B, N, E)[:, 0]
    np.testing.assert_array_equal(O.causal_shift(p, B, N), e.view(B * N, E).numpy())


# ---- I2 / I8: identical experts, single expert -> dense FFN -----------------
@pytest.mark.parametrize("E", [1, 4])
def test_identical_experts_reduce_to_dense_ffn(E):
    p = rand_problem(E=E, seed=5)
    for k in ("W1", "W2", "W3"):
        p[k] = np.repeat(p[k][:1], E, axis=0)
    y, _, _ = fwd(p)
    x = t64(p["x"], True)
    W1, W2, W3 = t64(p["W1"][0], True), t64(p["W2"][0], True), t64(p["W3"][0], True)
    y_ref = dense_ffn_torch(x, W1, W2, W3)
    np.testing.assert_allclose(y, y_ref.detach().numpy(), rtol=1e-11, atol=1e-12)
    y_ref.backward(t64(p["dy"]))
    g = bwd(p)
    # the routing gradient is the same for every expert -> softmax backward gives zero
    np.testing.assert_allclose(g["dw_r"], 0.0, atol=1e-10)
    np.testing.assert_allclose(g["dx"], x.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(g["dW1"].sum(0), W1.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(g["dW2"].sum(0), W2.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(g["dW3"].sum(0), W3.grad.numpy(), rtol=1e-10, atol=1e-11)


# ---- I3: one-hot injected weights select an expert ------------------------
def test_one_hot_weights_select_single_expert():
    p = rand_problem(E=4, seed=7)
    B, L, d = p["x"].shape
    T = p["T"]
    S = B * L // T
    seg_x = p["x"].reshape(S, T, d)
    seg_dy = p["dy"].reshape(S, T, d)
    pick = np.arange(S) % 4
    w = np.eye(4)[pick]
    seg_y = O.moe_ffn(seg_x, w, p["W1"], p["W2"], p["W3"])
    dseg_x, dW1, dW2, dW3, dw = O.moe_ffn_backward(seg_x, w, p["W1"], p["W2"], p["W3"], seg_dy)
    W1, W2, W3 = t64(p["W1"], True), t64(p["W2"], True), t64(p["W3"], True)
    xs = t64(seg_x, True)
    ys = torch.stack([dense_ffn_torch(xs[s], W1[pick[s]], W2[pick[s]], W3[pick[s]]) for s in range(S)])
    np.testing.assert_allclose(seg_y, ys.detach().numpy(), rtol=1e-11, atol=1e-12)
    ys.backward(t64(seg_dy))
    np.testing.assert_allclose(dseg_x, xs.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(dW1, W1.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(dW2, W2.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(dW3, W3.grad.numpy(), rtol=1e-10, atol=1e-11)
    assert dw.shape == (S, 4)


# ---- I7: zero router -> uniform merge ----------------------------------------
def test_zero_router_gives_mean_of_experts():
    p = rand_problem(E=5, seed=9)
    p["w_r"] = np.zeros_like(p["w_r"])
    y, w, _ = fwd(p)
    np.testing.assert_allclose(w, 1.0 / 5, rtol=0, atol=1e-15)
    y_ref = dense_ffn_torch(t64(p["x"]), t64(p["W1"].mean(0)), t64(p["W2"].mean(0)), t64(p["W3"].mean(0)))
    np.testing.assert_allclose(y, y_ref.numpy(), rtol=1e-11, atol=1e-12)


# ---- I4: segment causality --------------------------------------------------
@pytest.mark.parametrize("std", [0.02, 3.0])
def test_segment_causality(std):
    p = rand_problem(B=2, L=20, T=4, w_r_std=std, seed=11)
    y0, _, _ = fwd(p)
    T = p["T"]
    rng = np.random.default_rng(12)
    for k in range(0, 4):
        q = dict(p)
        x2 = p["x"].copy()
        x2[:, (k + 1) * T:] = rng.standard_normal(x2[:, (k + 1) * T:].shape)
        q["x"] = x2
        y1, _, _ = fwd(q)
        # outputs of segments <= k are bit-identical
        assert np.array_equal(y0[:, :(k + 1) * T], y1[:, :(k + 1) * T])


def test_previous_segment_must_influence_next():
    """Changing segment k-1 while keeping segment k's tokens must change segment
    k's output: it is routed by segment k-1 (catches a missing shift)."""
    p = rand_problem(B=1, L=16, T=4, w_r_std=3.0, seed=13)
    y0, w0, _ = fwd(p)
    q = dict(p)
    x2 = p["x"].copy()
    x2[:, 4:8] += 1.0                      # segment 1
    q["x"] = x2
    y1, w1, _ = fwd(q)
    assert np.abs(y1[:, 8:12] - y0[:, 8:12]).max() > 1e-3      # segment 2 changed
    assert np.array_equal(y1[:, 12:16], y0[:, 12:16])           # segment 3 (routed by 2) did not
    assert np.array_equal(y1[:, 0:4], y0[:, 0:4])
    # segment 1 itself is routed by segment 0: its weights did not move
    np.testing.assert_array_equal(w0[1], w1[1])


def test_first_segment_routes_itself():
    p = rand_problem(B=2, L=12, T=4, w_r_std=3.0, seed=14)
    _, w, pr = fwd(p)
    N = 3
    for b in range(2):
        np.testing.assert_array_equal(w[b * N], pr[b * N])
        np.testing.assert_array_equal(w[b * N + 1], pr[b * N])
        np.testing.assert_array_equal(w[b * N + 2], pr[b * N + 1])


# ---- I14: independent autograd formulation of the layer -----------------------
def lory_layer_torch(x, w_r, W1, W2, W3, T):
    """The layer written per sequence with torch ops: segment s of a sequence is weighted by the router
    output of segment s-1, the first segment by its own output cut from the graph."""
    B, L, d = x.shape
    N = L // T
    segs = x.reshape(B, N, T, d)
    p = torch.softmax(torch.einsum("bnd,ed->bne", segs.mean(dim=2), w_r), dim=-1)
    w = torch.cat([p[:, :1].detach(), p[:, :-1]], dim=1)
    up = lambda Wk: torch.einsum("bntd,bne,efd->bntf", segs, w, Wk)
    h = F.silu(up(W1)) * up(W3)
    y = torch.einsum("bntf,bne,edf->bntd", h, w, W2)
    return y.reshape(B, L, d), w.reshape(B * N, -1)


@pytest.mark.parametrize("std,shape", [(0.02, dict()), (2.0, dict()), (4.0, dict(B=3, L=10, T=2, d=5, f=7, E=4)),
                                       (1.0, dict(B=2, L=6, T=6))])
def test_autograd_transcription_agrees(std, shape):
    p = rand_problem(w_r_std=std, seed=21, **shape)
    ts = {k: t64(p[k], True) for k in ("x", "w_r", "W1", "W2", "W3")}
    y_t, e_t = lory_layer_torch(ts["x"], ts["w_r"], ts["W1"], ts["W2"], ts["W3"], p["T"])
    y, w, _ = fwd(p)
    np.testing.assert_allclose(y, y_t.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(w, e_t.detach().numpy(), rtol=1e-13, atol=0)
    y_t.backward(t64(p["dy"]))
    g = bwd(p)
    for ok, tk in (("dx", "x"), ("dw_r", "w_r"), ("dW1", "W1"), ("dW2", "W2"), ("dW3", "W3")):
        ref = ts[tk].grad.numpy() if ts[tk].grad is not None else np.zeros_like(g[ok])
        np.testing.assert_allclose(g[ok], ref, rtol=1e-9, atol=1e-10 * max(1.0, np.abs(ref).max()), err_msg=ok)


def test_injected_weight_gradient_matches_autograd():
    p = rand_problem(seed=23)
    B, L, d = p["x"].shape
    T = p["T"]
    S = B * L // T
    rng = np.random.default_rng(24)
    w = rng.random((S, 3))
    seg_x, seg_dy = p["x"].reshape(S, T, d), p["dy"].reshape(S, T, d)
    _, _, _, _, dw = O.moe_ffn_backward(seg_x, w, p["W1"], p["W2"], p["W3"], seg_dy)
    wt = t64(w, True)
    Wb1 = torch.einsum("se,efd->sfd", wt, t64(p["W1"]))
    Wb3 = torch.einsum("se,efd->sfd", wt, t64(p["W3"]))
    Wb2 = torch.einsum("se,edf->sdf", wt, t64(p["W2"]))
    xs = t64(seg_x)
    ys = torch.einsum("stf,sdf->std", F.silu(torch.einsum("std,sfd->stf", xs, Wb1)) * torch.einsum("std,sfd->stf", xs, Wb3), Wb2)
    ys.backward(t64(seg_dy))
    np.testing.assert_allclose(dw, wt.grad.numpy(), rtol=1e-10, atol=1e-11)


# ---- I10: central finite differences ----------------------------------------
@pytest.mark.parametrize("std", [0.5, 3.0])
def test_finite_differences(std):
    p = rand_problem(B=2, L=8, T=2, d=4, f=6, E=3, seed=31, w_r_std=std)
    g = bwd(p)

    B, L, d = p["x"].shape
    N = L // p["T"]
    _, _, w_base = O.route(p["x"], p["w_r"], p["T"])

    def loss(q):
        # the stop-gradient makes the first segment's weights constants: freeze them at
        # their unperturbed values, everything else follows the perturbed inputs
        _, _, w = O.route(q["x"], q["w_r"], q["T"])
        w = w.copy()
        w[::N] = w_base[::N]
        seg_y = O.moe_ffn(q["x"].reshape(B * N, q["T"], d), w, q["W1"], q["W2"], q["W3"])
        return float((seg_y.reshape(B, L, d) * p["dy"]).sum())

    rng = np.random.default_rng(32)
    h = 1e-6
    for key, gkey in (("x", "dx"), ("w_r", "dw_r"), ("W1", "dW1"), ("W2", "dW2"), ("W3", "dW3")):
        a = p[key]
        idxs = [tuple(rng.integers(0, n) for n in a.shape) for _ in range(12)]
        for idx in idxs:
            q = dict(p)
            ap, am = a.copy(), a.copy()
            ap[idx] += h
            am[idx] -= h
            q[key] = ap
            lp = loss(q)
            q[key] = am
            lm = loss(q)
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g[gkey][idx]) <= 1e-6 * max(1.0, abs(fd)), (key, idx, fd, g[gkey][idx])


def test_finite_difference_of_injected_weights():
    p = rand_problem(B=1, L=6, T=2, d=4, f=5, E=3, seed=33)
    S, T, d = 3, 2, 4
    seg_x, seg_dy = p["x"].reshape(S, T, d), p["dy"].reshape(S, T, d)
    w = np.random.default_rng(34).random((S, 3))
    _, _, _, _, dw = O.moe_ffn_backward(seg_x, w, p["W1"], p["W2"], p["W3"], seg_dy)
    h = 1e-6
    for s in range(S):
        for e in range(3):
            wp, wm = w.copy(), w.copy()
            wp[s, e] += h
            wm[s, e] -= h
            lp = (O.moe_ffn(seg_x, wp, p["W1"], p["W2"], p["W3"]) * seg_dy).sum()
            lm = (O.moe_ffn(seg_x, wm, p["W1"], p["W2"], p["W3"]) * seg_dy).sum()
            fd = (lp - lm) / (2 * h)
            assert abs(fd - dw[s, e]) <= 1e-6 * max(1.0, abs(fd))


# ---- I5 / I6: identities that hold at any size --------------------------------
def test_linearity_identities():
    """Y_s is linear in Wbar2_s and in Wbar3_s, so
    sum_e w_se <dWbar2_s, W2_e> = <dY_s, Y_s> = sum_e w_se <dWbar3_s, W3_e>."""
    p = rand_problem(B=2, L=12, T=4, d=5, f=7, E=3, seed=41, w_r_std=2.0)
    B, L, d = p["x"].shape
    T = p["T"]
    S = B * L // T
    y, w, _ = fwd(p)
    seg_x, seg_dy = p["x"].reshape(S, T, d), p["dy"].reshape(S, T, d)
    g = O.moe_ffn_backward(seg_x, w, p["W1"], p["W2"], p["W3"], seg_dy)
    dw = g[4]
    # sum_e w_se dw_se = <dWbar1,Wbar1> + <dWbar2,Wbar2> + <dWbar3,Wbar3>; the last two equal <dY,Y>
    # and the first equals <dG, G>.  Recompute <dG,G> from scratch with torch for an independent value.
    lhs = (w * dw).sum(1)
    rhs = np.empty(S)
    for s in range(S):
        Wb1 = t64(np.tensordot(w[s], p["W1"], axes=(0, 0)), True)
        Wb2 = t64(np.tensordot(w[s], p["W2"], axes=(0, 0)), True)
        Wb3 = t64(np.tensordot(w[s], p["W3"], axes=(0, 0)), True)
        ys = dense_ffn_torch(t64(seg_x[s]), Wb1, Wb2, Wb3)
        ys.backward(t64(seg_dy[s]))
        rhs[s] = float(((Wb1.grad * Wb1).sum() + (Wb2.grad * Wb2).sum() + (Wb3.grad * Wb3).sum()).detach())
        yd = float((ys.detach() * t64(seg_dy[s])).sum())
        np.testing.assert_allclose(float((Wb2.grad * Wb2).sum().detach()), yd, rtol=1e-10)
        np.testing.assert_allclose(float((Wb3.grad * Wb3).sum().detach()), yd, rtol=1e-10)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-10)
    np.testing.assert_allclose(y.reshape(S, T, d), O.moe_ffn(seg_x, w, p["W1"], p["W2"], p["W3"]), rtol=0, atol=0)


def test_router_gradient_rows_sum_to_zero():
    p = rand_problem(E=4, seed=43, w_r_std=2.0)
    g = bwd(p)
    np.testing.assert_allclose(g["dw_r"].sum(0), 0.0, atol=1e-10 * np.abs(g["dw_r"]).max())
    assert np.abs(g["dw_r"]).max() > 1e-6


def test_single_segment_has_no_router_gradient():
    """N = 1: the only routing weights are the stop-gradient ones."""
    p = rand_problem(B=3, L=4, T=4, seed=45, w_r_std=2.0)
    g = bwd(p)
    assert np.all(g["dw_r"] == 0.0)


def test_last_segment_probability_is_unused():
    """p of the last segment of each sequence feeds nothing: perturbing W_r's effect
    there cannot matter; equivalently dx of the router path is zero on last segments."""
    p = rand_problem(B=2, L=12, T=4, seed=46, w_r_std=2.0)
    h_bar, pr, w = O.route(p["x"], p["w_r"], p["T"])
    B, L, d = p["x"].shape
    g = bwd(p)
    dxr, _ = O.router_backward(p["x"].shape, p["T"], h_bar, pr, p["w_r"], g["d_route_w"])
    assert np.all(dxr[:, 8:12] == 0.0)
    assert np.abs(dxr[:, 0:8]).max() > 0


# ---- I11 / I12 -----------------------------------------------------------------
def test_expert_permutation_equivariance():
    p = rand_problem(E=4, seed=51, w_r_std=2.0)
    perm = np.array([2, 0, 3, 1])
    q = dict(p)
    for k in ("w_r", "W1", "W2", "W3"):
        q[k] = p[k][perm]
    y0, w0, _ = fwd(p)
    y1, w1, _ = fwd(q)
    np.testing.assert_allclose(y1, y0, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(w1, w0[:, perm], rtol=1e-13)
    g0, g1 = bwd(p), bwd(q)
    np.testing.assert_allclose(g1["dx"], g0["dx"], rtol=1e-10, atol=1e-12)
    for k in ("dw_r", "dW1", "dW2", "dW3"):
        np.testing.assert_allclose(g1[k], g0[k][perm], rtol=1e-10, atol=1e-12)


def test_sequences_are_independent():
    p = rand_problem(B=3, seed=53, w_r_std=2.0)
    y, _, _ = fwd(p)
    g = bwd(p)
    dW1_sum = np.zeros_like(g["dW1"])
    for b in range(3):
        q = dict(p)
        q["x"], q["dy"] = p["x"][b:b + 1], p["dy"][b:b + 1]
        yb, _, _ = fwd(q)
        gb = bwd(q)
        np.testing.assert_allclose(yb[0], y[b], rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(gb["dx"][0], g["dx"][b], rtol=1e-12, atol=1e-13)
        dW1_sum += gb["dW1"]
    np.testing.assert_allclose(dW1_sum, g["dW1"], rtol=1e-11, atol=1e-12)


# ---- sampled variants agree with the plain ones ---------------------------------
def test_sampled_variants_match_full():
    p = rand_problem(B=2, L=12, T=4, d=6, f=10, E=3, seed=61, w_r_std=2.0)
    a = (p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"])
    y, _, _ = fwd(p)
    g = bwd(p)
    segs = O.forward_segments(*a, [0, 3, 5])
    for s, ys in segs.items():
        np.testing.assert_array_equal(ys, y.reshape(6, 4, 6)[s])
    rows = [7, 0, 4]
    dW1r, dW2c, dW3r = O.backward_frows(*a, p["dy"], rows)
    np.testing.assert_allclose(dW1r, g["dW1"][:, rows], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dW3r, g["dW3"][:, rows], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dW2c, g["dW2"][:, :, rows], rtol=1e-12, atol=1e-13)
    bs = O.backward_segments(*a, p["dy"], [1, 4])
    h_bar, pr, _ = O.route(p["x"], p["w_r"], p["T"])
    dxr, _ = O.router_backward(p["x"].shape, p["T"], h_bar, pr, p["w_r"], g["d_route_w"])
    dx_ffn = (g["dx"] - dxr).reshape(6, 4, 6)
    for s, (dxs, dws) in bs.items():
        np.testing.assert_allclose(dxs, dx_ffn[s], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(dws, g["d_route_w"][s], rtol=1e-11, atol=1e-12)
    d_rows = [5, 0, 2]
    for group in (8, 4, 1):     # one group, a ragged last group, segment by segment
        dx_all, dw_all, dW2r, dW1c, dW3c = O.backward_every_segment(*a, p["dy"], d_rows, group=group)
        np.testing.assert_allclose(dx_all, dx_ffn, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(dw_all, g["d_route_w"], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(dW2r, g["dW2"][:, d_rows, :], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(dW1c, g["dW1"][:, :, d_rows], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(dW3c, g["dW3"][:, :, d_rows], rtol=1e-11, atol=1e-12)


# ---- I15: Appendix B figures --------------------------------------------------
def test_flop_model_reproduces_appendix_b():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "appendix_b_overhead.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 2
    for E, T, pct in rows:
        E, T = int(E), int(T)
        assert round(100 * O.merge_overhead(E, T), 1) == float(pct)
        d, f, L = 1024, 2752, 4096
        extra = (L // T) * O.merge_flops(E, d, f) / O.ffn_flops(L, d, f)
        assert round(100 * extra, 1) == float(pct)
    assert O.layer_flops(8, 4096, 256, 1024, 2752, 32) == 18 * 1024 * 2752 * (256 + 32) * 128


def test_rejects_ragged_length():
    p = rand_problem(L=10, T=4)
    with pytest.raises(ValueError):
        fwd(p)


# ---- inference routing and expert utilisation -----------------------------------
def test_prompt_only_inference_is_a_dense_ffn_per_sequence():
    p = rand_problem(B=3, L=10, T=10, d=6, f=8, E=4, seed=71, w_r_std=2.0)
    rng = np.random.default_rng(72)
    x_new = rng.standard_normal((3, 5, 6))
    y_prompt, y_new, w = O.prompt_only_inference(p["x"], x_new, p["w_r"], p["W1"], p["W2"], p["W3"])
    # weights: softmax of the router applied to the mean of the whole prompt (library routines)
    ref_w = torch.softmax(t64(p["x"]).mean(dim=1) @ t64(p["w_r"]).T, dim=-1).numpy()
    np.testing.assert_allclose(w, ref_w, rtol=1e-12)
    for b in range(3):
        Wb = [t64(np.tensordot(ref_w[b], p[k], axes=(0, 0))) for k in ("W1", "W2", "W3")]
        np.testing.assert_allclose(y_new[b], dense_ffn_torch(t64(x_new[b]), *Wb).numpy(), rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(y_prompt[b], dense_ffn_torch(t64(p["x"][b]), *Wb).numpy(), rtol=1e-11, atol=1e-12)
    # a prompt that is one segment long is what the training forward computes for that segment
    y_train, w_train, _ = fwd(p)
    np.testing.assert_allclose(y_prompt, y_train, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(w, w_train, rtol=1e-13)


def test_expert_utilization_counts_weights_above_two_over_e():
    w = np.array([[0.7, 0.1, 0.1, 0.1], [0.25, 0.25, 0.25, 0.25], [0.5, 0.5, 0.0, 0.0], [0.51, 0.0, 0.49, 0.0]])
    # threshold 2/E = 0.5, strictly larger
    np.testing.assert_array_equal(O.expert_utilization(w), [2, 0, 0, 0])
    w8 = np.full((5, 8), 1 / 8)
    w8[2, 3] = 0.3; w8[2, 0] = 0.125 - (0.3 - 0.125)          # 0.3 > 2/8
    np.testing.assert_array_equal(O.expert_utilization(w8), [0, 0, 0, 1, 0, 0, 0, 0])


# ---- prefix routing (ablation of Section 5.1) -----------------------------------------
def prefix_routing_torch(x, w_r, W1, W2, W3, T):
    """Independent transcription: merge once per sequence from its first segment."""
    B, L, d = x.shape
    N = L // T
    E = w_r.shape[0]
    seg_x = x.view(B, N, T, d)
    e0 = torch.softmax(seg_x[:, 0].mean(dim=1) @ w_r.T, dim=-1)            # [B, E]
    e = e0[:, None, :].expand(B, N, E).clone()
    e[:, 0] = e0.detach()                                                  # the first segment routes itself: no gradient
    Wb1 = torch.einsum("bne,efd->bnfd", e, W1)
    Wb3 = torch.einsum("bne,efd->bnfd", e, W3)
    Wb2 = torch.einsum("bne,edf->bndf", e, W2)
    g = torch.einsum("bntd,bnfd->bntf", seg_x, Wb1)
    u = torch.einsum("bntd,bnfd->bntf", seg_x, Wb3)
    y = torch.einsum("bntf,bndf->bntd", F.silu(g) * u, Wb2)
    return y.reshape(B, L, d), e.reshape(B * N, E)


def test_prefix_routing_agrees_with_autograd():
    p = rand_problem(B=2, L=12, T=3, d=5, f=7, E=4, seed=81, w_r_std=2.0)
    ts = {k: t64(p[k], True) for k in ("x", "w_r", "W1", "W2", "W3")}
    y_t, e_t = prefix_routing_torch(ts["x"], ts["w_r"], ts["W1"], ts["W2"], ts["W3"], p["T"])
    y, w, _ = O.forward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], prefix=True)
    np.testing.assert_allclose(y, y_t.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(w, e_t.detach().numpy(), rtol=1e-13)
    # every segment of a sequence uses the same weights
    w3 = w.reshape(2, 4, 4)
    assert np.all(w3 == w3[:, :1])
    y_t.backward(t64(p["dy"]))
    g = O.backward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"], prefix=True)
    for ok, tk in (("dx", "x"), ("dw_r", "w_r"), ("dW1", "W1"), ("dW2", "W2"), ("dW3", "W3")):
        ref = ts[tk].grad.numpy()
        np.testing.assert_allclose(g[ok], ref, rtol=1e-9, atol=1e-10 * max(1.0, np.abs(ref).max()), err_msg=ok)
    # only first segments reach the router: later segments' tokens get no router-path gradient
    h_bar, pr, _ = O.route(p["x"], p["w_r"], p["T"], prefix=True)
    dxr, _ = O.router_backward(p["x"].shape, p["T"], h_bar, pr, p["w_r"], g["d_route_w"], prefix=True)
    assert np.all(dxr[:, 3:] == 0.0) and np.abs(dxr[:, :3]).max() > 0


# ---- whole-sequence routing (Section 2.2) and the first segment's gradient -----------------------
def sequence_routing_torch(x, w_r, W1, W2, W3):
    """Independent transcription of routing from the pooled whole sequence: one merged FFN per sequence,
    the router inside the autograd graph (no stop-gradient)."""
    e = torch.softmax(x.mean(dim=1) @ w_r.T, dim=-1)                       # [B, E]
    Wb1 = torch.einsum("be,efd->bfd", e, W1)
    Wb3 = torch.einsum("be,efd->bfd", e, W3)
    Wb2 = torch.einsum("be,edf->bdf", e, W2)
    h = F.silu(torch.einsum("btd,bfd->btf", x, Wb1)) * torch.einsum("btd,bfd->btf", x, Wb3)
    return torch.einsum("btf,bdf->btd", h, Wb2), e


def test_whole_sequence_routing_agrees_with_autograd():
    p = rand_problem(B=3, L=6, T=6, d=5, f=7, E=4, seed=91, w_r_std=2.0)
    ts = {k: t64(p[k], True) for k in ("x", "w_r", "W1", "W2", "W3")}
    y_t, e_t = sequence_routing_torch(ts["x"], ts["w_r"], ts["W1"], ts["W2"], ts["W3"])
    y, w, _ = O.forward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"])
    np.testing.assert_allclose(y, y_t.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(w, e_t.detach().numpy(), rtol=1e-13)
    y_t.backward(t64(p["dy"]))
    g = O.backward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"], first_grad=True)
    for ok, tk in (("dx", "x"), ("dw_r", "w_r"), ("dW1", "W1"), ("dW2", "W2"), ("dW3", "W3")):
        ref = ts[tk].grad.numpy()
        np.testing.assert_allclose(g[ok], ref, rtol=1e-9, atol=1e-10 * max(1.0, np.abs(ref).max()), err_msg=ok)
    assert np.abs(g["dw_r"]).max() > 0          # the router does learn here
    # with the stop-gradient the same problem gives the router nothing, and only the router path differs
    g0 = O.backward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"])
    assert np.all(g0["dw_r"] == 0.0)
    np.testing.assert_array_equal(g0["dW1"], g["dW1"])


def test_first_segment_gradient_with_several_segments():
    """Causal routing without the stop-gradient on the first segment, against autograd."""
    p = rand_problem(B=2, L=12, T=3, d=5, f=6, E=3, seed=92, w_r_std=2.0)
    ts = {k: t64(p[k], True) for k in ("x", "w_r", "W1", "W2", "W3")}
    B, L, d = p["x"].shape
    N, T = L // p["T"], p["T"]
    seg_x = ts["x"].view(B, N, T, d)
    pr = torch.softmax(seg_x.mean(dim=2) @ ts["w_r"].T, dim=-1)           # [B, N, E]
    e = torch.cat([pr[:, :1], pr[:, :-1]], dim=1)                          # no detach on the first segment
    Wb1 = torch.einsum("bne,efd->bnfd", e, ts["W1"])
    Wb3 = torch.einsum("bne,efd->bnfd", e, ts["W3"])
    Wb2 = torch.einsum("bne,edf->bndf", e, ts["W2"])
    h = F.silu(torch.einsum("bntd,bnfd->bntf", seg_x, Wb1)) * torch.einsum("bntd,bnfd->bntf", seg_x, Wb3)
    y_t = torch.einsum("bntf,bndf->bntd", h, Wb2).reshape(B, L, d)
    y_t.backward(t64(p["dy"]))
    g = O.backward(p["x"], p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"], first_grad=True)
    for ok, tk in (("dx", "x"), ("dw_r", "w_r"), ("dW1", "W1"), ("dW2", "W2"), ("dW3", "W3")):
        ref = ts[tk].grad.numpy()
        np.testing.assert_allclose(g[ok], ref, rtol=1e-9, atol=1e-10 * max(1.0, np.abs(ref).max()), err_msg=ok)


# ---- the layer inside a pre-norm residual block ------------------------------------------------------
def test_rmsnorm_matches_library_routine_and_autograd():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 5, 7)) * 3.0
    gamma = rng.standard_normal(7)
    dxh = rng.standard_normal((2, 5, 7))
    eps = 1e-5
    xh, inv = O.rmsnorm(x, gamma, eps)
    xt, gt = t64(x, True), t64(gamma, True)
    ref = F.rms_norm(xt, (7,), weight=gt, eps=eps)
    np.testing.assert_allclose(xh, ref.detach().numpy(), rtol=1e-12, atol=1e-13)
    ref.backward(t64(dxh))
    dx, dgamma = O.rmsnorm_backward(x, gamma, inv, dxh)
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dgamma, gt.grad.numpy(), rtol=1e-10, atol=1e-12)
    # closed forms: unit rows stay unit up to gamma; scaling the input does not change the output (eps = 0)
    xh1, _ = O.rmsnorm(x, np.ones(7), 0.0)
    np.testing.assert_allclose((xh1 ** 2).mean(-1), 1.0, rtol=1e-12)
    xh2, _ = O.rmsnorm(5.0 * x, np.ones(7), 0.0)
    np.testing.assert_allclose(xh2, xh1, rtol=1e-12)


def test_block_agrees_with_autograd():
    p = rand_problem(B=2, L=12, T=3, d=5, f=7, E=4, seed=95, w_r_std=2.0)
    rng = np.random.default_rng(96)
    gamma = 1.0 + 0.3 * rng.standard_normal(5)
    eps = 1e-5
    ts = {k: t64(p[k], True) for k in ("x", "w_r", "W1", "W2", "W3")}
    gt = t64(gamma, True)
    xh = F.rms_norm(ts["x"], (5,), weight=gt, eps=eps)
    # Algorithm 1 on the normalised input, independent of the oracle's forward
    B, L, d = p["x"].shape
    N, T = L // p["T"], p["T"]
    seg = xh.view(B, N, T, d)
    pr = torch.softmax(seg.mean(dim=2) @ ts["w_r"].T, dim=-1)
    e = torch.cat([pr[:, :1].detach(), pr[:, :-1]], dim=1)
    Wb1 = torch.einsum("bne,efd->bnfd", e, ts["W1"])
    Wb3 = torch.einsum("bne,efd->bnfd", e, ts["W3"])
    Wb2 = torch.einsum("bne,edf->bndf", e, ts["W2"])
    h = F.silu(torch.einsum("bntd,bnfd->bntf", seg, Wb1)) * torch.einsum("bntd,bnfd->bntf", seg, Wb3)
    y_t = ts["x"] + torch.einsum("bntf,bndf->bntd", h, Wb2).reshape(B, L, d)
    y, w, _ = O.block_forward(p["x"], gamma, eps, p["w_r"], p["W1"], p["W2"], p["W3"], p["T"])
    np.testing.assert_allclose(y, y_t.detach().numpy(), rtol=1e-11, atol=1e-12)
    y_t.backward(t64(p["dy"]))
    g = O.block_backward(p["x"], gamma, eps, p["w_r"], p["W1"], p["W2"], p["W3"], p["T"], p["dy"])
    for ok, ref in (("dx", ts["x"].grad), ("dw_r", ts["w_r"].grad), ("dW1", ts["W1"].grad), ("dW2", ts["W2"].grad),
                    ("dW3", ts["W3"].grad), ("dgamma", gt.grad)):
        ref = ref.numpy()
        np.testing.assert_allclose(g[ok], ref, rtol=1e-9, atol=1e-10 * max(1.0, np.abs(ref).max()), err_msg=ok)
    # zero experts' output (W2 = 0) leaves the residual: y = x and dx = dy
    y0, _, _ = O.block_forward(p["x"], gamma, eps, p["w_r"], p["W1"], 0 * p["W2"], p["W3"], p["T"])
    np.testing.assert_array_equal(y0, p["x"])
    g0 = O.block_backward(p["x"], gamma, eps, p["w_r"], p["W1"], 0 * p["W2"], p["W3"], p["T"], p["dy"])
    np.testing.assert_allclose(g0["dx"], p["dy"], rtol=0, atol=1e-15)
