"""CPU oracle for the Lory MoE layer (causal segment routing + expert merging).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition of what
the layer computes, written from the paper.  It is used by the tests, by the
smoke check and by the benchmark's CPU-baseline leg; the product path never
imports it, and it imports nothing from the product.

Every array is taken as given (callers round inputs to bf16 beforehand when
they want the bf16 workload), converted to float64, and every sum is carried
in float64.  A numpy matmul is used as a step where the definition is a
matrix product; there is no tiling, fusion or reordering.

Notation (Section 3 "Notations", Algorithm 1):
    B sequences, L tokens each, T segment length, N = L / T segments per
    sequence, S = B*N segments, d hidden size, f FFN hidden size, E experts.
    x    [B, L, d]      layer input (hidden states h_x)
    w_r  [E, d]         router R, a bias-free linear layer
    W1   [E, f, d]      gate projections  (SwiGLU, LLaMA convention)
    W3   [E, f, d]      up projections
    W2   [E, d, f]      down projections
    p    [S, E]         softmax(R(mean of segment))            (Eq. 3)
    w    [S, E]         routing weights actually used (shifted, Algorithm 1)

Pins (tests/test_oracle_*.py): softmax rows sum to one; identical experts and
E = 1 reduce to a dense SwiGLU FFN written with torch ops; one-hot injected
weights select one expert; W_r = 0 gives the mean of the experts; segment
causality; expert permutation; sequence independence; central finite
differences of every gradient; an independent float64 autograd transcription
of Algorithm 1; linearity identities <dWbar2, Wbar2> = <dY, Y>; the FLOP
model's E/T overhead figures of Appendix B.  No function here is unpinned.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(a):
    return np.ascontiguousarray(a, dtype=F64)


# --------------------------------------------------------------------------
# Forward
# --------------------------------------------------------------------------
def segment_mean(x, T):
    """h_bar_s = (1/T) * sum of the hidden states of segment s  (Eq. 3;
    Algorithm 1 'repr = mean(seg_x, dim=1)').  Returns [S, d]."""
    x = _f64(x)
    B, L, d = x.shape
    if L % T != 0:
        raise ValueError("L must be a multiple of T (Algorithm 1 uses N = L // T and a view)")
    seg_x = x.reshape(B * (L // T), T, d)
    return seg_x.sum(axis=1) / T


def router_probs(h_bar, w_r):
    """p_s = softmax_e(W_r h_bar_s)  (Eq. 3; R is a linear layer, Section 3).
    Max-subtracted softmax, float64."""
    z = _f64(h_bar) @ _f64(w_r).T                     # [S, E]
    z = z - z.max(axis=1, keepdims=True)
    ez = np.exp(z)
    return ez / ez.sum(axis=1, keepdims=True)


def causal_shift(p, B, N, prefix=False):
    """Routing weights used by each segment (Section 3.1 'Training design',
    Algorithm 1): segment n >= 1 of a sequence uses the probabilities computed
    from segment n-1; segment 0 uses its own (and is a constant for the
    backward pass: stop-gradient).
    prefix=True is the 'prefix routing' ablation (Section 5.1): every segment of a
    sequence uses the probabilities of the sequence's first segment."""
    E = p.shape[1]
    p3 = p.reshape(B, N, E)
    w3 = np.empty_like(p3)
    w3[:, 0] = p3[:, 0]
    if prefix:
        w3[:, 1:] = p3[:, :1]
    else:
        w3[:, 1:] = p3[:, :-1]
    return w3.reshape(B * N, E)


def route(x, w_r, T, prefix=False):
    """F1-F4: returns (h_bar [S,d], p [S,E], w [S,E])."""
    B, L, _ = np.shape(x)
    h_bar = segment_mean(x, T)
    p = router_probs(h_bar, w_r)
    w = causal_shift(p, B, L // T, prefix)
    return h_bar, p, w


def merge_experts(w_s, Wk):
    """theta_bar = sum_e w_{s,e} * theta_e for one stacked matrix  (Eq. 2, Eq. 3).
    w_s [E], Wk [E, r, c] -> [r, c]."""
    return np.tensordot(w_s, Wk, axes=(0, 0))


def silu(g):
    return g / (1.0 + np.exp(-g))


def moe_ffn(seg_x, w, W1, W2, W3):
    """The paper's moe_ffn(seg_x, e): merge the experts with the given weights
    and run each segment through its merged SwiGLU FFN (Eq. 2; Section 3.1
    o_x = FFN(h_x; theta_bar) for every x in the segment).
    seg_x [S, T, d], w [S, E] -> seg_y [S, T, d]."""
    seg_x, w, W1, W2, W3 = map(_f64, (seg_x, w, W1, W2, W3))
    S = seg_x.shape[0]
    seg_y = np.empty_like(seg_x)
    for s in range(S):
        Wb1 = merge_experts(w[s], W1)                 # [f, d]
        Wb3 = merge_experts(w[s], W3)                 # [f, d]
        Wb2 = merge_experts(w[s], W2)                 # [d, f]
        G = seg_x[s] @ Wb1.T                          # [T, f]
        U = seg_x[s] @ Wb3.T
        H = silu(G) * U
        seg_y[s] = H @ Wb2.T
    return seg_y


def forward(x, w_r, W1, W2, W3, T, prefix=False):
    """Algorithm 1 end to end.  Returns (y [B,L,d], w [S,E], p [S,E])."""
    x = _f64(x)
    B, L, d = x.shape
    _, p, w = route(x, w_r, T, prefix)
    seg_y = moe_ffn(x.reshape(B * (L // T), T, d), w, W1, W2, W3)
    return seg_y.reshape(B, L, d), w, p


def forward_segments(x, w_r, W1, W2, W3, T, seg_ids):
    """Outputs of selected segments only (sampled checks at sizes where the
    whole layer is too slow on a CPU).  Returns {s: y_s [T, d]}."""
    x = _f64(x)
    B, L, d = x.shape
    _, _, w = route(x, w_r, T)
    seg_x = x.reshape(B * (L // T), T, d)
    out = {}
    for s in seg_ids:
        out[int(s)] = moe_ffn(seg_x[s:s + 1], w[s:s + 1], W1, W2, W3)[0]
    return out


# --------------------------------------------------------------------------
# Backward (chain rule through Algorithm 1; the paper states the layer is
# fully differentiable and places a stop-gradient on the first segment's
# routing weights, and does not write the gradients out).
# --------------------------------------------------------------------------
def _segment_grads(X, dY, Wb1, Wb2, Wb3):
    """Gradients of one segment's merged FFN.
    Returns dX [T,d], dWb1 [f,d], dWb2 [d,f], dWb3 [f,d]."""
    G = X @ Wb1.T
    U = X @ Wb3.T
    sig = 1.0 / (1.0 + np.exp(-G))
    H = G * sig * U
    dH = dY @ Wb2                                     # [T, f]
    dWb2 = dY.T @ H                                   # [d, f]
    dG = dH * U * sig * (1.0 + G * (1.0 - sig))
    dU = dH * G * sig
    dWb1 = dG.T @ X                                   # [f, d]
    dWb3 = dU.T @ X
    dX = dG @ Wb1 + dU @ Wb3
    return dX, dWb1, dWb2, dWb3


def moe_ffn_backward(seg_x, w, W1, W2, W3, seg_dy):
    """Backward of moe_ffn with w treated as an independent input.
    Returns (dseg_x, dW1, dW2, dW3, dw) with
        dWk_e  = sum_s w_{s,e} * dWbar_k,s        (adjoint of the merge)
        dw_s,e = sum_k <dWbar_k,s , Wk_e>          (Frobenius inner products)
    The per-segment merged-weight gradients are all kept, then the two sums
    are taken as the matrix products they are."""
    seg_x, w, W1, W2, W3, seg_dy = map(_f64, (seg_x, w, W1, W2, W3, seg_dy))
    S, T, d = seg_x.shape
    E, f, _ = W1.shape
    dseg_x = np.empty_like(seg_x)
    dWb1 = np.empty((S, f, d), F64)
    dWb2 = np.empty((S, d, f), F64)
    dWb3 = np.empty((S, f, d), F64)
    for s in range(S):
        Wb1 = merge_experts(w[s], W1)
        Wb3 = merge_experts(w[s], W3)
        Wb2 = merge_experts(w[s], W2)
        dseg_x[s], dWb1[s], dWb2[s], dWb3[s] = _segment_grads(seg_x[s], seg_dy[s], Wb1, Wb2, Wb3)
    wT = np.ascontiguousarray(w.T)                    # [E, S]
    dW1 = (wT @ dWb1.reshape(S, -1)).reshape(E, f, d)
    dW2 = (wT @ dWb2.reshape(S, -1)).reshape(E, d, f)
    dW3 = (wT @ dWb3.reshape(S, -1)).reshape(E, f, d)
    dw = (dWb1.reshape(S, -1) @ W1.reshape(E, -1).T
          + dWb2.reshape(S, -1) @ W2.reshape(E, -1).T
          + dWb3.reshape(S, -1) @ W3.reshape(E, -1).T)      # [S, E]
    return dseg_x, dW1, dW2, dW3, dw


def router_backward(x_shape, T, h_bar, p, w_r, dw, prefix=False, first_grad=False):
    """From the gradient wrt the shifted weights w back to x and W_r.
    dp_{b,n} = dw_{b,n+1} for n <= N-2, dp_{b,N-1} = 0, and dw_{b,0} is dropped
    (stop-gradient on the first segment, Section 3.1 / Algorithm 1).
    first_grad=True keeps dw_{b,0} instead (dp_{b,0} += dw_{b,0}): with one segment
    per sequence (T = L) that is the whole-sequence routing of Section 2.2, whose
    router learns from the sequence it routes.
    Softmax: dz = p * (dp - <dp, p>).  Linear router: dW_r = dz^T h_bar,
    dh_bar = dz W_r.  Mean: every token of the segment receives dh_bar / T.
    Returns (dx_router [B,L,d], dW_r [E,d])."""
    B, L, d = x_shape
    N = L // T
    E = p.shape[1]
    dw3 = dw.reshape(B, N, E)
    dp3 = np.zeros_like(dw3)
    if prefix:
        # the first segment's probabilities feed segments 1..N-1 (its own use is the stop-gradient one)
        dp3[:, 0] = dw3[:, 1:].sum(axis=1)
    else:
        dp3[:, :-1] = dw3[:, 1:]
    if first_grad:
        dp3[:, 0] += dw3[:, 0]
    dp = dp3.reshape(B * N, E)
    dz = p * (dp - (dp * p).sum(axis=1, keepdims=True))
    w_r = _f64(w_r)
    dW_r = dz.T @ h_bar
    dh_bar = dz @ w_r                                  # [S, d]
    dx_router = np.repeat(dh_bar[:, None, :] / T, T, axis=1).reshape(B, L, d)
    return dx_router, dW_r


def backward(x, w_r, W1, W2, W3, T, dy, prefix=False, first_grad=False):
    """Full backward of Algorithm 1 given dL/dy.
    Returns dict(dx, dw_r, dW1, dW2, dW3, d_route_w) where d_route_w [S,E] is
    the gradient wrt the shifted routing weights (row n = 0 included, before
    the stop-gradient discards it) and dx includes the router path."""
    x, dy = _f64(x), _f64(dy)
    B, L, d = x.shape
    N = L // T
    h_bar, p, w = route(x, w_r, T, prefix)
    dseg_x, dW1, dW2, dW3, dw = moe_ffn_backward(
        x.reshape(B * N, T, d), w, W1, W2, W3, dy.reshape(B * N, T, d))
    dx_router, dW_r = router_backward(x.shape, T, h_bar, p, w_r, dw, prefix, first_grad)
    return dict(dx=dseg_x.reshape(B, L, d) + dx_router, dw_r=dW_r,
                dW1=dW1, dW2=dW2, dW3=dW3, d_route_w=dw)


# --------------------------------------------------------------------------
# The layer inside a pre-norm residual block (Section 4.1: the models follow
# LLaMA, whose feed-forward sub-layer is  y = x + FFN(RMSNorm(x))).  The paper
# does not write the normalisation out; the reading taken here is the usual
# RMSNorm(x) = x / sqrt(mean_j x_j^2 + eps) * gamma, per token.
# --------------------------------------------------------------------------
def rmsnorm(x, gamma, eps):
    """Returns (x_hat [B,L,d], inv_rms [B,L,1])."""
    x, gamma = _f64(x), _f64(gamma)
    inv = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    return x * inv * gamma, inv


def rmsnorm_backward(x, gamma, inv, dxh):
    """Gradient of rmsnorm wrt x and gamma given dL/dx_hat.  With n = x * inv:
    dn = dxh * gamma,  dx = inv * (dn - n * mean_j(dn_j n_j)),  dgamma = sum over tokens of dxh * n."""
    x, gamma, dxh = _f64(x), _f64(gamma), _f64(dxh)
    n = x * inv
    dn = dxh * gamma
    dx = inv * (dn - n * (dn * n).mean(axis=-1, keepdims=True))
    dgamma = (dxh * n).reshape(-1, x.shape[-1]).sum(axis=0)
    return dx, dgamma


def block_forward(x, gamma, eps, w_r, W1, W2, W3, T, prefix=False):
    """y = x + Lory(RMSNorm(x)).  Returns (y, w, p)."""
    xh, _ = rmsnorm(x, gamma, eps)
    y, w, p = forward(xh, w_r, W1, W2, W3, T, prefix)
    return _f64(x) + y, w, p


def block_backward(x, gamma, eps, w_r, W1, W2, W3, T, dy, prefix=False, first_grad=False):
    """Backward of block_forward.  Returns the dict of `backward` with dx replaced by the gradient wrt the block
    input (the residual path adds dy) and with dgamma added."""
    xh, inv = rmsnorm(x, gamma, eps)
    g = backward(xh, w_r, W1, W2, W3, T, dy, prefix, first_grad)
    dx_norm, dgamma = rmsnorm_backward(x, gamma, inv, g["dx"])
    g = dict(g)
    g["dx"] = dx_norm + _f64(dy)
    g["dgamma"] = dgamma
    return g


# --------------------------------------------------------------------------
# Sampled backward for sizes where keeping every segment's merged-weight
# gradient does not fit: everything that carries an FFN-hidden index i
# (rows of W1/W3, columns of W2, columns of G, U, H and their gradients) is
# computed for the chosen rows only.  dx and dw contract over all of f and
# are therefore not produced here.
# --------------------------------------------------------------------------
def backward_frows(x, w_r, W1, W2, W3, T, dy, rows):
    """dW1[:, rows, :], dW3[:, rows, :], dW2[:, :, rows] of the full layer.
    Returns (dW1_rows [E,r,d], dW2_cols [E,d,r], dW3_rows [E,r,d])."""
    rows = np.asarray(rows, dtype=np.int64)
    x, dy = _f64(x), _f64(dy)
    B, L, d = x.shape
    N = L // T
    S = B * N
    _, _, w = route(x, w_r, T)
    W1r = _f64(np.asarray(W1)[:, rows, :])
    W3r = _f64(np.asarray(W3)[:, rows, :])
    W2c = _f64(np.asarray(W2)[:, :, rows])
    E, r = W1r.shape[0], len(rows)
    seg_x = x.reshape(S, T, d)
    seg_dy = dy.reshape(S, T, d)
    dWb1 = np.empty((S, r, d), F64)
    dWb2 = np.empty((S, d, r), F64)
    dWb3 = np.empty((S, r, d), F64)
    for s in range(S):
        Wb1 = merge_experts(w[s], W1r)
        Wb3 = merge_experts(w[s], W3r)
        Wb2 = merge_experts(w[s], W2c)
        X, dY = seg_x[s], seg_dy[s]
        G = X @ Wb1.T
        U = X @ Wb3.T
        sig = 1.0 / (1.0 + np.exp(-G))
        H = G * sig * U
        dH = dY @ Wb2
        dG = dH * U * sig * (1.0 + G * (1.0 - sig))
        dU = dH * G * sig
        dWb2[s] = dY.T @ H
        dWb1[s] = dG.T @ X
        dWb3[s] = dU.T @ X
    wT = np.ascontiguousarray(w.T)
    dW1r = (wT @ dWb1.reshape(S, -1)).reshape(E, r, d)
    dW2c = (wT @ dWb2.reshape(S, -1)).reshape(E, d, r)
    dW3r = (wT @ dWb3.reshape(S, -1)).reshape(E, r, d)
    return dW1r, dW2c, dW3r


def backward_segments(x, w_r, W1, W2, W3, T, dy, seg_ids):
    """For selected segments s: the FFN-path part of dx_s, and the routing
    gradient row dw_s (which contracts over every parameter).
    Returns {s: (dx_ffn_s [T,d], dw_s [E])}."""
    x, dy = _f64(x), _f64(dy)
    W1, W2, W3 = map(_f64, (W1, W2, W3))
    B, L, d = x.shape
    S = B * (L // T)
    E = W1.shape[0]
    _, _, w = route(x, w_r, T)
    seg_x = x.reshape(S, T, d)
    seg_dy = dy.reshape(S, T, d)
    out = {}
    for s in seg_ids:
        s = int(s)
        Wb1 = merge_experts(w[s], W1)
        Wb3 = merge_experts(w[s], W3)
        Wb2 = merge_experts(w[s], W2)
        dX, dWb1, dWb2, dWb3 = _segment_grads(seg_x[s], seg_dy[s], Wb1, Wb2, Wb3)
        dw_s = (W1.reshape(E, -1) @ dWb1.ravel() + W2.reshape(E, -1) @ dWb2.ravel()
                + W3.reshape(E, -1) @ dWb3.ravel())
        out[s] = (dX, dw_s)
    return out


def backward_every_segment(x, w_r, W1, W2, W3, T, dy, d_rows, group=8):
    """Everything of the backward that contracts over the whole FFN-hidden dimension, for every segment
    and without keeping the per-segment merged-weight gradients of the whole batch: the FFN-path part of
    dx, the routing gradient dw (whole table), and, for the chosen hidden-state indices `d_rows`, the
    slices dW2[:, d_rows, :], dW1[:, :, d_rows], dW3[:, :, d_rows] of the expert gradients
    (dWk_e = sum_s w_{s,e} dWbar_k,s, accumulated over the segments).
    Segments are taken `group` at a time only so that the experts are read once per group: the merge of a
    group is the matrix product w[group] . theta (Eq. 2 for several s), dw of a group is dWbar[group] . theta^T.
    Returns (dx_ffn [S,T,d], dw [S,E], dW2_rows [E,r,f], dW1_cols [E,f,r], dW3_cols [E,f,r])."""
    d_rows = np.asarray(d_rows, dtype=np.int64)
    x, dy = _f64(x), _f64(dy)
    W1, W2, W3 = map(_f64, (W1, W2, W3))
    B, L, d = x.shape
    S = B * (L // T)
    E, f, _ = W1.shape
    _, _, w = route(x, w_r, T)
    seg_x = x.reshape(S, T, d)
    seg_dy = dy.reshape(S, T, d)
    W1f, W2f, W3f = W1.reshape(E, -1), W2.reshape(E, -1), W3.reshape(E, -1)
    dx_ffn = np.empty((S, T, d), F64)
    dw = np.empty((S, E), F64)
    r = len(d_rows)
    dW2_rows = np.zeros((E, r, f), F64)
    dW1_cols = np.zeros((E, f, r), F64)
    dW3_cols = np.zeros((E, f, r), F64)
    for s0 in range(0, S, group):
        s1 = min(S, s0 + group)
        g = s1 - s0
        Wb1 = (w[s0:s1] @ W1f).reshape(g, f, d)
        Wb3 = (w[s0:s1] @ W3f).reshape(g, f, d)
        Wb2 = (w[s0:s1] @ W2f).reshape(g, d, f)
        dWb1, dWb2, dWb3 = np.empty_like(Wb1), np.empty_like(Wb2), np.empty_like(Wb3)
        for i in range(g):
            dx_ffn[s0 + i], dWb1[i], dWb2[i], dWb3[i] = _segment_grads(seg_x[s0 + i], seg_dy[s0 + i], Wb1[i], Wb2[i], Wb3[i])
        dw[s0:s1] = (dWb1.reshape(g, -1) @ W1f.T + dWb2.reshape(g, -1) @ W2f.T + dWb3.reshape(g, -1) @ W3f.T)
        wT = np.ascontiguousarray(w[s0:s1].T)                    # [E, g]
        dW2_rows += (wT @ dWb2[:, d_rows, :].reshape(g, -1)).reshape(E, r, f)
        dW1_cols += (wT @ dWb1[:, :, d_rows].reshape(g, -1)).reshape(E, f, r)
        dW3_cols += (wT @ dWb3[:, :, d_rows].reshape(g, -1)).reshape(E, f, r)
    return dx_ffn, dw, dW2_rows, dW1_cols, dW3_cols


# --------------------------------------------------------------------------
# Inference (Section 3.1 "Prompt-only routing during inference"; appendix
# "Inference Methods") and the expert-utilisation statistic (appendix
# "Expert Utilization")
# --------------------------------------------------------------------------
def prompt_routing_weights(x_prompt, w_r):
    """One routing decision per sequence from the mean hidden state of its whole
    prompt: w_b = softmax(R(mean over the prompt)).  x_prompt [B, Lp, d] -> [B, E]."""
    x_prompt = _f64(x_prompt)
    return router_probs(x_prompt.sum(axis=1) / x_prompt.shape[1], w_r)


def prompt_only_inference(x_prompt, x_new, w_r, W1, W2, W3):
    """The prompt fixes one merged FFN per sequence, which then processes the
    prompt's tokens and every later token of that sequence like a dense FFN.
    x_prompt [B, Lp, d], x_new [B, n, d] -> (y_prompt, y_new, w [B, E])."""
    w = prompt_routing_weights(x_prompt, w_r)
    return moe_ffn(x_prompt, w, W1, W2, W3), moe_ffn(x_new, w, W1, W2, W3), w


def expert_utilization(route_w):
    """Number of segments that activate each expert, an expert counting as activated
    for a segment when its routing weight exceeds 2/E.  route_w [S, E] -> int64 [E]."""
    route_w = _f64(route_w)
    return (route_w > 2.0 / route_w.shape[1]).sum(axis=0).astype(np.int64)


# --------------------------------------------------------------------------
# FLOP model (Appendix B)
# --------------------------------------------------------------------------
def ffn_flops(tokens, d, f):
    """Forward FLOPs of a SwiGLU FFN over `tokens` tokens: 6 * L * d * d'."""
    return 6 * tokens * d * f


def merge_flops(E, d, f):
    """Forward FLOPs of one merge of E experts (three matrices): 6 * E * d * d'."""
    return 6 * E * d * f


def layer_flops(B, L, T, d, f, E, backward=True):
    """FFN plus one merge per segment; the backward costs twice the forward
    (each product has two adjoints)."""
    fwd = ffn_flops(B * L, d, f) + (B * L // T) * merge_flops(E, d, f)
    return 3 * fwd if backward else fwd


def merge_overhead(E, T):
    """Extra FLOPs of the MoE layer relative to a dense FFN: E / T."""
    return E / T
