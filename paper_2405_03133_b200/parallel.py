"""Expert-wise model parallelism of the layer (Section 6 of the Lory paper).

Every rank holds the same slice of the FFN hidden dimension of ALL experts: rows [f0, f1) of every W1_e and
W3_e and columns [f0, f1) of every W2_e.  Activations x, dY and the router W_r are replicated, so every rank
computes the same routing weights.  Each rank runs the ordinary layer on its slice (the C-ABI calls with
f = f1 - f0); what is exchanged are activations only:

  forward    y       = sum over ranks of the partial outputs                       (one all-reduce)
  backward   dx      = sum over ranks of the partial input gradients               (one all-reduce)
             dW_r    = sum over ranks                                              (one all-reduce)
             dW1_e, dW3_e rows / dW2_e columns of the slice are complete locally   (no exchange)

The router path needs no extra exchange: the gradient of the routing weights a rank obtains is the partial sum
over its slice of <dtheta_s, theta_e>, and the router's backward (shift, softmax, linear, mean) is linear in that
gradient, so the sum over ranks of the per-rank router gradients equals the router gradient of the full sum.
Summing dx (which contains the router path) and dW_r over ranks is therefore exact.

This module holds only the slicing and the order of the exchanges; the computation is passed in as callables
(the CUDA binding in production, see `cuda_layer_fns`), the exchange as an `all_reduce(tensor)` callable
(torch.distributed over NCCL in production).
"""
from __future__ import annotations

from typing import Callable, Dict, Tuple


def shard_range(f: int, rank: int, world: int, multiple: int = 8) -> Tuple[int, int]:
    """Slice [f0, f1) of the hidden dimension owned by `rank`: as even as possible in units of `multiple`
    (the bf16 kernels want f % 8 == 0 on every rank); the last rank takes what is left."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    if f % multiple != 0:
        raise ValueError(f"f = {f} is not a multiple of {multiple}")
    units = f // multiple
    if units < world:
        raise ValueError(f"f = {f} has fewer than {world} slices of {multiple}")
    base, extra = divmod(units, world)
    start = rank * base + min(rank, extra)
    size = base + (1 if rank < extra else 0)
    return start * multiple, (start + size) * multiple


def shard_experts(W1, W2, W3, rank: int, world: int, multiple: int = 8):
    """This rank's contiguous slices of the stacked experts: W1, W3 [E, f, d] by rows, W2 [E, d, f] by columns.
    Works on anything sliceable with `.contiguous()` (torch) or numpy arrays."""
    f = W1.shape[1]
    f0, f1 = shard_range(f, rank, world, multiple)

    def contiguous(a):
        return a.contiguous() if hasattr(a, "contiguous") else a.copy()

    return contiguous(W1[:, f0:f1, :]), contiguous(W2[:, :, f0:f1]), contiguous(W3[:, f0:f1, :])


def sharded_forward(run_forward: Callable, all_reduce: Callable, x, w_r, W1s, W2s, W3s):
    """run_forward(x, w_r, W1s, W2s, W3s) -> (y_partial, route_w).  Returns (y, route_w) with y summed over ranks."""
    y, route_w = run_forward(x, w_r, W1s, W2s, W3s)
    all_reduce(y)
    return y, route_w


def sharded_backward(run_backward: Callable, all_reduce: Callable, x, w_r, W1s, W2s, W3s, dy) -> Dict[str, object]:
    """run_backward(x, w_r, W1s, W2s, W3s, dy) -> dict(dx, dw_r, dW1, dW2, dW3[, d_route_w]) of this rank's slice.
    dx, dw_r (and d_route_w if present) are summed over ranks in place; dW1, dW2, dW3 stay local."""
    g = run_backward(x, w_r, W1s, W2s, W3s, dy)
    all_reduce(g["dx"])
    all_reduce(g["dw_r"])
    if g.get("d_route_w") is not None:
        all_reduce(g["d_route_w"])
    return g


def cuda_layer_fns(B: int, L: int, T: int, dtype: str = "bf16", flags: int = 0):
    """The two callables for `sharded_forward` / `sharded_backward` on this process's current CUDA device, built
    on the C-ABI calls; the workspace is allocated on the first call and kept for the backward."""
    import torch
    from . import binding as lory

    state = {}

    def dims_for(W1s):
        E, f_local, d = W1s.shape
        return lory.make_dims(B, L, T, d, f_local, E, dtype, flags)

    def run_forward(x, w_r, W1s, W2s, W3s):
        dims = dims_for(W1s)
        _, bwd = lory.lory_moe_workspace_bytes(dims)
        if state.get("ws") is None or state["ws"].numel() < bwd:
            state["ws"] = torch.empty(bwd, dtype=torch.uint8, device=x.device)
        y = torch.empty_like(x)
        S = B * (L // T)
        route_w = torch.empty((S, W1s.shape[0]), dtype=torch.float32, device=x.device)
        lory.lory_moe_forward(dims, x, w_r, W1s, W2s, W3s, y, route_w, None, state["ws"])
        return y, route_w

    def run_backward(x, w_r, W1s, W2s, W3s, dy):
        dims = dims_for(W1s)
        S = B * (L // T)
        g = dict(dx=torch.empty_like(x), dw_r=torch.empty_like(w_r), dW1=torch.empty_like(W1s),
                 dW2=torch.empty_like(W2s), dW3=torch.empty_like(W3s),
                 d_route_w=torch.empty((S, W1s.shape[0]), dtype=torch.float32, device=x.device))
        lory.lory_moe_backward(dims, x, w_r, W1s, W2s, W3s, dy, g["dx"], g["dw_r"], g["dW1"], g["dW2"], g["dW3"],
                               g["d_route_w"], state["ws"])
        lory.lory_check_status(dims, state["ws"])
        return g

    return run_forward, run_backward


def torch_all_reduce(group=None, accumulate_in_fp32: bool = True):
    """all_reduce callable over torch.distributed (NCCL on GPUs, gloo on CPU): sum, in place.

    The partial y and dx of the slices are bf16 tensors in bf16 mode.  Summed as they are, a ring or tree of R
    ranks rounds the running sum to bf16 up to R - 1 times, on top of the rounding each slice already carries.
    With accumulate_in_fp32 (the default) a 16-bit tensor is widened to fp32, all-reduced, and rounded ONCE on
    the way back: twice the bytes on the wire for the small activation tensors (never for weights, which are
    not exchanged), and a result that does not depend on the number of ranks or on the reduction order beyond
    fp32 rounding."""
    import torch
    import torch.distributed as dist

    def all_reduce(t):
        if accumulate_in_fp32 and t.dtype in (torch.bfloat16, torch.float16):
            wide = t.float()
            dist.all_reduce(wide, op=dist.ReduceOp.SUM, group=group)
            t.copy_(wide)
        else:
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)

    return all_reduce
