"""The layer as a torch.nn.Module: autograd glue over the C-ABI calls (argument marshalling only).

    layer = LoryMoE(d=1024, f=2752, E=32, T=256, dtype=torch.bfloat16, device="cuda")
    y = layer(x)                 # x [B, L, d], L % T == 0
    y.sum().backward()           # x.grad, layer.w_r.grad, layer.W1.grad, layer.W2.grad, layer.W3.grad

Every step of the computation runs in the CUDA library (lory_moe_forward / lory_moe_backward); this file only
allocates the outputs and the workspace and hands pointers over.  Each forward that needs gradients keeps its own
workspace (the merged weights and activations saved for the backward) until its backward has run, so several
calls may be in flight (gradient checkpointing, several micro-batches).  Without gradients the workspace is the
smaller forward-only one and is dropped at once.
"""
from __future__ import annotations

import torch

from . import binding as _lory


def _dtype_name(dtype: torch.dtype) -> str:
    if dtype == torch.bfloat16:
        return "bf16"
    if dtype == torch.float32:
        return "fp32"
    raise TypeError("LoryMoE supports torch.bfloat16 and torch.float32")


class _LoryFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, w_r, W1, W2, W3, T, flags):
        if x.dim() != 3:
            raise ValueError("x must be [B, L, d]")
        B, L, d = x.shape
        E, f, _ = W1.shape
        dims = _lory.make_dims(B, L, T, d, f, E, _dtype_name(x.dtype), flags)
        need_grad = any(ctx.needs_input_grad[:5])
        fwd_b, bwd_b = _lory.lory_moe_workspace_bytes(dims)
        ws = torch.empty(bwd_b if need_grad else fwd_b, dtype=torch.uint8, device=x.device)
        x = x.contiguous()
        y = torch.empty_like(x)
        route_w = torch.empty((B * (L // T), E), dtype=torch.float32, device=x.device)
        stream = torch.cuda.current_stream(x.device).cuda_stream
        _lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, route_w, None, ws, stream)
        if need_grad:
            ctx.save_for_backward(x, w_r, W1, W2, W3)
            ctx.ws, ctx.dims = ws, dims
        ctx.mark_non_differentiable(route_w)
        return y, route_w

    @staticmethod
    def backward(ctx, dy, _d_route_w):
        x, w_r, W1, W2, W3 = ctx.saved_tensors
        dy = dy.contiguous()
        dx = torch.empty_like(x)
        dw_r, dW1, dW2, dW3 = (torch.empty_like(t) for t in (w_r, W1, W2, W3))
        stream = torch.cuda.current_stream(x.device).cuda_stream
        _lory.lory_moe_backward(ctx.dims, x, w_r, W1, W2, W3, dy, dx, dw_r, dW1, dW2, dW3, None, ctx.ws, stream)
        ctx.ws = None                      # the saved merged weights and activations are no longer needed
        return dx, dw_r, dW1, dW2, dW3, None, None


class LoryMoE(torch.nn.Module):
    """Lory mixture-of-experts FFN layer (causal segment routing + expert merging, Sections 3 and 3.1).

    Parameters: w_r [E, d] (router), W1, W3 [E, f, d] (gate, up), W2 [E, d, f] (down), initialised N(0, std).
    forward(x) returns y [B, L, d]; `last_route_w` holds the routing weights [B*L/T, E] of the last call.
    `flags`: LORY_FLAG_* of the binding (prefix routing, first-segment gradient, ...).
    """

    def __init__(self, d: int, f: int, E: int, T: int, dtype=torch.bfloat16, device="cuda", std: float = 0.02,
                 flags: int = 0, generator: torch.Generator | None = None):
        super().__init__()
        self.T, self.flags = int(T), int(flags)

        def init(*shape):
            w = torch.randn(*shape, dtype=torch.float32, device=device, generator=generator) * std
            return torch.nn.Parameter(w.to(dtype))

        self.w_r = init(E, d)
        self.W1 = init(E, f, d)
        self.W2 = init(E, d, f)
        self.W3 = init(E, f, d)
        self.last_route_w = None

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        if not x.is_cuda:
            raise RuntimeError("LoryMoE runs on a CUDA device only (there is no CPU path)")
        y, route_w = _LoryFn.apply(x, self.w_r, self.W1, self.W2, self.W3, self.T, self.flags)
        self.last_route_w = route_w
        return y


class _LoryBlockFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, gamma, w_r, W1, W2, W3, T, eps, flags):
        B, L, d = x.shape
        E, f, _ = W1.shape
        dims = _lory.make_dims(B, L, T, d, f, E, _dtype_name(x.dtype), flags)
        need_grad = any(ctx.needs_input_grad[:6])
        fwd_b, bwd_b = _lory.lory_block_workspace_bytes(dims)
        ws = torch.empty(bwd_b if need_grad else fwd_b, dtype=torch.uint8, device=x.device)
        x = x.contiguous()
        y = torch.empty_like(x)
        route_w = torch.empty((B * (L // T), E), dtype=torch.float32, device=x.device)
        stream = torch.cuda.current_stream(x.device).cuda_stream
        _lory.lory_block_forward(dims, x, gamma, eps, w_r, W1, W2, W3, y, route_w, None, ws, stream)
        if need_grad:
            ctx.save_for_backward(x, gamma, w_r, W1, W2, W3)
            ctx.ws, ctx.dims = ws, dims
        ctx.mark_non_differentiable(route_w)
        return y, route_w

    @staticmethod
    def backward(ctx, dy, _d_route_w):
        x, gamma, w_r, W1, W2, W3 = ctx.saved_tensors
        dy = dy.contiguous()
        dx = torch.empty_like(x)
        dgamma, dw_r, dW1, dW2, dW3 = (torch.empty_like(t) for t in (gamma, w_r, W1, W2, W3))
        stream = torch.cuda.current_stream(x.device).cuda_stream
        _lory.lory_block_backward(ctx.dims, x, gamma, w_r, W1, W2, W3, dy, dx, dgamma, dw_r, dW1, dW2, dW3, None,
                                  ctx.ws, stream)
        ctx.ws = None
        return dx, dgamma, dw_r, dW1, dW2, dW3, None, None, None


class LoryBlock(LoryMoE):
    """The layer inside a pre-norm residual block (the LLaMA block the paper's models use, Section 4.1):
    y = x + LoryMoE(RMSNorm(x; gamma, eps)).  Adds the parameter gamma [d], initialised to one."""

    def __init__(self, d: int, f: int, E: int, T: int, eps: float = 1e-5, dtype=torch.bfloat16, device="cuda",
                 std: float = 0.02, flags: int = 0, generator: torch.Generator | None = None):
        super().__init__(d, f, E, T, dtype=dtype, device=device, std=std, flags=flags, generator=generator)
        self.eps = float(eps)
        self.gamma = torch.nn.Parameter(torch.ones(d, dtype=dtype, device=device))

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        if not x.is_cuda:
            raise RuntimeError("LoryBlock runs on a CUDA device only (there is no CPU path)")
        y, route_w = _LoryBlockFn.apply(x, self.gamma, self.w_r, self.W1, self.W2, self.W3, self.T, self.eps, self.flags)
        self.last_route_w = route_w
        return y


class LoryPromptRoutedFFN:
    """Prompt-only routing at inference (Section 3.1): `prefill` routes each sequence once from its whole prompt
    and leaves the merged FFN of every sequence in a workspace; `decode` then applies that cached FFN to new
    tokens like a dense FFN, with no routing and no merging."""

    def __init__(self, layer: LoryMoE):
        self.layer = layer
        self.ws = None
        self.batch = None

    @torch.no_grad()
    def prefill(self, x_prompt: torch.Tensor) -> torch.Tensor:
        m = self.layer
        B, L, d = x_prompt.shape
        E, f, _ = m.W1.shape
        dims = _lory.make_dims(B, L, L, d, f, E, _dtype_name(x_prompt.dtype), m.flags)
        fwd_b, _ = _lory.lory_moe_workspace_bytes(dims)
        self.ws = torch.empty(fwd_b, dtype=torch.uint8, device=x_prompt.device)
        self.batch = B
        x_prompt = x_prompt.contiguous()
        y = torch.empty_like(x_prompt)
        self.route_w = torch.empty((B, E), dtype=torch.float32, device=x_prompt.device)
        # on the stream torch is issuing this tensor's work on, so that the call is ordered with its producers and
        # consumers (and with later decode() calls, which share the cached workspace)
        _lory.lory_moe_forward(dims, x_prompt, m.w_r, m.W1, m.W2, m.W3, y, self.route_w, None, self.ws,
                               torch.cuda.current_stream(x_prompt.device))
        return y

    @torch.no_grad()
    def decode(self, x_new: torch.Tensor) -> torch.Tensor:
        if self.ws is None:
            raise RuntimeError("call prefill() first")
        m = self.layer
        B, n, d = x_new.shape
        if B != self.batch:
            raise ValueError("decode() needs the batch of the prefill() whose merged FFNs are cached")
        E, f, _ = m.W1.shape
        dims = _lory.make_dims(B, n, n, d, f, E, _dtype_name(x_new.dtype), m.flags | _lory.LORY_FLAG_REUSE_MERGED)
        need, _ = _lory.lory_moe_workspace_bytes(dims)
        if need > self.ws.numel():
            raise ValueError("more new tokens per sequence than the prompt had: the cached workspace is too small")
        x_new = x_new.contiguous()
        y = torch.empty_like(x_new)
        _lory.lory_moe_ffn(dims, x_new, None, m.W1, m.W2, m.W3, y, self.ws, torch.cuda.current_stream(x_new.device))
        return y
