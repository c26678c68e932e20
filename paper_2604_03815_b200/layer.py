"""The full multi-head k-MIP self-attention layer of the paper (Eq. 2; Algorithm 1 with its
"Require" line and line 8): Q, K, V projections of the node features in front of the attention
core and the output projection sum_h O^h W_O^h behind it, as a torch module with autograd.

The attention core (scores, top-k, softmax, gather-V and its sparse backward) runs in the
library's kernels through the two C-ABI calls; the four projections are plain dense GEMMs and
use torch's (library GEMMs are what the paper's own implementation uses there too).  The
selection is held constant in the backward pass (Sec. 3.1): gradients flow through the k kept
scores only.
"""
import math

import torch

from . import binding as kb


class KMIPAttentionFunction(torch.autograd.Function):
    """out = kMIP-Attn(Q, K, V) over CSR-batched graphs; Q, K, V: [N, H, d] contiguous."""

    @staticmethod
    def forward(ctx, Q, K, V, graph_offsets, k, mode):
        Q, K, V = Q.contiguous(), K.contiguous(), V.contiguous()
        fb = kb.forward(Q, K, V, graph_offsets, k, mode, check=False)
        ctx.save_for_backward(Q, K, V, fb.out, fb.topk_idx, fb.topk_score)
        ctx.graph_offsets, ctx.k, ctx.mode, ctx.fwd_workspace = graph_offsets, k, mode, fb.workspace
        ctx.mark_non_differentiable(fb.topk_idx)
        return fb.out, fb.topk_idx

    @staticmethod
    def backward(ctx, d_out, _d_idx):
        Q, K, V, out, topk_idx, topk_score = ctx.saved_tensors
        st = kb.kmip_last_status(ctx.fwd_workspace)  # device-side problems of the forward surface here at the latest
        if st != kb.KMIP_OK:
            raise kb.KmipError(st, "kmip_attn_forward (device)")
        fwd = _Saved(out, topk_idx, topk_score)
        bb = kb.backward(Q, K, V, ctx.graph_offsets, ctx.k, ctx.mode, fwd, d_out.contiguous(), check=True)
        return bb.dQ, bb.dK, bb.dV, None, None, None


class _Saved:
    def __init__(self, out, topk_idx, topk_score):
        self.out, self.topk_idx, self.topk_score = out, topk_idx, topk_score


class KMIPSelfAttention(torch.nn.Module):
    """x [N, d_model] -> [N, d_model]: per head h, Q^h = x W_Q^h, K^h = x W_K^h, V^h = x W_V^h,
    O^h = kMIP-Attn(Q^h, K^h, V^h) restricted to each graph, y = sum_h O^h W_O^h (Eq. 2).

    d_head must be 16, 32, 64 or 128 and k <= 128.  dtype bfloat16 selects the tensor-core mode,
    float32 the fp32 mode."""

    def __init__(self, d_model, num_heads, d_head, k, dtype=torch.bfloat16, device="cuda", bias=False):
        super().__init__()
        if dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("dtype must be torch.bfloat16 or torch.float32")
        self.d_model, self.H, self.d, self.k = d_model, num_heads, d_head, k
        self.mode = kb.KMIP_BF16_TC if dtype == torch.bfloat16 else kb.KMIP_FP32_EXACT
        inner = num_heads * d_head
        self.w_q = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_k = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_v = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_o = torch.nn.Linear(inner, d_model, bias=bias, device=device, dtype=dtype)
        for lin in (self.w_q, self.w_k, self.w_v, self.w_o):
            torch.nn.init.normal_(lin.weight, std=1.0 / math.sqrt(lin.in_features))

    def forward(self, x, graph_offsets=None, return_indices=False):
        N = x.shape[0]
        q = self.w_q(x).view(N, self.H, self.d)
        k = self.w_k(x).view(N, self.H, self.d)
        v = self.w_v(x).view(N, self.H, self.d)
        o, idx = KMIPAttentionFunction.apply(q, k, v, graph_offsets, self.k, self.mode)
        y = self.w_o(o.reshape(N, self.H * self.d))
        return (y, idx) if return_indices else y
