"""The full multi-head k-MIP self-attention layer of the paper (Eq. 2; Algorithm 1 with its
"Require" line and line 8): Q, K, V projections of the node features in front of the attention
core and the output projection sum_h O^h W_O^h behind it, as a torch module with autograd.

In bfloat16 without attention dropout or pruning the whole layer - projections, attention core,
output projection and every product of the backward pass - runs in the library's kernels through
kmip_layer_forward / kmip_layer_backward (the projections on the tensor cores, csrc/gemm_tn.cu).
Otherwise (float32, dropout, the pruned mode) the attention core runs through kmip_attn_forward /
kmip_attn_backward and the four projections are torch's dense GEMMs.  The selection is held constant
in the backward pass (Sec. 3.1): gradients flow through the k kept scores only.
"""
import math

import torch

from . import binding as kb


class KMIPAttentionFunction(torch.autograd.Function):
    """out = kMIP-Attn(Q, K, V) over CSR-batched graphs; Q, K, V: [N, H, d] contiguous."""

    @staticmethod
    def forward(ctx, Q, K, V, graph_offsets, k, mode, drop_p=0.0, seed=0):
        Q, K, V = Q.contiguous(), K.contiguous(), V.contiguous()
        N, H, d = Q.shape
        G = 1 if graph_offsets is None else int(graph_offsets.numel()) - 1
        fb = kb.ForwardBuffers(N, G, H, d, k, mode, Q.device)
        rc = kb.kmip_attn_forward_dropout(Q, K, V, graph_offsets, k, mode, drop_p, seed, fb.out, fb.topk_idx,
                                          fb.topk_score, fb.workspace)
        if rc != kb.KMIP_OK:
            raise kb.KmipError(rc, "kmip_attn_forward_dropout")
        if not any(ctx.needs_input_grad[:3]):
            # no backward call will follow (eval, no_grad), so a device-side problem (malformed offsets, an
            # expired bounded wait) has to surface here: the kernels after it leave `out` unwritten
            st = kb.kmip_last_status(fb.workspace)
            if st != kb.KMIP_OK:
                raise kb.KmipError(st, "kmip_attn_forward (device)")
        ctx.save_for_backward(Q, K, V, fb.out, fb.topk_idx, fb.topk_score)
        ctx.graph_offsets, ctx.k, ctx.mode, ctx.fwd_workspace = graph_offsets, k, mode, fb.workspace
        ctx.drop_p, ctx.seed = drop_p, seed
        ctx.mark_non_differentiable(fb.topk_idx)
        return fb.out, fb.topk_idx

    @staticmethod
    def backward(ctx, d_out, _d_idx):
        Q, K, V, out, topk_idx, topk_score = ctx.saved_tensors
        st = kb.kmip_last_status(ctx.fwd_workspace)  # device-side problems of the forward surface here at the latest
        if st != kb.KMIP_OK:
            raise kb.KmipError(st, "kmip_attn_forward (device)")
        N, H, d = Q.shape
        G = 1 if ctx.graph_offsets is None else int(ctx.graph_offsets.numel()) - 1
        bb = kb.BackwardBuffers(N, G, H, d, ctx.k, ctx.mode, Q.device)
        rc = kb.kmip_attn_backward_dropout(Q, K, V, ctx.graph_offsets, ctx.k, ctx.mode, ctx.drop_p, ctx.seed, out,
                                           d_out.contiguous(), topk_idx, topk_score, bb.dQ, bb.dK, bb.dV, bb.workspace)
        if rc != kb.KMIP_OK:
            raise kb.KmipError(rc, "kmip_attn_backward_dropout")
        st = kb.kmip_last_status(bb.workspace)
        if st != kb.KMIP_OK:
            raise kb.KmipError(st, "kmip_attn_backward_dropout (device)")
        return bb.dQ, bb.dK, bb.dV, None, None, None, None, None


class KMIPLayerFunction(torch.autograd.Function):
    """y = sum_h kMIP-Attn(x W_Q^h, x W_K^h, x W_V^h) W_O^h, bf16, through kmip_layer_forward / kmip_layer_backward."""

    @staticmethod
    def forward(ctx, x, w_q, w_k, w_v, w_o, graph_offsets, H, d_head, k):
        x, w_q, w_k, w_v, w_o = (t.contiguous() for t in (x, w_q, w_k, w_v, w_o))
        N, d_model = x.shape
        d_pad = next(w for w in (16, 32, 64, 128) if w >= d_head)
        G = 1 if graph_offsets is None else int(graph_offsets.numel()) - 1
        dev = x.device
        mk = lambda *shape, dtype=torch.bfloat16: torch.empty(shape, dtype=dtype, device=dev)
        t = {"x": x, "w_q": w_q, "w_k": w_k, "w_v": w_v, "w_o": w_o,
             "q": mk(N, H, d_pad), "k": mk(N, H, d_pad), "v": mk(N, H, d_pad), "o": mk(N, H, d_pad),
             "topk_idx": mk(N, H, k, dtype=torch.int32), "topk_score": mk(N, H, k, dtype=torch.float32),
             "y": mk(N, d_model), "d_y": None, "d_x": None, "dw_q": None, "dw_k": None, "dw_v": None, "dw_o": None}
        ws = torch.empty(kb.kmip_layer_workspace_bytes(N, G, d_model, H, d_head, k, kb.PASS_FORWARD), dtype=torch.uint8, device=dev)
        rc = kb.kmip_layer_forward(t, graph_offsets, N, d_model, H, d_head, k, ws)
        if rc != kb.KMIP_OK:
            raise kb.KmipError(rc, "kmip_layer_forward")
        if N > 0:
            st = kb.kmip_last_status(ws)     # the workspace is released right after, so device problems surface here
            if st != kb.KMIP_OK:
                raise kb.KmipError(st, "kmip_layer_forward (device)")
        ctx.save_for_backward(x, w_q, w_k, w_v, w_o, t["q"], t["k"], t["v"], t["o"], t["topk_idx"], t["topk_score"])
        ctx.meta = (graph_offsets, H, d_head, k)
        ctx.mark_non_differentiable(t["topk_idx"])
        return t["y"], t["topk_idx"]

    @staticmethod
    def backward(ctx, d_y, _d_idx):
        x, w_q, w_k, w_v, w_o, q, kk, v, o, idx, score = ctx.saved_tensors
        graph_offsets, H, d_head, k = ctx.meta
        N, d_model = x.shape
        G = 1 if graph_offsets is None else int(graph_offsets.numel()) - 1
        t = {"x": x, "w_q": w_q, "w_k": w_k, "w_v": w_v, "w_o": w_o, "q": q, "k": kk, "v": v, "o": o,
             "topk_idx": idx, "topk_score": score, "y": None, "d_y": d_y.contiguous().to(torch.bfloat16),
             "d_x": torch.empty_like(x), "dw_q": torch.empty_like(w_q), "dw_k": torch.empty_like(w_k),
             "dw_v": torch.empty_like(w_v), "dw_o": torch.empty_like(w_o)}
        ws = torch.empty(kb.kmip_layer_workspace_bytes(N, G, d_model, H, d_head, k, kb.PASS_BACKWARD), dtype=torch.uint8,
                         device=x.device)
        rc = kb.kmip_layer_backward(t, graph_offsets, N, d_model, H, d_head, k, ws)
        if rc != kb.KMIP_OK:
            raise kb.KmipError(rc, "kmip_layer_backward")
        if N > 0:
            st = kb.kmip_last_status(ws)
            if st != kb.KMIP_OK:
                raise kb.KmipError(st, "kmip_layer_backward (device)")
        return t["d_x"], t["dw_q"], t["dw_k"], t["dw_v"], t["dw_o"], None, None, None, None


class KMIPSelfAttention(torch.nn.Module):
    """x [N, d_model] -> [N, d_model]: per head h, Q^h = x W_Q^h, K^h = x W_K^h, V^h = x W_V^h,
    O^h = kMIP-Attn(Q^h, K^h, V^h) restricted to each graph, y = sum_h O^h W_O^h (Eq. 2).

    k <= 128.  The kernels take head widths 16, 32, 64 and 128; any other d_head <= 128 (the paper's own
    study uses 10) is zero-padded to the next of those behind the projections, which leaves every inner
    product unchanged, with the queries scaled by sqrt(padded / d_head) so that the softmax still divides
    the scores by sqrt(d_head) as Eq. 1 does.  dtype bfloat16 selects the tensor-core mode,
    float32 the fp32 mode.  attn_dropout is the dropout rate on the k attention weights, active in
    training mode only (the paper's graph models use 0.5); every forward call draws a fresh seed
    from torch's CPU generator, so torch.manual_seed makes a run repeatable.  prune=True selects the
    tensor-core mode with exact tile skipping (same results, faster on clustered or heavy-tailed keys).
    set_k changes k between calls (the paper's Sec. 6 suggests annealing k during training)."""

    def __init__(self, d_model, num_heads, d_head, k, dtype=torch.bfloat16, device="cuda", bias=False,
                 attn_dropout=0.0, prune=False):
        super().__init__()
        if dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("dtype must be torch.bfloat16 or torch.float32")
        self.d_model, self.H, self.d, self.k = d_model, num_heads, d_head, k
        if not 1 <= d_head <= 128:
            raise ValueError("d_head must be in 1..128")
        self.d_pad = next(w for w in (16, 32, 64, 128) if w >= d_head)
        if not 0.0 <= attn_dropout < 1.0:
            raise ValueError("attn_dropout must be in [0, 1)")
        self.attn_dropout = float(attn_dropout)
        if prune and dtype != torch.bfloat16:
            raise ValueError("prune needs dtype bfloat16 (it is a variant of the tensor-core mode)")
        self.mode = (kb.KMIP_BF16_TC_PRUNED if prune else kb.KMIP_BF16_TC) if dtype == torch.bfloat16 else kb.KMIP_FP32_EXACT
        inner = num_heads * d_head
        self.w_q = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_k = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_v = torch.nn.Linear(d_model, inner, bias=bias, device=device, dtype=dtype)
        self.w_o = torch.nn.Linear(inner, d_model, bias=bias, device=device, dtype=dtype)
        for lin in (self.w_q, self.w_k, self.w_v, self.w_o):
            torch.nn.init.normal_(lin.weight, std=1.0 / math.sqrt(lin.in_features))

    def set_k(self, k):
        if not 1 <= int(k) <= 128:
            raise ValueError("k must be in 1..128")
        self.k = int(k)

    def forward(self, x, graph_offsets=None, return_indices=False):
        N = x.shape[0]
        drop_now = self.attn_dropout if self.training else 0.0
        if (self.mode == kb.KMIP_BF16_TC and drop_now == 0.0 and self.w_q.bias is None and self.d_model % 8 == 0
                and x.dtype == torch.bfloat16):
            # the whole layer in the library's kernels
            y, idx = KMIPLayerFunction.apply(x, self.w_q.weight, self.w_k.weight, self.w_v.weight, self.w_o.weight,
                                             graph_offsets, self.H, self.d, self.k)
            return (y, idx) if return_indices else y
        q = self.w_q(x).view(N, self.H, self.d)
        k = self.w_k(x).view(N, self.H, self.d)
        v = self.w_v(x).view(N, self.H, self.d)
        if self.d_pad != self.d:
            pad = (0, self.d_pad - self.d)
            q = torch.nn.functional.pad(q * math.sqrt(self.d_pad / self.d), pad)
            k, v = torch.nn.functional.pad(k, pad), torch.nn.functional.pad(v, pad)
        drop = self.attn_dropout if self.training else 0.0
        seed = int(torch.randint(0, 2 ** 62, (1,)).item()) if drop > 0.0 else 0
        o, idx = KMIPAttentionFunction.apply(q, k, v, graph_offsets, self.k, self.mode, drop, seed)
        y = self.w_o(o[..., :self.d].reshape(N, self.H * self.d))
        return (y, idx) if return_indices else y
