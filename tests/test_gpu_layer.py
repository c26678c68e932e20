"""The full attention layer (Eq. 2: projections, k-MIP attention core, output projection) against an
fp64 PyTorch restatement on the CPU: same bf16-rounded weights and inputs, the selection the GPU made
is checked against dense fp64 scores and then held fixed, as the paper's backward pass holds it."""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _bf16_st(t):
    """Round to bf16 with a straight-through gradient (the GPU stores Q, K, V and O in bf16)."""
    return t + (t.to(torch.bfloat16).to(t.dtype) - t).detach()


def _reference(x, wq, wk, wv, wo, idx, H, d, rounding):
    N = x.shape[0]
    r = _bf16_st if rounding else (lambda t: t)
    q = r(x @ wq.T).view(N, H, d)
    k = r(x @ wk.T).view(N, H, d)
    v = r(x @ wv.T).view(N, H, d)
    safe = idx.clamp(min=0).long()                                  # [N, H, k]
    hh = torch.arange(H)[None, :, None].expand_as(safe)
    ks, vs = k[safe, hh], v[safe, hh]                               # [N, H, k, d]
    s = (q[:, :, None, :] * ks).sum(-1) / math.sqrt(d)
    s = s.masked_fill(idx < 0, float("-inf"))
    p = torch.softmax(s, dim=-1)
    o = r((p[..., None] * vs).sum(2))
    return r(o.reshape(N, H * d) @ wo.T), q, k


@pytest.mark.parametrize("dtype,d_head,k", [(torch.bfloat16, 16, 8), (torch.bfloat16, 32, 16), (torch.float32, 32, 5),
                                            (torch.float32, 10, 10), (torch.bfloat16, 40, 6)])
def test_layer_forward_and_gradients(dtype, d_head, k):
    from paper_2604_03815_b200.layer import KMIPSelfAttention

    torch.manual_seed(1234)
    d_model, H = 64, 4
    sizes = [200, 1, 300, 37]
    N = sum(sizes)
    offs = torch.tensor(np.concatenate([[0], np.cumsum(sizes)]), dtype=torch.int32, device="cuda")
    layer = KMIPSelfAttention(d_model, H, d_head, k, dtype=dtype)
    x = torch.randn(N, d_model, device="cuda").to(dtype).requires_grad_(True)
    g = torch.randn(N, d_model, device="cuda").to(dtype)
    y, idx = layer(x, offs, return_indices=True)
    (y.float() * g.float()).sum().backward()
    torch.cuda.synchronize()

    # fp64 restatement with the same (rounded) parameters
    x64 = x.detach().double().cpu().requires_grad_(True)
    ws = [p.detach().double().cpu().requires_grad_(True) for p in (layer.w_q.weight, layer.w_k.weight, layer.w_v.weight, layer.w_o.weight)]
    idx_c = idx.cpu()
    y64, q64, k64 = _reference(x64, *ws, idx_c, H, d_head, rounding=dtype == torch.bfloat16)
    (y64 * g.double().cpu()).sum().backward()

    # the selection: inside the query's graph, no duplicates, and no selected key worse than the
    # k-th best dense fp64 score by more than 1e-2 relative
    o = offs.cpu().numpy().astype(np.int64)
    qn, kn, idn = q64.detach().numpy(), k64.detach().numpy(), idx_c.numpy()
    for gi in range(len(sizes)):
        lo, hi = o[gi], o[gi + 1]
        if hi == lo:
            continue
        keff = min(k, hi - lo)
        for h in range(H):
            S = qn[lo:hi, h] @ kn[lo:hi, h].T
            kth = np.sort(S, axis=1)[:, ::-1][:, keff - 1]
            sel = idn[lo:hi, h, :keff]
            assert np.all((sel >= lo) & (sel < hi)) and np.all(idn[lo:hi, h, keff:] == -1)
            assert all(len(set(r)) == keff for r in sel.tolist())
            ssel = np.take_along_axis(S, sel - lo, axis=1)
            assert np.all(ssel.min(axis=1) >= kth - 1e-2 * np.abs(kth))

    def close(a, b, what):
        a, b = a.double().cpu(), b.double()
        tol = (3e-2 if dtype == torch.bfloat16 else 2e-4) * max(1.0, float(b.abs().max()))
        assert float((a - b).abs().max()) <= tol, f"{what}: {float((a - b).abs().max()):.3e} > {tol:.3e}"

    close(y.detach(), y64.detach(), "output")
    close(x.grad, x64.grad, "d/dx")
    for p, w64, name in zip((layer.w_q.weight, layer.w_k.weight, layer.w_v.weight, layer.w_o.weight), ws, "QKVO"):
        close(p.grad, w64.grad, f"d/dW_{name}")


def test_layer_attention_dropout_only_in_training():
    from paper_2604_03815_b200.layer import KMIPSelfAttention

    torch.manual_seed(7)
    layer = KMIPSelfAttention(32, 2, 16, 8, attn_dropout=0.5)
    x = torch.randn(300, 32, device="cuda").to(torch.bfloat16)
    layer.eval()
    a, b = layer(x), layer(x)
    assert torch.equal(a, b)
    layer.train()
    torch.manual_seed(11)
    c = layer(x)
    torch.manual_seed(11)
    d = layer(x)
    e = layer(x)
    assert torch.equal(c, d) and not torch.equal(c, e) and not torch.equal(c, a)
    xg = x.clone().requires_grad_(True)
    layer(xg).float().square().sum().backward()
    assert torch.isfinite(xg.grad.float()).all() and float(xg.grad.float().abs().max()) > 0


def test_forward_only_use_surfaces_device_errors():
    """Under torch.no_grad() no backward call follows, so malformed graph offsets (seen only by the
    device) must raise from the forward call instead of handing back unwritten memory."""
    from paper_2604_03815_b200 import binding as kb
    from paper_2604_03815_b200.layer import KMIPSelfAttention

    torch.manual_seed(7)
    layer = KMIPSelfAttention(32, 2, 16, 4, dtype=torch.bfloat16)
    x = torch.randn(600, 32, device="cuda").to(torch.bfloat16)
    bad = torch.tensor([0, 400, 300, 600], dtype=torch.int32, device="cuda")
    with torch.no_grad():
        with pytest.raises(kb.KmipError) as e:
            layer(x, bad)
    assert e.value.status == kb.KMIP_ERR_BAD_OFFSETS
    good = torch.tensor([0, 300, 600], dtype=torch.int32, device="cuda")
    with torch.no_grad():
        y = layer(x, good)          # the context is still usable
    assert torch.isfinite(y.float()).all()
