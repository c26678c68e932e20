"""The full attention layer (Eq. 2: projections, k-MIP attention core, output projection) against the
CPU oracle's layer functions: same bf16-rounded weights and inputs, the selection the GPU made is checked
against the oracle's dense fp64 scores and then held fixed, as the paper's backward pass holds it."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d_head,k", [(torch.bfloat16, 16, 8), (torch.bfloat16, 32, 16), (torch.float32, 32, 5),
                                            (torch.float32, 10, 10), (torch.bfloat16, 40, 6)])
def test_layer_forward_and_gradients(dtype, d_head, k):
    from oracle import kmip_oracle as oracle
    from paper_2604_03815_b200.layer import KMIPSelfAttention

    torch.manual_seed(1234)
    d_model, H = 64, 4
    sizes = [200, 1, 300, 37]
    N = sum(sizes)
    offs_np = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    offs = torch.tensor(offs_np, dtype=torch.int32, device="cuda")
    layer = KMIPSelfAttention(d_model, H, d_head, k, dtype=dtype)
    x = torch.randn(N, d_model, device="cuda").to(dtype).requires_grad_(True)
    g = torch.randn(N, d_model, device="cuda").to(dtype)
    y, idx = layer(x, offs, return_indices=True)
    (y.float() * g.float()).sum().backward()
    torch.cuda.synchronize()

    # the oracle's layer on the same (rounded) parameters, with the GPU's selection
    f64 = lambda t: t.detach().double().cpu().numpy()
    xs, ws = f64(x), [f64(p) for p in (layer.w_q.weight, layer.w_k.weight, layer.w_v.weight, layer.w_o.weight)]
    storage = "bf16" if dtype == torch.bfloat16 else "f32"
    idx_np = idx.cpu().numpy()
    fwd = oracle.layer_forward(xs, *ws, offs_np, H, k, idx=idx_np, storage=storage)
    grads = oracle.layer_backward(xs, *ws, H, fwd, f64(g))

    # the selection: inside the query's graph, no duplicates, and no selected key worse than the
    # k-th best dense fp64 score (of the oracle's own Q and K) by more than 1e-2 relative
    own = oracle.forward(fwd["q"], fwd["k"], fwd["v"], offs_np, k)
    _, exact = oracle.forward_given_idx(fwd["q"], fwd["k"], fwd["v"], idx_np)
    gi = np.searchsorted(offs_np, np.arange(N), side="right") - 1
    lo, hi = offs_np[gi].astype(np.int64), offs_np[gi + 1].astype(np.int64)
    keff = np.minimum(k, hi - lo)
    valid = np.arange(k)[None, None, :] < keff[:, None, None]
    assert np.all(((idx_np >= lo[:, None, None]) & (idx_np < hi[:, None, None])) | ~valid) and np.all((idx_np == -1) | valid)
    srt = np.sort(np.where(valid, idx_np, -1 - np.arange(k)[None, None, :]), axis=-1)
    assert np.all(np.diff(srt, axis=-1) != 0)
    kth = np.take_along_axis(own["score"], np.maximum(keff - 1, 0)[:, None, None].repeat(H, 1), axis=2)[..., 0]
    worst = np.where(valid, exact, np.inf).min(axis=-1)
    assert np.all(worst >= kth - 1e-2 * np.abs(kth))

    def close(a, b, what):
        a = a.detach().double().cpu().numpy()
        tol = (3e-2 if dtype == torch.bfloat16 else 2e-4) * max(1.0, float(np.abs(b).max()))
        assert float(np.abs(a - b).max()) <= tol, f"{what}: {float(np.abs(a - b).max()):.3e} > {tol:.3e}"

    close(y, fwd["y"], "output")
    close(x.grad, grads["dx"], "d/dx")
    for p, name in zip((layer.w_q.weight, layer.w_k.weight, layer.w_v.weight, layer.w_o.weight), "qkvo"):
        close(p.grad, grads["dw_" + name], f"d/dW_{name}")


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


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (300, 200, 72), (1000, 384, 128), (130, 70, 8), (5, 515, 200),
                                   (257, 129, 4104)])
def test_projection_gemm_against_fp64(M, N, K):
    """The tensor-core product behind the projections: ragged tile edges in all three dimensions, several
    K blocks (the ring of shared-memory stages wraps), fp32 and bf16 outputs."""
    from paper_2604_03815_b200 import binding as kb
    g = torch.Generator(device="cpu").manual_seed(M * 7 + N * 3 + K)
    A = torch.randn(M, K, generator=g).to(torch.bfloat16)
    B = torch.randn(N, K, generator=g).to(torch.bfloat16)
    ref = A.double() @ B.double().T
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for dt, tol in ((torch.float32, 1e-5), (torch.bfloat16, 2.0 ** -8)):
        C = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
        assert kb.kmip_test_gemm_tn(A.cuda(), B.cuda(), C, ws) == kb.KMIP_OK
        assert kb.kmip_last_status(ws) == kb.KMIP_OK
        got = C.double().cpu()
        assert torch.isfinite(got).all()
        assert float((got - ref).abs().max()) <= tol * max(1.0, float(ref.abs().max())) + 1e-4 * np.sqrt(K) * (dt == torch.float32)


def test_layer_calls_reject_bad_arguments():
    from paper_2604_03815_b200 import binding as kb
    with pytest.raises(kb.KmipError) as e:
        kb.kmip_layer_workspace_bytes(1000, 1, 60, 2, 16, 8, kb.PASS_FORWARD)      # d_model not a multiple of 8
    assert e.value.status == kb.KMIP_ERR_INVALID_ARG
    with pytest.raises(kb.KmipError) as e:
        kb.kmip_layer_workspace_bytes(1000, 1, 64, 2, 200, 8, kb.PASS_FORWARD)     # head wider than 128
    assert e.value.status == kb.KMIP_ERR_UNSUPPORTED
    f = kb.kmip_layer_workspace_bytes(100_000, 1, 128, 4, 32, 16, kb.PASS_FORWARD)
    b = kb.kmip_layer_workspace_bytes(100_000, 1, 128, 4, 32, 16, kb.PASS_BACKWARD)
    attn_f = kb.kmip_attn_workspace_bytes(100_000, 1, 4, 32, 16, kb.KMIP_BF16_TC, kb.PASS_FORWARD)
    attn_b = kb.kmip_attn_workspace_bytes(100_000, 1, 4, 32, 16, kb.KMIP_BF16_TC, kb.PASS_BACKWARD)
    assert attn_f < f < attn_f + (1 << 20)                                          # + four padded weight copies
    assert attn_b + 10 * 100_000 * 128 * 2 <= b < attn_b + 10 * 100_008 * 128 * 2 + (1 << 21)   # + ten [N, 128] bf16 arrays
