"""The pruned tensor-core mode (KMIP_BF16_TC_PRUNED): keys of large graphs swept in (norm class, pivot)
order, key tiles skipped by the centroid and norm bounds, a variable number of tiles per work item.
Same acceptance rule as the tensor-core mode: a stratified sample of rows against the oracle's brute
force over all keys, structure checks on every row, the backward pass in full on the returned indices."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2604_03815_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2604_03815_b200 import binding as kb
    from tests import parity_util as pu


def _pruned(w):
    return dataclasses.replace(w, mode=kb.KMIP_BF16_TC_PRUNED)


def _check(w, n_sample, backward=True):
    w = _pruned(w)
    dev = pu.to_device(w)
    fb = pu.run_forward(w, dev)
    rows = pu.stratified_rows(w, fb, n_sample)[0] if n_sample >= 4096 else wl.sample_rows(w, n_sample)
    st = pu.check_forward(w, fb, rows)
    idx = fb.topk_idx.cpu().numpy()
    sc = fb.topk_score.cpu().numpy()
    offs = w.graph_offsets.astype(np.int64)
    g = np.searchsorted(offs, np.arange(w.N), side="right") - 1
    keff = np.minimum(w.k, offs[g + 1] - offs[g])[:, None, None]
    valid = np.arange(w.k)[None, None, :] < keff
    assert np.all(((idx >= offs[g][:, None, None]) & (idx < offs[g + 1][:, None, None])) | ~valid)
    assert np.all((idx == -1) | valid)
    assert np.all((sc[..., 1:] <= sc[..., :-1]) | ~valid[..., 1:])
    srt = np.sort(np.where(valid, idx, -1 - np.arange(w.k)[None, None, :]), axis=-1)
    assert np.all(np.diff(srt, axis=-1) != 0), "a key is listed twice"
    if backward:
        st.update(pu.check_backward(w, fb, pu.run_backward(w, fb, dev)))
    return st


def test_clustered_single_graph():
    st = _check(wl.make_config(4, N=40000, H=2, d=32, k=16), 300)
    assert st["identical_rows"] > 0.9


def test_hub_keys_batch():
    st = _check(wl.make_config(5, n_per_graph=20000), 300)
    assert st["identical_rows"] > 0.9


def test_unstructured_data_prunes_nothing_and_still_agrees():
    _check(wl.make_config(3, N=36000), 200)


def test_mixed_batch_small_graphs_keep_their_order():
    sizes = [9000, 300, 20000, 10, 8192, 4000, 0, 8191]
    base = wl.make_config(4, N=sum(sizes), H=2, d=32, k=16)
    offs = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(sizes, out=offs[1:])
    w = wl.Workload(name="mixed", mode=base.mode, H=base.H, d=base.d, k=base.k, graph_offsets=offs.astype(np.int32),
                    Q=base.Q, K=base.K, V=base.V, dOut=base.dOut, backward=True, meta={})
    _check(w, 400)


@pytest.mark.parametrize("d,k", [(64, 32), (128, 8), (32, 64), (64, 64), (16, 128), (128, 64)])
def test_every_kernel_shape(d, k):
    """One case per (query tiles per CTA, key stages, list size) instantiation of the sweep."""
    _check(wl.make_config(4, N=33000, H=1, d=d, k=k), 96, backward=False)


def test_ragged_last_tile_and_short_last_item():
    _check(wl.make_config(4, N=32768 + 385 + 77, H=1, d=32, k=32), 128, backward=False)


def test_same_answer_as_the_full_sweep():
    """Skipping is exact: on data without tied scores both modes return the same keys."""
    w = wl.make_config(4, N=40000, H=2, d=32, k=16)
    dev = pu.to_device(w)
    full = pu.run_forward(w, dev)
    pruned = pu.run_forward(_pruned(w), dev)
    a, b = full.topk_score.cpu().numpy(), pruned.topk_score.cpu().numpy()
    same = np.all(a == b, axis=-1)
    assert same.mean() > 0.999, f"{(~same).sum()} rows differ"
    # where rows differ, it is by a near-tie at the k-th place (the two sweeps met the keys in another order)
    rel = np.abs(a - b).max(axis=-1) / np.maximum(np.abs(a[..., -1]), 1e-6)
    assert rel.max() < 1e-2


def test_config4_500k_point_cloud_pruned():
    st = _check(wl.make_config(4), 4096)
    assert st["identical_rows"] > 0.95


def test_config5_hub_batch_pruned():
    st = _check(wl.make_config(5), 4096)
    assert st["identical_rows"] > 0.95


def test_workspace_of_the_pruned_mode_is_reported_and_enforced():
    N, H, d, k = 40000, 2, 32, 16
    need = kb.kmip_attn_workspace_bytes(N, 1, H, d, k, kb.KMIP_BF16_TC_PRUNED, kb.PASS_FORWARD)
    # the fp32-accumulate sweep without pruning at this size: copies of K and Q, permutation, codes, work items
    plain = 2 * N * H * d * 2 + 6 * N + 20 * (N // 128 + 2) + 8 * 256
    assert plain < need < plain + N * (16 + 4 * H) + (N // 128 + 3) * H * (d + 4) * 4 * 5 + 16 * 256
    w = _pruned(wl.make_config(4, N=N, H=H, d=d, k=k))
    Q, K, V, _, offs = pu.to_device(w)
    fb = kb.ForwardBuffers(N, 1, H, d, k, w.mode)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    assert kb.kmip_attn_forward(Q, K, V, offs, k, w.mode, fb.out, fb.topk_idx, fb.topk_score, small) == kb.KMIP_ERR_WORKSPACE


def test_layer_with_pruning_matches_layer_without():
    """The layer's prune option only changes the mode of the attention core."""
    from paper_2604_03815_b200.layer import KMIPSelfAttention

    torch.manual_seed(5)
    N, d_model = 33000, 64
    cen = torch.randn(16, d_model, device="cuda")
    x = (cen[torch.randint(0, 16, (N,), device="cuda")] + 0.2 * torch.randn(N, d_model, device="cuda")).bfloat16()
    a = KMIPSelfAttention(d_model, 2, 32, 16)
    b = KMIPSelfAttention(d_model, 2, 32, 16, prune=True)
    b.load_state_dict(a.state_dict())
    assert b.mode == kb.KMIP_BF16_TC_PRUNED
    xa, xb = x.clone().requires_grad_(True), x.clone().requires_grad_(True)
    ya, ia = a(xa, return_indices=True)
    yb, ib = b(xb, return_indices=True)
    assert float((ia == ib).float().mean()) > 0.999
    same = (ia == ib).all(dim=-1).all(dim=-1)
    assert torch.allclose(ya[same].float(), yb[same].float(), rtol=2e-2, atol=2e-2)
    ya.float().square().sum().backward()
    yb.float().square().sum().backward()
    assert torch.isfinite(xb.grad.float()).all()
    rel = (xa.grad.float() - xb.grad.float()).norm() / xa.grad.float().norm()
    assert float(rel) < 2e-2
    b.set_k(8)
    assert b(x).shape == (N, d_model)


def _dense_check(Q, K, V, offs, k, n_rows=64, seed=0):
    """Sampled rows of a pruned-mode forward against dense fp32 scores computed by torch on the GPU:
    the kept scores are the row's k largest and every index scores what the list says."""
    fb = kb.forward(Q, K, V, offs, k, kb.KMIP_BF16_TC_PRUNED)   # raises on a device-side status
    N = Q.shape[0]
    lo, hi = offs[:-1].long(), offs[1:].long()
    g = torch.searchsorted(hi.contiguous(), torch.arange(N, device="cuda"), right=True)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for r in torch.randint(0, N, (n_rows,), device="cuda", generator=gen).tolist():
        a, b = int(lo[g[r]]), int(hi[g[r]])
        s = (Q[r].float()[:, None, :] * K[a:b].float().permute(1, 0, 2)).sum(-1)   # [H, n]
        kk = min(k, b - a)
        best = torch.topk(s, kk, dim=1).values
        tol = 2e-4 * max(1.0, float(best.abs().max()))
        assert float((fb.topk_score[r, :, :kk] - best).abs().max()) <= tol, f"row {r}: kept scores are not the k largest"
        idx = fb.topk_idx[r, :, :kk].long()
        assert bool(((idx >= a) & (idx < b)).all())
        got = torch.gather(s, 1, idx - a)
        assert float((got - fb.topk_score[r, :, :kk]).abs().max()) <= tol, f"row {r}: index and score disagree"
        assert all(len(set(row)) == kk for row in idx.tolist()), f"row {r}: a key is listed twice"
    return fb


@pytest.mark.parametrize("case", ["zero_keys", "identical_keys", "negative_scores", "one_giant_key", "zero_queries",
                                  "two_scales"])
def test_degenerate_values(case):
    """Values that stress the bounds: thresholds that stay at or below zero (the norm bound must not fire),
    radii of zero, norms spread over many orders of magnitude."""
    torch.manual_seed(3)
    N, H, d, k = 34000, 2, 32, 16
    offs = torch.tensor([0, 9000, 9100, N], dtype=torch.int32, device="cuda")
    Q, K = torch.randn(N, H, d, device="cuda"), torch.randn(N, H, d, device="cuda")
    if case == "zero_keys":
        K.zero_()
    elif case == "identical_keys":
        K[:] = K[0]
    elif case == "negative_scores":
        base = torch.randn(H, d, device="cuda")
        Q = base + 0.1 * torch.randn(N, H, d, device="cuda")
        K = -base + 0.1 * torch.randn(N, H, d, device="cuda")
    elif case == "one_giant_key":
        K[12345] *= 1.0e4
    elif case == "zero_queries":
        Q[::3] = 0.0
    elif case == "two_scales":
        K[: N // 2] *= 1.0e-3
        Q[N // 2:] *= 1.0e3
    V = torch.randn(N, H, d, device="cuda")
    fb = _dense_check(Q.bfloat16(), K.bfloat16(), V.bfloat16(), offs, k)
    assert torch.isfinite(fb.out.float()).all()
