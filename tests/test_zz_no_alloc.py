"""kmip_attn_forward_static_scratch: the forward pass for callers that are not allowed to allocate
device memory (its scratch is an array built into the library).  Collected last on purpose: if it
fails, a run that stops at the first failure has already run everything else.

The GPU test calls the entry point through the C ABI twice in a row and compares every output with
the regular entry point's on the same inputs; the array is shared by all calls and keeps the previous
call's contents, so the second call also checks that stale contents do no harm."""
import numpy as np
import pytest
import torch

from paper_2604_03815_b200 import workloads as wl


def test_too_large_problem_is_refused_on_the_host():
    from paper_2604_03815_b200 import build
    build.build()
    from paper_2604_03815_b200 import binding as kb
    import ctypes
    p = ctypes.c_void_p(4096)     # never dereferenced: the size check comes first
    rc = kb.lib().kmip_attn_forward_static_scratch(p, p, p, None, 0, 500_000, 4, 32, 32, kb.KMIP_BF16_TC,
                                                   p, p, p, None, None)
    assert rc == kb.KMIP_ERR_TOO_LARGE and "scratch" in kb.status_string(rc)
    rc = kb.lib().kmip_attn_forward_static_scratch(p, p, p, None, 0, 1000, 4, 48, 8, kb.KMIP_BF16_TC,
                                                   p, p, p, None, None)
    assert rc == kb.KMIP_ERR_UNSUPPORTED


@pytest.mark.gpu
@pytest.mark.parametrize("mode", [wl.MODE_BF16_TC, wl.MODE_FP32_EXACT])
def test_static_scratch_forward_matches_regular_forward_twice(mode):
    from paper_2604_03815_b200 import binding as kb
    from tests import parity_util as pu
    first = wl.iid_workload("a", 901, [700, 129, 1500], 2, 32, 16, mode, input_scale=1.0 / np.sqrt(32.0))
    second = wl.make_config(4, N=3000) if mode == wl.MODE_BF16_TC else wl.make_config(1)
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for w in (first, second):                       # two calls in a row, different shapes
        Q, K, V, dO, offs = pu.to_device(w)
        ref = kb.forward(Q, K, V, offs, w.k, w.mode)
        got = kb.ForwardBuffers(w.N, w.G, w.H, w.d, w.k, w.mode)
        got.out.fill_(float("nan")); got.topk_idx.fill_(-7); got.topk_score.fill_(float("nan"))
        rc = kb.kmip_attn_forward_static_scratch(Q, K, V, offs, w.k, w.mode, got.out, got.topk_idx,
                                                 got.topk_score, device_status=status)
        assert rc == kb.KMIP_OK, kb.status_string(rc)
        torch.cuda.synchronize()
        assert int(status.item()) == kb.KMIP_OK
        assert torch.equal(got.topk_idx, ref.topk_idx)
        a, b = got.topk_score.cpu().numpy(), ref.topk_score.cpu().numpy()
        assert np.all(np.abs(a - b) <= pu.SCORE_ATOL + pu.SCORE_RTOL * np.abs(b))
        x, y = got.out.float().cpu().numpy(), ref.out.float().cpu().numpy()
        assert np.all(np.abs(x - y) <= pu.OUT_ATOL + pu.OUT_RTOL * np.abs(y))
        pu.check_forward(w, got)                    # and against the oracle, like every other path
    # malformed offsets are reported through device_status, and the next call is clean again
    Q, K, V, dO, offs = pu.to_device(first)
    got = kb.ForwardBuffers(first.N, first.G, first.H, first.d, first.k, first.mode)
    bad = torch.tensor([0, 900, 700, first.N], dtype=torch.int32, device="cuda")
    rc = kb.kmip_attn_forward_static_scratch(Q, K, V, bad, first.k, first.mode, got.out, got.topk_idx,
                                             got.topk_score, device_status=status)
    torch.cuda.synchronize()
    assert rc == kb.KMIP_OK and int(status.item()) == kb.KMIP_ERR_BAD_OFFSETS
    rc = kb.kmip_attn_forward_static_scratch(Q, K, V, offs, first.k, first.mode, got.out, got.topk_idx,
                                             got.topk_score, device_status=status)
    torch.cuda.synchronize()
    assert rc == kb.KMIP_OK and int(status.item()) == kb.KMIP_OK
    pu.check_forward(first, got)


@pytest.mark.gpu
def test_static_scratch_empty_batch_and_no_status_pointer():
    """N = 0 enqueues no kernel but must clear a status word the caller polls (it may hold the previous
    call's error); device_status = NULL is allowed on every path."""
    from paper_2604_03815_b200 import binding as kb
    from tests import parity_util as pu
    w = wl.iid_workload("a", 902, [300, 40], 2, 16, 8, wl.MODE_BF16_TC)
    Q, K, V, dO, offs = pu.to_device(w)
    got = kb.ForwardBuffers(w.N, w.G, w.H, w.d, w.k, w.mode)
    status = torch.full((1,), kb.KMIP_ERR_BAD_OFFSETS, dtype=torch.int32, device="cuda")   # a stale error
    e = torch.empty((0, w.H, w.d), dtype=Q.dtype, device="cuda")
    ei, es = torch.empty((0, w.H, w.k), dtype=torch.int32, device="cuda"), torch.empty((0, w.H, w.k), device="cuda")
    rc = kb.kmip_attn_forward_static_scratch(e, e, e, None, w.k, w.mode, e, ei, es, device_status=status)
    torch.cuda.synchronize()
    assert rc == kb.KMIP_OK and int(status.item()) == kb.KMIP_OK
    rc = kb.kmip_attn_forward_static_scratch(e, e, e, None, w.k, w.mode, e, ei, es, device_status=None)
    assert rc == kb.KMIP_OK
    rc = kb.kmip_attn_forward_static_scratch(Q, K, V, offs, w.k, w.mode, got.out, got.topk_idx, got.topk_score,
                                             device_status=None)
    torch.cuda.synchronize()
    assert rc == kb.KMIP_OK
    pu.check_forward(w, got)
