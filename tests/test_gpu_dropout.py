"""Attention dropout on the k softmax weights: the CUDA path against the oracle on the same
(drop_p, seed), forward through the GPU's own selection and backward with it held fixed."""
import numpy as np
import pytest
import torch

from paper_2604_03815_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import kmip_oracle as oracle
    from paper_2604_03815_b200 import binding as kb
    from tests import parity_util as pu


@pytest.mark.parametrize("mode,d,k,drop", [(wl.MODE_BF16_TC, 32, 16, 0.5), (wl.MODE_BF16_TC, 16, 40, 0.25),
                                           (wl.MODE_FP32_EXACT, 32, 8, 0.5)])
def test_dropout_matches_the_oracle(mode, d, k, drop):
    sizes = [300, 1, 129, 0, 50]
    w = wl.iid_workload("s", 4000 + k, sizes, 2, d, k, mode, input_scale=1.0 / np.sqrt(d))
    Q, K, V, dO, offs = pu.to_device(w)
    G = len(sizes)
    fb = kb.ForwardBuffers(w.N, G, w.H, d, k, mode)
    bb = kb.BackwardBuffers(w.N, G, w.H, d, k, mode)
    seed = 0x1234567890ABCDEF
    assert kb.kmip_attn_forward_dropout(Q, K, V, offs, k, mode, drop, seed, fb.out, fb.topk_idx, fb.topk_score,
                                        fb.workspace) == kb.KMIP_OK
    assert kb.kmip_attn_backward_dropout(Q, K, V, offs, k, mode, drop, seed, fb.out, dO, fb.topk_idx, fb.topk_score,
                                         bb.dQ, bb.dK, bb.dV, bb.workspace) == kb.KMIP_OK
    torch.cuda.synchronize()
    assert kb.kmip_last_status(fb.workspace) == kb.KMIP_OK and kb.kmip_last_status(bb.workspace) == kb.KMIP_OK
    idx = fb.topk_idx.cpu().numpy()

    # the selection itself is untouched by dropout: same indices as the plain call
    plain = kb.forward(Q, K, V, offs, k, mode)
    assert torch.equal(plain.topk_idx, fb.topk_idx) and torch.equal(plain.topk_score, fb.topk_score)

    ref_out, _ = oracle.forward_given_idx(w.Q, w.K, w.V, idx, drop=drop, seed=seed)
    out = fb.out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(out - ref_out) <= pu.OUT_ATOL + pu.OUT_RTOL * np.abs(ref_out))
    none_out, _ = oracle.forward_given_idx(w.Q, w.K, w.V, idx)
    assert np.abs(ref_out - none_out).max() > 0.05        # the draws did change the result

    rQ, rK, rV = oracle.backward(w.Q, w.K, w.V, w.dOut, idx, drop=drop, seed=seed)
    for got, ref, name in ((bb.dQ, rQ, "dQ"), (bb.dK, rK, "dK"), (bb.dV, rV, "dV")):
        g = got.float().cpu().numpy().astype(np.float64)
        err = np.abs(g - ref)
        assert np.all(err <= pu.OUT_ATOL + pu.OUT_RTOL * np.abs(ref)), f"{name} off by {err.max():.3e}"


def test_dropout_argument_checks():
    w = wl.iid_workload("s", 4100, [64], 1, 16, 4, wl.MODE_BF16_TC)
    Q, K, V, dO, offs = pu.to_device(w)
    fb = kb.ForwardBuffers(w.N, 1, 1, 16, 4, w.mode)
    for bad in (-0.1, 1.0, float("nan")):
        assert kb.kmip_attn_forward_dropout(Q, K, V, offs, 4, w.mode, bad, 1, fb.out, fb.topk_idx, fb.topk_score,
                                            fb.workspace) == kb.KMIP_ERR_INVALID_ARG
