"""The cumulative-attention-weight diagnostic (App. I): the CUDA path against the oracle's plain
definition (all scores, full softmax, sum of the k largest probabilities)."""
import numpy as np
import pytest
import torch

from paper_2604_03815_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import kmip_oracle as oracle
    from paper_2604_03815_b200 import binding as kb
    from tests import parity_util as pu


@pytest.mark.parametrize("mode,d,k,scale", [(wl.MODE_BF16_TC, 32, 16, 1.0), (wl.MODE_BF16_TC, 16, 5, 0.25),
                                            (wl.MODE_BF16_TC, 64, 40, 0.5), (wl.MODE_BF16_TC, 128, 7, 0.3),
                                            (wl.MODE_FP32_EXACT, 64, 8, 0.5)])
def test_topk_mass_matches_the_oracle(mode, d, k, scale):
    sizes = [700, 3, 0, 129, 64, 1]
    w = wl.iid_workload("s", 5000 + d, sizes, 2, d, k, mode, input_scale=scale)
    Q, K, V, dO, offs = pu.to_device(w)
    fb = kb.forward(Q, K, V, offs, k, mode)
    mass = torch.full((w.N, w.H), -1.0, dtype=torch.float32, device="cuda")
    assert kb.kmip_attn_topk_mass(Q, K, offs, k, mode, fb.topk_score, mass, fb.workspace) == kb.KMIP_OK
    torch.cuda.synchronize()
    assert kb.kmip_last_status(fb.workspace) == kb.KMIP_OK
    got = mass.cpu().numpy().astype(np.float64)
    ref = oracle.topk_mass(w.Q, w.K, w.graph_offsets, k)
    assert got.min() > 0.0 and got.max() <= 1.0
    np.testing.assert_allclose(got, ref, rtol=2e-3, atol=1e-6)
    o = np.cumsum([0] + sizes)
    np.testing.assert_allclose(got[o[1]:o[2]], 1.0, rtol=1e-5)             # graphs with at most k nodes
    np.testing.assert_allclose(got[-1], 1.0, rtol=1e-5)
    assert ref.min() < 0.9                                                   # and the case is not trivial


def test_topk_mass_on_a_graph_of_many_tiles_with_clusters():
    """Clustered queries and keys (peaked softmax, large scores) over a graph that spans dozens of key tiles
    and several work items, with a ragged last tile; the tensor-core pass against the oracle."""
    w = wl.make_config(4, N=5003, H=2, d=32, k=32)
    Q, K, V, dO, offs = pu.to_device(w)
    fb = kb.forward(Q, K, V, offs, w.k, w.mode)
    mass = torch.full((w.N, w.H), -1.0, dtype=torch.float32, device="cuda")
    assert kb.kmip_attn_topk_mass(Q, K, offs, w.k, w.mode, fb.topk_score, mass, fb.workspace) == kb.KMIP_OK
    assert kb.kmip_last_status(fb.workspace) == kb.KMIP_OK
    got = mass.cpu().numpy().astype(np.float64)
    ref = oracle.topk_mass(w.Q, w.K, w.graph_offsets, w.k)
    np.testing.assert_allclose(got, ref, rtol=2e-3, atol=1e-6)


def test_topk_mass_argument_checks():
    w = wl.iid_workload("s", 5100, [64], 1, 128, 4, wl.MODE_FP32_EXACT)
    Q, K, V, dO, offs = pu.to_device(w)
    fb = kb.forward(Q, K, V, offs, 4, w.mode)
    mass = torch.zeros((w.N, 1), dtype=torch.float32, device="cuda")
    assert kb.kmip_attn_topk_mass(Q, K, offs, 4, w.mode, fb.topk_score, mass, fb.workspace) == kb.KMIP_ERR_UNSUPPORTED
    w = wl.iid_workload("s", 5101, [64], 1, 16, 4, wl.MODE_BF16_TC)
    Q, K, V, dO, offs = pu.to_device(w)
    fb = kb.forward(Q, K, V, offs, 4, w.mode)
    assert kb.kmip_attn_topk_mass(Q, K, offs, 4, w.mode, fb.topk_score, None, fb.workspace) == kb.KMIP_ERR_INVALID_ARG
    assert kb.kmip_attn_topk_mass(Q, K, offs, 4, w.mode, fb.topk_score, mass, fb.workspace[:64]) == kb.KMIP_ERR_WORKSPACE
