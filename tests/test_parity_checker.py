"""The parity checker itself (CPU only): it accepts a result built from the oracle and rejects
corrupted ones, so a green GPU run means what it says."""
import types

import numpy as np
import pytest
import torch

from oracle import kmip_oracle as oracle
from paper_2604_03815_b200 import workloads as wl
from tests import parity_util as pu


def _fake_buffers(w, rows=None):
    r = oracle.forward(w.Q, w.K, w.V, w.graph_offsets, w.k)
    fb = types.SimpleNamespace(topk_idx=torch.from_numpy(r["idx"].copy()),
                               topk_score=torch.from_numpy(r["score"].astype(np.float32)),
                               out=torch.from_numpy(r["out"].astype(np.float32)))
    return fb


@pytest.mark.parametrize("mode", [wl.MODE_BF16_TC, wl.MODE_FP32_EXACT])
def test_checker_accepts_oracle_and_rejects_corruption(mode):
    w = wl.iid_workload("s", 5, [40, 3, 0, 70], 2, 16, 6, mode)
    fb = _fake_buffers(w)
    st = pu.check_forward(w, fb)
    assert st["identical_rows"] == 1.0
    st = pu.check_forward(w, fb, rows=np.array([0, 41, 43, 112]))
    assert st["rows"] == 4

    bad = _fake_buffers(w)
    bad.out[7, 1, 3] += 0.05
    with pytest.raises(AssertionError):
        pu.check_forward(w, bad)

    bad = _fake_buffers(w)                      # replace the best key of a row by a poor one
    S = w.Q[50, 0].astype(np.float64) @ w.K[43:, 0].astype(np.float64).T
    bad.topk_idx[50, 0, 0] = 43 + int(np.argmin(S))
    with pytest.raises(AssertionError):
        pu.check_forward(w, bad)

    bad = _fake_buffers(w)                      # key of another graph
    bad.topk_idx[50, 0, 1] = 3
    with pytest.raises(AssertionError):
        pu.check_forward(w, bad)

    bad = _fake_buffers(w)                      # duplicate key
    bad.topk_idx[50, 0, 1] = bad.topk_idx[50, 0, 0]
    with pytest.raises(AssertionError):
        pu.check_forward(w, bad)

    bad = _fake_buffers(w)                      # padding missing in the 3-node graph
    bad.topk_idx[41, 0, 5] = 41
    with pytest.raises(AssertionError):
        pu.check_forward(w, bad)


def test_backward_checker():
    w = wl.iid_workload("s", 6, [60], 2, 16, 5, wl.MODE_BF16_TC)
    fb = _fake_buffers(w)
    dQ, dK, dV = oracle.backward(w.Q, w.K, w.V, w.dOut, fb.topk_idx.numpy())
    bb = types.SimpleNamespace(dQ=torch.from_numpy(dQ), dK=torch.from_numpy(dK), dV=torch.from_numpy(dV))
    pu.check_backward(w, fb, bb)
    bb.dK[3, 1, 2] += 0.1
    with pytest.raises(AssertionError):
        pu.check_backward(w, fb, bb)
