"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.
The oracle brute-forces a seeded, stratified sample of query rows against all keys of their
graph (selection, scores, outputs); the backward oracle, which is linear in N, runs in full on
the GPU's validated index set."""
import numpy as np
import pytest
import torch

from paper_2604_03815_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from tests import parity_util as pu


def _full(cfg, n_sample):
    w = wl.make_config(cfg)
    dev = pu.to_device(w)
    fb = pu.run_forward(w, dev)
    rows = wl.sample_rows(w, n_sample)
    st = pu.check_forward(w, fb, rows)
    # every row: structure checks that hold at any size
    idx = fb.topk_idx.cpu().numpy()
    offs = w.graph_offsets.astype(np.int64)
    g = np.searchsorted(offs, np.arange(w.N), side="right") - 1
    assert np.all((idx >= offs[g][:, None, None]) & (idx < offs[g + 1][:, None, None]))
    sc = fb.topk_score.cpu().numpy()
    assert np.all(np.diff(sc, axis=-1) <= 0) and np.isfinite(sc).all()
    bb = pu.run_backward(w, fb, dev)
    st.update(pu.check_backward(w, fb, bb))
    return st


def test_config3_100k_nodes():
    st = _full(3, 384)
    assert st["identical_rows"] > 0.99


def test_config4_500k_point_cloud():
    st = _full(4, 256)
    assert st["identical_rows"] > 0.95


def test_config5_hub_batch():
    st = _full(5, 256)
    assert st["identical_rows"] > 0.95
