"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.
The oracle brute-forces a seeded, stratified sample of at least 4096 query rows against all keys of
their graph (selection, scores, outputs) - stratified by the row's place in the sweep (work-item and
query-tile borders in sweep order, whole work items of the schedule's split tail), by cluster and by
hub / non-hub, see parity_util.stratified_rows; the backward oracle, which is linear in N, runs in
full on the GPU's validated index set."""
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
    rows, info = pu.stratified_rows(w, fb, n_sample)
    assert len(rows) >= n_sample
    st = pu.check_forward(w, fb, rows)
    st.update(info)
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
    st = _full(3, 4096)
    assert st["identical_rows"] > 0.99


def test_config4_500k_point_cloud():
    st = _full(4, 4096)
    assert st["identical_rows"] > 0.95
    assert st["tail_items"] >= 4        # the sample holds whole work items of the schedule's tail


def test_config5_hub_batch():
    st = _full(5, 4096)
    assert st["identical_rows"] > 0.95


def test_mixed_batch_with_reordered_and_untouched_graphs():
    """From 32768 nodes on, the sweep runs the rows of graphs with at least 8192 nodes in locality
    order and leaves smaller graphs alone; every row's result must still land at the row's own
    place.  Clustered queries (so that the order really changes), all rows checked for structure,
    a stratified sample against the oracle, the backward pass in full."""
    sizes = [9000, 300, 20000, 10, 8192, 4000, 0, 8191]
    base = wl.make_config(4, N=sum(sizes), H=2, d=32, k=16)
    offs = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(sizes, out=offs[1:])
    w = wl.Workload(name="mixed", mode=base.mode, H=base.H, d=base.d, k=base.k, graph_offsets=offs.astype(np.int32),
                    Q=base.Q, K=base.K, V=base.V, dOut=base.dOut, backward=True, meta={})
    dev = pu.to_device(w)
    fb = pu.run_forward(w, dev)
    rows = wl.sample_rows(w, 400)
    pu.check_forward(w, fb, rows)
    idx = fb.topk_idx.cpu().numpy()
    g = np.searchsorted(offs, np.arange(w.N), side="right") - 1
    keff = np.minimum(w.k, offs[g + 1] - offs[g])[:, None, None]
    valid = np.arange(w.k)[None, None, :] < keff
    assert np.all(((idx >= offs[g][:, None, None]) & (idx < offs[g + 1][:, None, None])) | ~valid)
    assert np.all((idx == -1) | valid)
    pu.check_backward(w, fb, pu.run_backward(w, fb, dev))
