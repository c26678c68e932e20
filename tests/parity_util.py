"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the CPU oracle on
the same seeded inputs, compare.  Tolerances (stated once, used everywhere):

  fp32 mode   topk_idx bit-exact against the oracle on every row whose selection margin
              (k-th kept score minus best excluded score) exceeds FP32_SCORE_ERR*max(1,|k-th|); rows below it
              are ties at fp32 resolution and are only required to satisfy the bf16-mode rule.
  bf16 mode   every selected key's exact (oracle, fp64) score >= oracle k-th score - 1e-2*|k-th|;
              indices distinct and inside the query's own graph; padding exactly where n_g < k.
  scores      |gpu - exact| <= SCORE_ATOL + SCORE_RTOL*|exact| (fp32 accumulation of exact products).
  outputs and gradients   |gpu - ref| <= 2e-3 + 1e-2*|ref|, ref = oracle evaluated on the GPU's
              validated index set (several index sets are acceptable in bf16 mode; given the set the
              result is unique).
"""
import numpy as np
import torch

from oracle import kmip_oracle as oracle
from paper_2604_03815_b200 import binding as kb

OUT_ATOL, OUT_RTOL = 2e-3, 1e-2
SCORE_ATOL, SCORE_RTOL = 1e-5, 2e-5
FP32_SCORE_ERR = 2e-6   # relative to max(1, |k-th score|): a few fp32 ulps of a d-term sum
SEL_RTOL = 1e-2


def to_device(w):
    dt = kb.storage_dtype(w.mode)
    t = lambda a: torch.from_numpy(a).to(device="cuda", dtype=dt)
    offs = torch.from_numpy(w.graph_offsets).to(device="cuda", dtype=torch.int32)
    return t(w.Q), t(w.K), t(w.V), t(w.dOut), offs


def run_forward(w, dev=None):
    Q, K, V, dO, offs = dev or to_device(w)
    fb = kb.forward(Q, K, V, offs, w.k, w.mode)
    torch.cuda.synchronize()
    return fb


def check_forward(w, fb, rows=None):
    """Compare forward results with the oracle on `rows` (all rows when None). Returns stats."""
    idx = fb.topk_idx.cpu().numpy()
    score = fb.topk_score.cpu().numpy().astype(np.float64)
    out = fb.out.float().cpu().numpy().astype(np.float64)
    if rows is not None:
        idx, score, out = idx[rows], score[rows], out[rows]
    ref = oracle.forward(w.Q, w.K, w.V, w.graph_offsets, w.k, rows=rows)
    rws = np.arange(w.N) if rows is None else np.asarray(rows)

    # structure: padding where the graph is smaller than k, distinct in-graph indices elsewhere
    offs = w.graph_offsets.astype(np.int64)
    g = np.searchsorted(offs, rws, side="right") - 1
    lo, hi = offs[g], offs[g + 1]
    keff = np.minimum(w.k, hi - lo)
    slot = np.arange(w.k)[None, None, :]
    valid = np.broadcast_to(slot < keff[:, None, None], idx.shape)
    assert np.all(idx[~valid] == -1), "padded slots must hold -1"
    assert np.all(np.isneginf(score[~valid])), "padded slots must hold -inf"
    assert np.all((idx >= lo[:, None, None]) & (idx < hi[:, None, None]) | ~valid), "index outside the query's graph"
    srt = np.sort(np.where(valid, idx, -1 - slot), axis=-1)
    assert np.all(np.diff(srt, axis=-1) != 0), "duplicate key in a row"
    sc = np.where(valid, score, 0.0)
    assert np.all(np.diff(np.where(valid, score, -1e300), axis=-1) <= 0), "scores must be listed in descending order"

    # exact scores of the keys the GPU selected, and the output the oracle derives from that set
    ref_out, exact = oracle.forward_given_idx(w.Q, w.K, w.V, idx, rows=rows)
    err = np.abs(sc - np.where(valid, exact, 0.0))
    assert np.all(err <= SCORE_ATOL + SCORE_RTOL * np.abs(np.where(valid, exact, 0.0))), \
        f"topk_score off by {err.max():.3e}"

    kth = np.take_along_axis(ref["score"], np.maximum(keff - 1, 0)[:, None, None].repeat(w.H, 1), axis=2)[..., 0]
    worst = np.where(valid, exact, np.inf).min(axis=-1)
    assert np.all(worst >= kth - SEL_RTOL * np.abs(kth)), "a selected key is worse than the k-th best by more than 1e-2"

    same = np.all(idx == ref["idx"], axis=-1)
    if w.mode == kb.KMIP_FP32_EXACT:
        # fp32 arithmetic cannot order two scores that differ by less than its own rounding error.  The
        # selected SET is decided when the k-th and (k+1)-th exact scores are further apart than that; the
        # ORDER of the list is decided when, in addition, every two neighbours of the oracle's list are.
        thr = FP32_SCORE_ERR * np.maximum(1.0, np.abs(kth))
        set_decided = ref["gap"] > thr
        same_set = np.all(np.sort(idx, axis=-1) == np.sort(ref["idx"], axis=-1), axis=-1)
        assert np.all(same_set | ~set_decided), \
            f"fp32 mode: selected set differs on {int((~same_set & set_decided).sum())} decided rows"
        rs = np.where(valid, ref["score"], -1e300)
        inner = np.where(valid[..., 1:], rs[..., :-1] - rs[..., 1:], np.inf).min(axis=-1) if w.k > 1 else np.full(same.shape, np.inf)
        order_decided = set_decided & (inner > thr)
        assert np.all(same | ~order_decided), \
            f"fp32 mode: topk_idx differs on {int((~same & order_decided).sum())} decided rows"
    d = np.abs(out - ref_out)
    assert np.all(d <= OUT_ATOL + OUT_RTOL * np.abs(ref_out)), f"out off by {d.max():.3e}"
    # rows whose set equals the oracle's are also compared with the oracle's own output
    if same.any():
        d2 = np.abs(out - ref["out"])[same]
        assert np.all(d2 <= OUT_ATOL + OUT_RTOL * np.abs(ref["out"][same]))
    return {"rows": len(rws), "identical_rows": float(same.mean()), "max_out_err": float(d.max()),
            "max_score_err": float(err.max()), "min_gap": float(ref["gap"].min())}


def run_backward(w, fb, dev=None):
    Q, K, V, dO, offs = dev or to_device(w)
    bb = kb.backward(Q, K, V, offs, w.k, w.mode, fb, dO)
    torch.cuda.synchronize()
    return bb


def check_backward(w, fb, bb):
    """Gradients against the oracle's backward evaluated on the GPU's own (validated) index set."""
    idx = fb.topk_idx.cpu().numpy()
    rq, rk, rv = oracle.backward(w.Q, w.K, w.V, w.dOut, idx)
    stats = {}
    for name, got, ref in (("dQ", bb.dQ, rq), ("dK", bb.dK, rk), ("dV", bb.dV, rv)):
        got = got.float().cpu().numpy().astype(np.float64)
        d = np.abs(got - ref)
        bad = d > OUT_ATOL + OUT_RTOL * np.abs(ref)
        assert not bad.any(), f"{name}: {int(bad.sum())} elements off, max err {d.max():.3e} at {np.unravel_index(d.argmax(), d.shape)}"
        stats["max_" + name + "_err"] = float(d.max())
    return stats
