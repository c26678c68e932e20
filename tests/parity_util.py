"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the CPU oracle on
the same seeded inputs, compare.  Tolerances (stated once, used everywhere):

  fp32 mode   topk_idx bit-exact against the oracle on every row whose selection margin
              (k-th kept score minus best excluded score) exceeds FP32_SCORE_ERR*max(1,|k-th|); rows below it
              are ties at fp32 resolution and are only required to satisfy the bf16-mode rule.  The
              The (row, head) pairs the rule could excuse are counted (`undecided_set_rows`,
              `undecided_order_rows`), and so are those it does excuse, i.e. that differ from the
              oracle (`excused_rows`); every fp32 test bounds the latter (config 1 and the small
              cases: zero).
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
from paper_2604_03815_b200 import workloads as wl

OUT_ATOL, OUT_RTOL = 2e-3, 1e-2
SCORE_ATOL, SCORE_RTOL = 1e-5, 2e-5
FP32_SCORE_ERR = 2e-6   # relative to max(1, |k-th score|): a few fp32 ulps of a d-term sum
SEL_RTOL = 1e-2


def to_device(w):
    dt = kb.storage_dtype(w.mode)
    t = lambda a: torch.from_numpy(a).to(device="cuda", dtype=dt)
    offs = torch.from_numpy(w.graph_offsets).to(device="cuda", dtype=torch.int32)
    return t(w.Q), t(w.K), t(w.V), t(w.dOut), offs


def run_forward(w, dev=None, fp32_path=0):
    Q, K, V, dO, offs = dev or to_device(w)
    fb = kb.forward(Q, K, V, offs, w.k, w.mode, fp32_path=fp32_path)
    torch.cuda.synchronize()
    return fb


def stratified_rows(w, fb, n, seed=2468):
    """At least `n` query rows for the full-size parity checks, chosen by where the KERNEL puts a row and
    by the structure of the data, not only by row number:
      * borders of work items and of their 128-row query tiles in SWEEP order (the sweep runs the rows of
        large graphs in a data-dependent locality order), for the first, last and a few middle items;
      * every row of up to four work items of the schedule's tail (the units past the last full wave of
        CTAs, which the sweep may cut into single query tiles with one CTA each: a different code path);
      * every cluster of the point-cloud workload and hub / non-hub rows of every graph of the hub batch;
      * the row-number strata of workloads.sample_rows (graph borders, block borders) and seeded uniform picks.
    Returns sorted unique int64 row numbers."""
    order, rpi = kb.kmip_test_sweep_order(fb.workspace, w.N, w.G, w.H, w.d, w.k, w.mode)
    order = order.astype(np.int64)
    offs = w.graph_offsets.astype(np.int64)
    items = []                      # (first sweep position, rows), as the plan kernel lists them
    for g in range(w.G):
        lo, hi = int(offs[g]), int(offs[g + 1])
        items += [(lo + t * rpi, min(rpi, hi - lo - t * rpi)) for t in range((hi - lo + rpi - 1) // rpi)]
    picks = [wl.sample_rows(w, 64)]
    n_items = len(items)
    for it in sorted({0, 1, n_items // 3, n_items // 2, (2 * n_items) // 3, n_items - 2, n_items - 1} & set(range(n_items))):
        r0, nr = items[it]
        picks.append(order[[r0 + o for o in (0, 127, 128, 255, 256, nr - 1) if 0 <= o < nr]])
    # the tail of the persistent schedule: units (work item, head) past the last full wave of CTAs
    n_sms = torch.cuda.get_device_properties(0).multi_processor_count
    total, nqt = n_items * w.H, rpi // 128
    left = total % n_sms if total > n_sms else 0
    # (cut into single query tiles with one CTA each when the pieces fit one wave, otherwise a last partial wave)
    tail = sorted({u % n_items for u in range(total - left, total)}) if (nqt > 1 and left) else []
    for it in (tail[:2] + tail[-2:]) if len(tail) > 4 else tail:
        r0, nr = items[it]
        picks.append(order[r0:r0 + nr])
    if "labels" in w.meta:          # every cluster of the mixture
        lab = np.asarray(w.meta["labels"])
        picks += [np.flatnonzero(lab == c)[:24] for c in np.unique(lab)]
    if "hubs" in w.meta:            # hub and non-hub rows of every graph
        hub = np.asarray(w.meta["hubs"])
        for g in range(w.G):
            lo, hi = int(offs[g]), int(offs[g + 1])
            picks += [lo + np.flatnonzero(hub[lo:hi])[:96], lo + np.flatnonzero(~hub[lo:hi])[:96]]
    rows = np.unique(np.concatenate([np.asarray(p, dtype=np.int64).reshape(-1) for p in picks]))
    rng = np.random.default_rng(seed)
    while len(rows) < min(n, w.N):
        rows = np.unique(np.concatenate([rows, rng.integers(0, w.N, size=n - len(rows) + 16)]))
    return rows, {"tail_items": len(tail), "rows_per_item": rpi}


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
    undecided_set = undecided_order = excused = 0
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
        # (row, head) pairs the rule above excuses: callers bound these counts
        undecided_set = int((~set_decided).sum())
        undecided_order = int((~order_decided).sum())
        excused = int((~same & ~order_decided).sum())   # pairs that DO differ from the oracle and are let through
    d = np.abs(out - ref_out)
    assert np.all(d <= OUT_ATOL + OUT_RTOL * np.abs(ref_out)), f"out off by {d.max():.3e}"
    # rows whose set equals the oracle's are also compared with the oracle's own output
    if same.any():
        d2 = np.abs(out - ref["out"])[same]
        assert np.all(d2 <= OUT_ATOL + OUT_RTOL * np.abs(ref["out"][same]))
    return {"rows": len(rws), "identical_rows": float(same.mean()), "max_out_err": float(d.max()),
            "max_score_err": float(err.max()), "min_gap": float(ref["gap"].min()),
            "undecided_set_rows": undecided_set, "undecided_order_rows": undecided_order, "excused_rows": excused}


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
