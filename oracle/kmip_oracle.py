"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, NOT THE PRODUCT).

Only the tests, the smoke check and the benchmark's cpu_baseline / reference leg may
import this module.  It compiles `kmip_oracle.c` with gcc on first use (or when the
source is newer than the shared object) and marshals numpy arrays; all arithmetic is
in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kmip_oracle.c")
_LIB = os.path.join(_HERE, "libkmip_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 -fopenmp; returns the path of the shared object."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        lib.kmip_oracle_threads.restype = ctypes.c_int
        lib.kmip_oracle_forward_rows.restype = ctypes.c_int
        lib.kmip_oracle_forward_rows.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, P, i64, P, P, P, P]
        lib.kmip_oracle_forward_given_idx.restype = ctypes.c_int
        lib.kmip_oracle_forward_given_idx.argtypes = [P, P, P, i64, i32, i32, i32, P, i64, P, P, P]
        lib.kmip_oracle_backward.restype = ctypes.c_int
        lib.kmip_oracle_backward.argtypes = [P, P, P, P, P, i64, i32, i32, i32, P, P, P]
        f64, u64 = ctypes.c_double, ctypes.c_uint64
        lib.kmip_oracle_topk_mass.restype = ctypes.c_int
        lib.kmip_oracle_topk_mass.argtypes = [P, P, P, i32, i64, i32, i32, i32, P, i64, P]
        lib.kmip_oracle_forward_given_idx_dropout.restype = ctypes.c_int
        lib.kmip_oracle_forward_given_idx_dropout.argtypes = [P, P, P, i64, i32, i32, i32, P, i64, P, f64, u64, P, P]
        lib.kmip_oracle_backward_dropout.restype = ctypes.c_int
        lib.kmip_oracle_backward_dropout.argtypes = [P, P, P, P, P, i64, i32, i32, i32, f64, u64, P, P, P]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().kmip_oracle_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.ndim == 3
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def forward(Q, K, V, graph_offsets, k, rows=None):
    """Oracle forward.  Returns dict(out, idx, score, gap); arrays are indexed by position
    in `rows` (all rows when rows is None)."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    N, H, d = Q.shape
    offs = None if graph_offsets is None else np.ascontiguousarray(graph_offsets, dtype=np.int32)
    G = 1 if offs is None else len(offs) - 1
    rws = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = N if rws is None else len(rws)
    out = np.zeros((n, H, d), dtype=np.float64)
    idx = np.full((n, H, k), -1, dtype=np.int32)
    score = np.full((n, H, k), -np.inf, dtype=np.float64)
    gap = np.full((n, H), np.inf, dtype=np.float64)
    rc = _load().kmip_oracle_forward_rows(_ptr(Q), _ptr(K), _ptr(V), _ptr(offs), G, N, H, d, k,
                                          _ptr(rws), n, _ptr(out), _ptr(idx), _ptr(score), _ptr(gap))
    if rc != 0:
        raise ValueError(f"kmip_oracle_forward_rows failed with status {rc}")
    return {"out": out, "idx": idx, "score": score, "gap": gap}


def forward_given_idx(Q, K, V, idx, rows=None, drop=0.0, seed=0):
    """Softmax-weighted sum over a caller-supplied index set (with attention dropout on the
    weights when drop > 0); returns (out, score)."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    N, H, d = Q.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    rws = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = N if rws is None else len(rws)
    assert idx.shape[0] == n and idx.shape[1] == H
    k = idx.shape[2]
    out = np.zeros((n, H, d), dtype=np.float64)
    score = np.zeros((n, H, k), dtype=np.float64)
    rc = _load().kmip_oracle_forward_given_idx_dropout(_ptr(Q), _ptr(K), _ptr(V), N, H, d, k, _ptr(rws), n, _ptr(idx),
                                                       ctypes.c_double(drop), ctypes.c_uint64(seed), _ptr(out), _ptr(score))
    if rc != 0:
        raise ValueError(f"kmip_oracle_forward_given_idx failed with status {rc}")
    return out, score


def backward(Q, K, V, dOut, idx, drop=0.0, seed=0):
    """Sparse backward with the selection (and the dropout draws) held constant; returns (dQ, dK, dV) in fp64."""
    Q, K, V, dOut = _f32(Q), _f32(K), _f32(V), _f32(dOut)
    N, H, d = Q.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.shape[:2] == (N, H)
    k = idx.shape[2]
    dQ = np.empty((N, H, d), dtype=np.float64)
    dK = np.empty((N, H, d), dtype=np.float64)
    dV = np.empty((N, H, d), dtype=np.float64)
    rc = _load().kmip_oracle_backward_dropout(_ptr(Q), _ptr(K), _ptr(V), _ptr(dOut), _ptr(idx), N, H, d, k,
                                              ctypes.c_double(drop), ctypes.c_uint64(seed), _ptr(dQ), _ptr(dK), _ptr(dV))
    if rc != 0:
        raise ValueError(f"kmip_oracle_backward failed with status {rc}")
    return dQ, dK, dV


def topk_mass(Q, K, graph_offsets, k, rows=None):
    """Share of the full softmax (over all keys of the query's graph) that falls on the k largest
    scores; [n_rows, H] fp64."""
    Q, K = _f32(Q), _f32(K)
    N, H, d = Q.shape
    offs = None if graph_offsets is None else np.ascontiguousarray(graph_offsets, dtype=np.int32)
    G = 1 if offs is None else len(offs) - 1
    rws = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = N if rws is None else len(rws)
    mass = np.zeros((n, H), dtype=np.float64)
    rc = _load().kmip_oracle_topk_mass(_ptr(Q), _ptr(K), _ptr(offs), G, N, H, d, k, _ptr(rws), n, _ptr(mass))
    if rc != 0:
        raise ValueError(f"kmip_oracle_topk_mass failed with status {rc}")
    return mass


# ------------------------------------------------------------------------------------------------
# The full layer of Eq. 2 / Algorithm 1 ("Require" line and lines 2-8): projections in front of the
# attention core and the output projection behind it.  Plain numpy matrix products in fp64 around the
# C functions above; the selection is the oracle's own top-k or an index set supplied by the caller.
# ------------------------------------------------------------------------------------------------
def _round_bf16(a):
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even), returned as float64."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(np.isfinite(f), out, f.astype(np.float64))


def _store(a, storage):
    """What the attention core receives: its inputs are stored as bf16 or fp32 arrays."""
    if storage == "bf16":
        return _round_bf16(a)
    return np.ascontiguousarray(a, dtype=np.float32).astype(np.float64)


def layer_forward(x, w_q, w_k, w_v, w_o, graph_offsets, H, k, idx=None, storage="f32"):
    """Y = sum_h O^h W_O^h with O^h = kMIP-Attn(X W_Q^h, X W_K^h, X W_V^h) per graph (Eq. 2).

    x [N, d_model]; w_q, w_k, w_v [H*d, d_model] (row h*d + c is column c of W^h); w_o [d_model, H*d].
    Q, K, V and O pass through `storage` ("bf16" or "f32": the arrays the core reads and writes).
    idx: index set [N, H, k] to use instead of the oracle's own top-k (Algorithm 1 line 3).
    Returns dict(y, q, k, v, o, idx) with fp64 arrays."""
    x = np.asarray(x, dtype=np.float64)
    N = x.shape[0]
    d = w_q.shape[0] // H
    q = _store(x @ np.asarray(w_q, np.float64).T, storage).reshape(N, H, d)
    kk = _store(x @ np.asarray(w_k, np.float64).T, storage).reshape(N, H, d)
    v = _store(x @ np.asarray(w_v, np.float64).T, storage).reshape(N, H, d)
    if idx is None:
        f = forward(q, kk, v, graph_offsets, k)
        o, idx = f["out"], f["idx"]
    else:
        o, _ = forward_given_idx(q, kk, v, idx)
    o = _store(o, storage)
    y = o.reshape(N, H * d) @ np.asarray(w_o, np.float64).T
    return {"y": y, "q": q, "k": kk, "v": v, "o": o, "idx": np.asarray(idx, dtype=np.int32)}


def layer_backward(x, w_q, w_k, w_v, w_o, H, fwd, d_y):
    """Gradients of sum(y * d_y) through layer_forward with the selection fwd["idx"] held constant (Sec. 3.1)
    and the storage roundings treated as the identity; returns dict(dx, dw_q, dw_k, dw_v, dw_o) in fp64."""
    x = np.asarray(x, dtype=np.float64)
    d_y = np.asarray(d_y, dtype=np.float64)
    N = x.shape[0]
    d = w_q.shape[0] // H
    o_cat = fwd["o"].reshape(N, H * d)
    dw_o = d_y.T @ o_cat
    d_o = (d_y @ np.asarray(w_o, np.float64)).reshape(N, H, d)
    dq, dk, dv = backward(fwd["q"], fwd["k"], fwd["v"], d_o, fwd["idx"])
    dq, dk, dv = (g.reshape(N, H * d) for g in (dq, dk, dv))
    dx = dq @ np.asarray(w_q, np.float64) + dk @ np.asarray(w_k, np.float64) + dv @ np.asarray(w_v, np.float64)
    return {"dx": dx, "dw_q": dq.T @ x, "dw_k": dk.T @ x, "dw_v": dv.T @ x, "dw_o": dw_o}
