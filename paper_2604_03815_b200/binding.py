"""Thin Python binding of the C-ABI library `libkmip.so` (argument marshalling only).

Function names follow `include/kmip.h`.  Tensors are torch CUDA tensors used purely as
device buffers; every step of the computation runs inside the library's CUDA kernels.
There is no CPU or PyTorch fallback: if the shared library is missing the import fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

KMIP_OK = 0
KMIP_ERR_INVALID_ARG = 1
KMIP_ERR_UNSUPPORTED = 2
KMIP_ERR_WORKSPACE = 3
KMIP_ERR_CUDA = 4
KMIP_ERR_TIMEOUT = 5
KMIP_ERR_BAD_OFFSETS = 6
KMIP_ERR_TOO_LARGE = 7
KMIP_BF16_TC = 0
KMIP_FP32_EXACT = 1
KMIP_BF16_TC_PRUNED = 2
PASS_FORWARD = 0
PASS_BACKWARD = 1

# KMIP_LIBRARY selects another build of the same library, e.g. libkmip_checks.so (canary blocks and device-side
# index tests, see kmip_build_flags in include/kmip.h)
LIB_PATH = os.environ.get("KMIP_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libkmip.so")
KMIP_ERR_CHECK = 8
_lib = None


class TestOptions(ctypes.Structure):
    """kmip_test_options_t of include/kmip_test.h."""
    _fields_ = [("wait_limit_cycles", ctypes.c_int64), ("drop_first_tile", ctypes.c_int32),
                ("fp32_path", ctypes.c_int32)]


class LayerTensors(ctypes.Structure):
    """kmip_layer_tensors_t of include/kmip.h (device pointers)."""
    _fields_ = [(n, ctypes.c_void_p) for n in ("x", "w_q", "w_k", "w_v", "w_o", "q", "k", "v", "o", "topk_idx", "topk_score",
                                                "y", "d_y", "d_x", "dw_q", "dw_k", "dw_v", "dw_o")]


class KmipError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2604_03815_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        P, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.kmip_version.restype = ctypes.c_int
        L.kmip_build_flags.restype = ctypes.c_int
        L.kmip_status_string.restype = ctypes.c_char_p
        L.kmip_status_string.argtypes = [ctypes.c_int]
        L.kmip_attn_workspace_bytes.restype = ctypes.c_int
        L.kmip_attn_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, ctypes.c_int, ctypes.c_int,
                                                ctypes.POINTER(sz)]
        L.kmip_attn_forward.restype = ctypes.c_int
        L.kmip_attn_forward.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, P, P, P, P, sz, P]
        L.kmip_attn_backward.restype = ctypes.c_int
        L.kmip_attn_backward.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, P, P, P, P,
                                         P, P, P, P, sz, P]
        f32, u64 = ctypes.c_float, ctypes.c_uint64
        L.kmip_attn_forward_dropout.restype = ctypes.c_int
        L.kmip_attn_forward_dropout.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, f32, u64, P, P, P, P, sz, P]
        L.kmip_attn_backward_dropout.restype = ctypes.c_int
        L.kmip_attn_backward_dropout.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, f32, u64, P, P, P, P,
                                                 P, P, P, P, sz, P]
        L.kmip_attn_topk_mass.restype = ctypes.c_int
        L.kmip_attn_topk_mass.argtypes = [P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, P, P, P, sz, P]
        L.kmip_last_status.restype = ctypes.c_int
        L.kmip_last_status.argtypes = [P, P, ctypes.POINTER(ctypes.c_int)]
        L.kmip_attn_forward_static_scratch.restype = ctypes.c_int
        L.kmip_attn_forward_static_scratch.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, P, P, P, P, P]
        L.kmip_profile_enable.restype = ctypes.c_int
        L.kmip_profile_enable.argtypes = [ctypes.c_int]
        L.kmip_profile_read.restype = ctypes.c_int
        L.kmip_profile_read.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int)]
        L.kmip_layer_workspace_bytes.restype = ctypes.c_int
        L.kmip_layer_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32, ctypes.c_int, ctypes.POINTER(sz)]
        for fn in (L.kmip_layer_forward, L.kmip_layer_backward):
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.POINTER(LayerTensors), P, i32, i64, i32, i32, i32, i32, P, sz, P]
        L.kmip_attn_sweep_counters.restype = ctypes.c_int
        L.kmip_attn_sweep_counters.argtypes = [P, P, ctypes.POINTER(ctypes.c_int64)]
        # kmip_test.h
        L.kmip_test_tc_scores.restype = ctypes.c_int
        L.kmip_test_tc_scores.argtypes = [P, P, i64, i32, i32, P, P, sz, P]
        L.kmip_test_f16_scores.restype = ctypes.c_int
        L.kmip_test_f16_scores.argtypes = [P, P, i64, i32, i32, P, P, P, sz, P]
        L.kmip_test_gemm_tn.restype = ctypes.c_int
        L.kmip_test_gemm_tn.argtypes = [P, P, P, i32, i32, i32, ctypes.c_int, P, sz, P]
        L.kmip_test_sweep_order.restype = ctypes.c_int
        L.kmip_test_sweep_order.argtypes = [P, i64, i32, i32, i32, i32, ctypes.c_int, P, ctypes.POINTER(i32), P]
        L.kmip_test_attn_forward.restype = ctypes.c_int
        L.kmip_test_attn_forward.argtypes = [P, P, P, P, i32, i64, i32, i32, i32, ctypes.c_int, P, P, P, P, sz, P,
                                             ctypes.POINTER(TestOptions)]
        _lib = L
    return _lib


def kmip_version() -> int:
    return int(lib().kmip_version())


def kmip_build_flags() -> int:
    """Bit 0: the loaded library is a -DKMIP_CHECKS build."""
    return int(lib().kmip_build_flags())


def status_string(status: int) -> str:
    return lib().kmip_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def kmip_attn_workspace_bytes(N, G, H, d, k, mode, pass_) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().kmip_attn_workspace_bytes(N, G, H, d, k, mode, pass_, ctypes.byref(out))
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_attn_workspace_bytes")
    return int(out.value)


def kmip_attn_forward(Q, K, V, graph_offsets, k, mode, out, topk_idx, topk_score, workspace, stream=None) -> int:
    """Enqueue the forward pass; returns the library's status code (no exception, no sync)."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_forward(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k, mode,
                                       _ptr(out), _ptr(topk_idx), _ptr(topk_score), _ptr(workspace),
                                       0 if workspace is None else workspace.numel() * workspace.element_size(),
                                       _stream(stream)))


def kmip_attn_forward_dropout(Q, K, V, graph_offsets, k, mode, drop_p, seed, out, topk_idx, topk_score, workspace,
                              stream=None) -> int:
    """Forward pass with attention dropout on the k softmax weights (counter-based draws from `seed`)."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_forward_dropout(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k, mode,
                                               float(drop_p), int(seed), _ptr(out), _ptr(topk_idx), _ptr(topk_score),
                                               _ptr(workspace),
                                               0 if workspace is None else workspace.numel() * workspace.element_size(),
                                               _stream(stream)))


def kmip_attn_backward_dropout(Q, K, V, graph_offsets, k, mode, drop_p, seed, out, d_out, topk_idx, topk_score,
                               dQ, dK, dV, workspace, stream=None) -> int:
    """Backward pass of kmip_attn_forward_dropout with the same (drop_p, seed)."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_backward_dropout(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k, mode,
                                                float(drop_p), int(seed), _ptr(out), _ptr(d_out), _ptr(topk_idx),
                                                _ptr(topk_score), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(workspace),
                                                0 if workspace is None else workspace.numel() * workspace.element_size(),
                                                _stream(stream)))


def kmip_attn_topk_mass(Q, K, graph_offsets, k, mode, topk_score, mass, workspace, stream=None) -> int:
    """Share of the full softmax held by the kept scores, [N, H] float32 (diagnostic; one more pass over all scores)."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_topk_mass(_ptr(Q), _ptr(K), _ptr(graph_offsets), G, N, H, d, k, mode, _ptr(topk_score),
                                         _ptr(mass), _ptr(workspace),
                                         0 if workspace is None else workspace.numel() * workspace.element_size(),
                                         _stream(stream)))


def kmip_attn_forward_static_scratch(Q, K, V, graph_offsets, k, mode, out, topk_idx, topk_score,
                                     device_status=None, stream=None) -> int:
    """Forward pass that uses the library's built-in scratch array instead of a caller workspace
    (for callers that may not allocate device memory); returns the library's status code.
    `device_status`, if given, is an int32 CUDA tensor that receives the device status word."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_forward_static_scratch(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k,
                                                      mode, _ptr(out), _ptr(topk_idx), _ptr(topk_score),
                                                      _ptr(device_status), _stream(stream)))


def kmip_layer_workspace_bytes(N, G, d_model, H, d_head, k, pass_) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().kmip_layer_workspace_bytes(N, G, d_model, H, d_head, k, pass_, ctypes.byref(out))
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_layer_workspace_bytes")
    return int(out.value)


def _layer_call(fn, tensors: dict, graph_offsets, N, d_model, H, d_head, k, workspace, stream):
    t = LayerTensors(**{n: (None if v is None else v.data_ptr()) for n, v in tensors.items()})
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(fn(ctypes.byref(t), _ptr(graph_offsets), G, N, d_model, H, d_head, k, _ptr(workspace),
                  0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream)))


def kmip_layer_forward(tensors: dict, graph_offsets, N, d_model, H, d_head, k, workspace, stream=None) -> int:
    """Eq. 2 forward: `tensors` maps the field names of kmip_layer_tensors_t to torch CUDA tensors (or None)."""
    return _layer_call(lib().kmip_layer_forward, tensors, graph_offsets, N, d_model, H, d_head, k, workspace, stream)


def kmip_layer_backward(tensors: dict, graph_offsets, N, d_model, H, d_head, k, workspace, stream=None) -> int:
    """Eq. 2 backward with the saved selection; `tensors` as for kmip_layer_forward."""
    return _layer_call(lib().kmip_layer_backward, tensors, graph_offsets, N, d_model, H, d_head, k, workspace, stream)


def kmip_attn_backward(Q, K, V, graph_offsets, k, mode, out, d_out, topk_idx, topk_score, dQ, dK, dV,
                       workspace, stream=None) -> int:
    """Enqueue the backward pass; returns the library's status code (no exception, no sync)."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    return int(lib().kmip_attn_backward(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k, mode,
                                        _ptr(out), _ptr(d_out), _ptr(topk_idx), _ptr(topk_score),
                                        _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(workspace),
                                        0 if workspace is None else workspace.numel() * workspace.element_size(),
                                        _stream(stream)))


def kmip_last_status(workspace, stream=None) -> int:
    """Synchronise the stream and return the device-side status recorded in the workspace."""
    st = ctypes.c_int(0)
    rc = lib().kmip_last_status(_ptr(workspace), _stream(stream), ctypes.byref(st))
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_last_status")
    return int(st.value)


STAGES = ("plan", "score_select", "refine", "softmax_gather", "bwd_rows", "bwd_inverse_index", "bwd_segments")
N_FWD_STAGES = 4


def kmip_profile_enable(max_calls: int) -> None:
    rc = lib().kmip_profile_enable(int(max_calls))
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_profile_enable")


def kmip_profile_read():
    """Returns ({stage: total milliseconds}, forward calls, backward calls) since the last read."""
    ms = (ctypes.c_double * 7)()
    calls = (ctypes.c_int * 2)()
    rc = lib().kmip_profile_read(ms, calls)
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_profile_read")
    return dict(zip(STAGES, list(ms))), int(calls[0]), int(calls[1])


def kmip_test_tc_scores(Q, K, scores, workspace, stream=None) -> int:
    """kmip_test.h: dense q.k scores [H, N, N] of one small graph through the tensor-core pipeline."""
    N, H, d = Q.shape
    return int(lib().kmip_test_tc_scores(_ptr(Q), _ptr(K), N, H, d, _ptr(scores), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def kmip_test_f16_scores(Q, K, scores, stats, workspace, stream=None) -> int:
    """kmip_test.h: scaled fp16-accumulated scores [H, N, N] of one small graph and the per-head statistics [H, 4]."""
    N, H, d = Q.shape
    return int(lib().kmip_test_f16_scores(_ptr(Q), _ptr(K), N, H, d, _ptr(scores), _ptr(stats), _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream)))


def kmip_test_gemm_tn(A, B, C, workspace, stream=None) -> int:
    """kmip_test.h: C[M, N] = A[M, K] B[N, K]^T (bf16 in, C bf16 or fp32) on the tensor cores."""
    M, K = A.shape
    N = B.shape[0]
    return int(lib().kmip_test_gemm_tn(_ptr(A), _ptr(B), _ptr(C), M, N, K, 1 if C.dtype == torch.float32 else 0,
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def kmip_test_attn_forward(Q, K, V, graph_offsets, k, mode, out, topk_idx, topk_score, workspace, stream=None,
                           wait_limit_cycles=0, drop_first_tile=0, fp32_path=0) -> int:
    """kmip_test.h: the forward pass with per-call test options; returns the library's status code."""
    N, H, d = Q.shape
    G = 0 if graph_offsets is None else int(graph_offsets.numel()) - 1
    opt = TestOptions(int(wait_limit_cycles), int(drop_first_tile), int(fp32_path))
    return int(lib().kmip_test_attn_forward(_ptr(Q), _ptr(K), _ptr(V), _ptr(graph_offsets), G, N, H, d, k, mode,
                                            _ptr(out), _ptr(topk_idx), _ptr(topk_score), _ptr(workspace),
                                            0 if workspace is None else workspace.numel() * workspace.element_size(),
                                            _stream(stream), ctypes.byref(opt)))


def kmip_test_sweep_order(workspace, N, G, H, d, k, mode, stream=None):
    """kmip_test.h: (order, rows_per_item) of the last forward call on `workspace`; order[s] is the row the
    sweep handled at position s (numpy int32 [N])."""
    import numpy as np
    order = np.empty(N, dtype=np.int32)
    rpi = ctypes.c_int32(0)
    rc = lib().kmip_test_sweep_order(_ptr(workspace), N, G, H, d, k, mode, order.ctypes.data_as(ctypes.c_void_p),
                                     ctypes.byref(rpi), _stream(stream))
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_test_sweep_order")
    return order, int(rpi.value)


def kmip_attn_sweep_counters(workspace, stream=None):
    """Work counters of the last forward call on `workspace` (synchronises the stream): (key tiles, key tiles
    loaded, (key tile, query tile) pairs, pairs scored) of the pruned sweep, then the rows the half-precision
    prefilter handed to the exact kernel, then three zeros."""
    c = (ctypes.c_int64 * 8)()
    rc = lib().kmip_attn_sweep_counters(_ptr(workspace), _stream(stream), c)
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_attn_sweep_counters")
    return tuple(int(x) for x in c)


# ------------------------------------------------------------------------------------------------
# Buffer helpers (allocation only)
# ------------------------------------------------------------------------------------------------
def storage_dtype(mode: int):
    return torch.float32 if mode == KMIP_FP32_EXACT else torch.bfloat16


class ForwardBuffers:
    """Outputs and scratch of one forward problem size, allocated once with torch."""

    def __init__(self, N, G, H, d, k, mode, device="cuda"):
        dt = storage_dtype(mode)
        self.out = torch.empty((N, H, d), dtype=dt, device=device)
        self.topk_idx = torch.empty((N, H, k), dtype=torch.int32, device=device)
        self.topk_score = torch.empty((N, H, k), dtype=torch.float32, device=device)
        nbytes = kmip_attn_workspace_bytes(N, G, H, d, k, mode, PASS_FORWARD)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)


class BackwardBuffers:
    """Gradients and scratch of one backward problem size, allocated once with torch."""

    def __init__(self, N, G, H, d, k, mode, device="cuda"):
        dt = storage_dtype(mode)
        self.dQ = torch.empty((N, H, d), dtype=dt, device=device)
        self.dK = torch.empty((N, H, d), dtype=dt, device=device)
        self.dV = torch.empty((N, H, d), dtype=dt, device=device)
        nbytes = kmip_attn_workspace_bytes(N, G, H, d, k, mode, PASS_BACKWARD)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)


def forward(Q, K, V, graph_offsets, k, mode, buffers: ForwardBuffers | None = None, stream=None, check=True,
            fp32_path=0):
    """Allocate (unless given) and run the forward pass; returns the buffers.  fp32_path != 0 goes through
    kmip_test_attn_forward to pin which fp32-mode sweep runs (tests only)."""
    N, H, d = Q.shape
    G = 1 if graph_offsets is None else int(graph_offsets.numel()) - 1
    b = buffers or ForwardBuffers(N, G, H, d, k, mode, Q.device)
    if fp32_path:
        rc = kmip_test_attn_forward(Q, K, V, graph_offsets, k, mode, b.out, b.topk_idx, b.topk_score, b.workspace,
                                    stream, fp32_path=fp32_path)
    else:
        rc = kmip_attn_forward(Q, K, V, graph_offsets, k, mode, b.out, b.topk_idx, b.topk_score, b.workspace, stream)
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_attn_forward")
    if check:
        st = kmip_last_status(b.workspace, stream)
        if st != KMIP_OK:
            raise KmipError(st, "kmip_attn_forward (device)")
    return b


def backward(Q, K, V, graph_offsets, k, mode, fwd: ForwardBuffers, d_out,
             buffers: BackwardBuffers | None = None, stream=None, check=True):
    """Allocate (unless given) and run the backward pass; returns the buffers."""
    N, H, d = Q.shape
    G = 1 if graph_offsets is None else int(graph_offsets.numel()) - 1
    b = buffers or BackwardBuffers(N, G, H, d, k, mode, Q.device)
    rc = kmip_attn_backward(Q, K, V, graph_offsets, k, mode, fwd.out, d_out, fwd.topk_idx, fwd.topk_score,
                            b.dQ, b.dK, b.dV, b.workspace, stream)
    if rc != KMIP_OK:
        raise KmipError(rc, "kmip_attn_backward")
    if check:
        st = kmip_last_status(b.workspace, stream)
        if st != KMIP_OK:
            raise KmipError(st, "kmip_attn_backward (device)")
    return b
