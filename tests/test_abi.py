"""The C-ABI library: it loads without a GPU, exports every symbol the header declares, and
rejects bad arguments on the host before any CUDA call (CPU only)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kb():
    from paper_2604_03815_b200 import build
    build.build()
    from paper_2604_03815_b200 import binding
    return binding


def test_exports_every_declared_symbol(kb):
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(kmip_[a-z0-9_]+)\s*\(", text)
    assert {"kmip_attn_forward", "kmip_attn_backward", "kmip_attn_workspace_bytes", "kmip_last_status",
            "kmip_status_string", "kmip_version"} <= set(names)
    L = kb.lib()
    for n in set(names):
        assert hasattr(L, n), f"{n} is declared in include/ but not exported"
    # and the other direction: the library exports no kmip_* symbol that no header declares
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", kb.LIB_PATH], capture_output=True, text=True, check=True).stdout
    exported = {ln.split()[-1] for ln in out.splitlines() if ln.split() and ln.split()[-1].startswith("kmip_")}
    assert exported == set(names), f"undeclared exports: {sorted(exported - set(names))}"


def test_version_and_status_strings(kb):
    assert kb.kmip_version() >= 100
    assert kb.status_string(0) == "ok"
    assert "offset" in kb.status_string(kb.KMIP_ERR_BAD_OFFSETS)
    assert kb.status_string(12345) == "unknown status"


def test_workspace_bytes_host_only(kb):
    f = kb.kmip_attn_workspace_bytes(500_000, 1, 4, 32, 32, kb.KMIP_BF16_TC, kb.PASS_FORWARD)
    b = kb.kmip_attn_workspace_bytes(500_000, 1, 4, 32, 32, kb.KMIP_BF16_TC, kb.PASS_BACKWARD)
    rows = 500_000 * 4
    kq = 2 * rows * 32 * 2                                    # 2-byte copies of K (regrouped) and Q (sweep order)
    lists = rows * (48 * 6 + 4)                               # half-precision prefilter: 48 groups of 6 bytes per row, redo list
    assert kq + lists < f < kq + lists + 500_000 * 6 + (1 << 20)   # + permutation, codes, work items
    assert f < 2 * rows * 32 * 2 * 4                          # linear in N*H*(d + k): nothing like N^2
    small = kb.kmip_attn_workspace_bytes(20_000, 1, 4, 32, 32, kb.KMIP_BF16_TC, kb.PASS_FORWARD)
    srows = 20_000 * 4
    assert 2 * srows * 64 + srows * 292 < small < 2 * srows * 64 + srows * 292 + (1 << 20)
    # d = 64 runs the fp32-accumulate sweep: one bf16 copy of K only while the row order is kept
    wide = kb.kmip_attn_workspace_bytes(20_000, 1, 4, 64, 32, kb.KMIP_BF16_TC, kb.PASS_FORWARD)
    assert srows * 128 < wide < srows * 128 + (1 << 20)
    assert 256 < kb.kmip_attn_workspace_bytes(500_000, 1, 4, 32, 32, kb.KMIP_FP32_EXACT, kb.PASS_FORWARD) < (1 << 20)
    # pruned mode (fp32-accumulate sweep): copies of K and Q, 16 bytes per node + 4 per (node, head) + (d + 4)
    # floats per (128 nodes, head) for the key tiles and three times that for the query tiles of the work
    # items; below 32768 nodes it keeps the row order and needs the K copy only
    fp = kb.kmip_attn_workspace_bytes(500_000, 1, 4, 32, 32, kb.KMIP_BF16_TC_PRUNED, kb.PASS_FORWARD)
    extra = 500_000 * (16 + 4 * 4) + 4 * (500_000 // 128 + 3) * 4 * 36 * 4
    assert kq + 500_000 * 16 < fp < kq + 500_000 * 6 + extra + (1 << 20)
    sp = kb.kmip_attn_workspace_bytes(20_000, 1, 4, 32, 32, kb.KMIP_BF16_TC_PRUNED, kb.PASS_FORWARD)
    assert srows * 64 < sp < srows * 64 + (1 << 20)
    assert kb.kmip_attn_workspace_bytes(500_000, 1, 4, 32, 32, kb.KMIP_BF16_TC_PRUNED, kb.PASS_BACKWARD) == b
    pairs = 500_000 * 4 * 32
    # p, dS and two buffers of 16-byte hit records (the radix sort that orders them): 40 bytes per selected pair,
    # 12 per (node, head), and the table of digit counts (1024 digits x 4 bytes per block of 4096 pairs)
    assert 40 * pairs < b < 41 * pairs + 14 * 500_000 * 4 + (8 << 20)
    for bad in [dict(d=24), dict(k=129), dict(mode=7)]:
        args = dict(N=1000, G=1, H=2, d=32, k=8, mode=kb.KMIP_BF16_TC)
        args.update(bad)
        with pytest.raises(kb.KmipError) as e:
            kb.kmip_attn_workspace_bytes(args["N"], args["G"], args["H"], args["d"], args["k"], args["mode"], 0)
        assert e.value.status == kb.KMIP_ERR_UNSUPPORTED
    with pytest.raises(kb.KmipError) as e:
        kb.kmip_attn_workspace_bytes(-1, 1, 2, 32, 8, kb.KMIP_BF16_TC, 0)
    assert e.value.status == kb.KMIP_ERR_INVALID_ARG
    with pytest.raises(kb.KmipError) as e:
        kb.kmip_attn_workspace_bytes(1 << 28, 1, 8, 32, 32, kb.KMIP_BF16_TC, 0)   # N*H*k >= 2^31
    assert e.value.status == kb.KMIP_ERR_INVALID_ARG


def test_forward_and_backward_reject_bad_arguments_before_any_cuda_call(kb):
    L = kb.lib()
    p = ctypes.c_void_p(4096)        # never dereferenced: validation fails first
    odd = ctypes.c_void_p(4100)
    fwd = lambda **o: L.kmip_attn_forward(o.get("Q", p), p, p, None, 0, o.get("N", 100), o.get("H", 2), o.get("d", 32),
                                          o.get("k", 8), o.get("mode", 0), p, p, p, o.get("ws", p), o.get("wsb", 1 << 30), None)
    assert fwd(k=0) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(H=0) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(N=-5) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(d=48) == kb.KMIP_ERR_UNSUPPORTED
    assert fwd(k=200) == kb.KMIP_ERR_UNSUPPORTED
    assert fwd(mode=3) == kb.KMIP_ERR_UNSUPPORTED
    assert fwd(Q=None) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(Q=odd) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(ws=None) == kb.KMIP_ERR_INVALID_ARG
    assert fwd(wsb=16) == kb.KMIP_ERR_WORKSPACE
    assert fwd(N=0) == kb.KMIP_OK            # nothing to do, nothing enqueued
    bwd = lambda **o: L.kmip_attn_backward(p, p, p, None, 0, o.get("N", 100), 2, o.get("d", 32), o.get("k", 8), 0,
                                           None, o.get("dO", p), p, p, p, p, p, p, o.get("wsb", 1 << 30), None)
    assert bwd(k=0) == kb.KMIP_ERR_INVALID_ARG
    assert bwd(d=20) == kb.KMIP_ERR_UNSUPPORTED
    assert bwd(dO=None) == kb.KMIP_ERR_INVALID_ARG
    assert bwd(wsb=100) == kb.KMIP_ERR_WORKSPACE
    assert bwd(N=0) == kb.KMIP_OK
    st = ctypes.c_int(0)
    assert L.kmip_last_status(None, None, ctypes.byref(st)) == kb.KMIP_ERR_INVALID_ARG
