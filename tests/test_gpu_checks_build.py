"""The -DKMIP_CHECKS build of the library (libkmip_checks.so) as a stand-in for a memory checker:
canary blocks between the workspace regions, verified after every pass, and device-side tests of
the indices the kernels follow; failures are recorded as KMIP_ERR_CHECK, nothing traps.  The small-shape
soak runs under it in a child process (the library is chosen by KMIP_LIBRARY at import time), every
call must leave the status word at KMIP_OK and pass the usual parity checks; one deliberately bad
input (an index no forward pass can have written) must be reported."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import numpy as np, torch
from paper_2604_03815_b200 import binding as kb, workloads as wl
from tests import parity_util as pu
assert kb.kmip_build_flags() & 1, "not the checks build"
plain = 20_000 * 4 * (32 * 2 * 2 + 48 * 6 + 4)
assert kb.kmip_attn_workspace_bytes(20_000, 1, 4, 32, 32, kb.KMIP_BF16_TC, kb.PASS_FORWARD) > plain   # canaries are counted
rng = np.random.default_rng(11)
cases = 0
for case in range(40):
    H = int(rng.integers(1, 4)); d = int(rng.choice([16, 32, 64, 128]))
    k = int(rng.choice([1, 5, 8, 16, 31, 32, 33, 64]))
    sizes = rng.integers(0, int(rng.choice([10, 140, 600, 1500])), size=int(rng.integers(1, 10))).tolist()
    if sum(sizes) == 0: sizes[0] = 3
    mode = wl.MODE_BF16_TC if rng.random() < 0.75 else wl.MODE_FP32_EXACT
    w = wl.iid_workload("s", 810000 + case, sizes, H, d, k, mode, input_scale=1.0 / np.sqrt(d))
    dev = pu.to_device(w)
    fb = pu.run_forward(w, dev)           # raises on any device status, KMIP_ERR_CHECK included
    pu.check_forward(w, fb)
    pu.check_backward(w, fb, pu.run_backward(w, fb, dev))
    cases += 1
for cfg, kw in ((4, dict(N=40000, H=2, d=32, k=32)), (5, dict(n_per_graph=12000)), (3, dict(N=36000))):
    for mode in (kb.KMIP_BF16_TC, kb.KMIP_BF16_TC_PRUNED):       # reordered rows, both prefilter kernels, the pruned sweep
        import dataclasses
        w = dataclasses.replace(wl.make_config(cfg, **kw), mode=mode)
        dev = pu.to_device(w)
        fb = pu.run_forward(w, dev)
        pu.check_forward(w, fb, wl.sample_rows(w, 64))
        pu.run_backward(w, fb, dev)
        cases += 1
# a host-made fault: an index beyond the batch in the saved selection must be reported by the checks build
w = wl.iid_workload("s", 820000, [300], 1, 32, 8, wl.MODE_BF16_TC)
Q, K, V, dO, offs = pu.to_device(w)
fb = pu.run_forward(w, (Q, K, V, dO, offs))
fb.topk_idx[7, 0, 3] = w.N + 5
bb = kb.BackwardBuffers(w.N, 1, w.H, w.d, w.k, w.mode)
assert kb.kmip_attn_backward(Q, K, V, offs, w.k, w.mode, fb.out, dO, fb.topk_idx, fb.topk_score, bb.dQ, bb.dK, bb.dV, bb.workspace) == kb.KMIP_OK
assert kb.kmip_last_status(bb.workspace) == kb.KMIP_ERR_CHECK
assert "canary" in kb.status_string(kb.KMIP_ERR_CHECK)
pu.check_forward(w, pu.run_forward(w, (Q, K, V, dO, offs)))     # the context is still usable
print("CHECKS_BUILD_OK", cases)
"""


def test_small_shape_soak_under_the_checks_build():
    lib = os.path.join(ROOT, "paper_2604_03815_b200", "libkmip_checks.so")
    if not os.path.exists(lib):
        from paper_2604_03815_b200 import build
        build.build(checks=True)
    env = dict(os.environ, KMIP_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "CHECKS_BUILD_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
