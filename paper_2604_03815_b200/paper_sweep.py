"""The paper's controlled size sweep (Sec. 5 "Objective 1", App. H.2 and the tables of App. J.1 / K)
on this library: one (N x d_K) Q/K/V triple with d_K = 10 and k = 10, normal inputs, time of an
inference pass (forward) and of a training pass (forward + backward) and peak device memory, for
N = 10^(i/2).  The library stores head widths 16/32/64/128, so d_K = 10 is zero-padded to 16.

    python -m paper_2604_03815_b200.paper_sweep [--min-exp 8] [--max-exp 13] [--mode bf16|fp32] [--reps 3]
                                                [--k 10] [--json out.json]

--k changes the number of keys kept (the paper's appendix "Additional results", "Influence of k", reports
whole-model epoch times for k up to 100, where its implementation slows down sharply).
Prints one JSON line per size and a markdown table at the end; --json also writes the rows to a file.
The paper's own figures (A100-40GB, fp32 on CUDA cores, Tables of App. J.1 / K) are printed beside ours
as context: another GPU, another precision, not a target.
"""
import argparse
import json

import numpy as np

from . import binding as kb
from . import workloads as wl

# N -> (inference seconds, training seconds) reported by the paper for k-MIP attention (App. J.1, App. K)
PAPER_SECONDS = {
    10 ** 4: (3.14e-3, None), 31623: (6.38e-3, 8.46e-3), 10 ** 5: (34.45e-3, 39.94e-3),
    316228: (0.231, 0.245), 10 ** 6: (2.146, 2.233), 3162278: (20.966, 21.232), 10 ** 7: (None, 208.338),
}


def run_size(N, mode, reps, k=10):
    import torch

    dev = torch.device("cuda", torch.cuda.current_device())
    w = wl.padded_workload(f"paper_sweep_{N}", 7, N, 1, 10, 16, k, mode)
    dt = kb.storage_dtype(mode)
    torch.cuda.empty_cache()
    torch.cuda.reset_peak_memory_stats(dev)
    Q, K, V, dO = (torch.from_numpy(getattr(w, n)).to(dev, dt) for n in ("Q", "K", "V", "dOut"))
    offs = torch.from_numpy(w.graph_offsets).to(dev)
    fb = kb.ForwardBuffers(N, 1, 1, 16, k, mode, dev)
    bb = kb.BackwardBuffers(N, 1, 1, 16, k, mode, dev)

    def fwd():
        rc = kb.kmip_attn_forward(Q, K, V, offs, k, mode, fb.out, fb.topk_idx, fb.topk_score, fb.workspace)
        assert rc == kb.KMIP_OK, kb.status_string(rc)

    def bwd():
        rc = kb.kmip_attn_backward(Q, K, V, offs, k, mode, fb.out, dO, fb.topk_idx, fb.topk_score, bb.dQ, bb.dK,
                                   bb.dV, bb.workspace)
        assert rc == kb.KMIP_OK, kb.status_string(rc)

    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 1e3 / reps

    fwd()
    bwd()
    torch.cuda.synchronize()
    assert kb.kmip_last_status(fb.workspace) == kb.KMIP_OK and kb.kmip_last_status(bb.workspace) == kb.KMIP_OK
    t_inf = timed(fwd)
    t_train = timed(lambda: (fwd(), bwd()))
    peak = torch.cuda.max_memory_allocated(dev)
    ref = PAPER_SECONDS.get(N, (None, None)) if k == 10 else (None, None)
    return {"N": N, "mode": "bf16" if mode == wl.MODE_BF16_TC else "fp32", "d_K": 10, "stored_d": 16, "k": k,
            "inference_s": t_inf, "training_s": t_train, "scores_per_s_inference": float(N) * N / t_inf,
            "peak_device_bytes": int(peak), "paper_a100_fp32_inference_s": ref[0], "paper_a100_fp32_training_s": ref[1]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--min-exp", type=int, default=8, help="smallest N = 10^(min_exp/2)")
    ap.add_argument("--max-exp", type=int, default=13, help="largest N = 10^(max_exp/2); 14 = ten million nodes")
    ap.add_argument("--mode", choices=["bf16", "fp32"], default="bf16")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--k", type=int, default=10, help="keys kept per query (the paper's sweep uses 10)")
    ap.add_argument("--json", default=None, help="also write the rows to this file")
    args = ap.parse_args()
    mode = wl.MODE_BF16_TC if args.mode == "bf16" else wl.MODE_FP32_EXACT
    rows = []
    for i in range(args.min_exp, args.max_exp + 1):
        N = int(round(10 ** (i / 2)))
        r = run_size(N, mode, args.reps if i < 13 else 1, args.k)
        rows.append(r)
        print(json.dumps(r), flush=True)
    if args.json:
        with open(args.json, "w") as f:
            json.dump(rows, f, indent=1)
    print("\n| N | inference | training | peak device memory | paper (A100-40GB, fp32): inference / training |")
    print("|---|---|---|---|---|")
    for r in rows:
        p = "%s / %s" % tuple("-" if v is None else ("%.3g s" % v) for v in (r["paper_a100_fp32_inference_s"], r["paper_a100_fp32_training_s"]))
        print(f"| {r['N']} | {r['inference_s'] * 1e3:.3f} ms | {r['training_s'] * 1e3:.3f} ms | {r['peak_device_bytes'] / 2**20:.1f} MiB | {p} |")


if __name__ == "__main__":
    main()
