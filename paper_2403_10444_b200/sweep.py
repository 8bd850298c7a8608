"""Sweep of the verification step over batch size, block length and draft quality.

    python -m paper_2403_10444_b200.sweep [--calls 20] [--algos block,token] [--markdown]

Every cell is one synthetic workload with V = 152064 (bf16 storage, T = 0.8): B sequences,
gamma drafted tokens, draft logits = target logits + Gaussian noise of the given sigma.  A cell
is timed with CUDA events around single calls after three warm-up calls; between calls a buffer
larger than L2 is overwritten whenever the cell's logits would fit into L2 twice over, so no
cell is served from cache.  Reported per cell: median milliseconds per call, verifications/s
(B gamma per call), the bytes of all logits divided by the time as a fraction of the HBM copy
bandwidth, the mean number of accepted tokens tau and, for Block Verification, the expectation of tau
over the uniforms given the drafted blocks (from the acceptance weights the library returns).  Small cells are bound by launch
latency and by the chain of dependent rows, not by bandwidth.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import torch

from . import binding as bv
from . import workloads as wl

L2_BYTES = 126 * 1024 * 1024


def hbm_peak_gbs() -> float:
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def time_cell(w: wl.Workload, algo: str, calls: int, flush: torch.Tensor):
    inp = wl.make_inputs(w, "cuda")
    fn = bv.bv_verify if algo == "block" else bv.tv_verify
    a = (inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"], inp["temperature"])
    need_flush = w.logit_bytes < 2 * L2_BYTES
    for _ in range(3):
        out = fn(*a)
    torch.cuda.synchronize()
    ms = []
    for _ in range(calls):
        if need_flush:
            flush.add_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn(*a)
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    med = statistics.median(ms)
    tau = float((out[1].float() - 1).mean().item())
    # For Block Verification the acceptance weights h_i that the library returns give the expectation
    # of tau over the uniforms, Pr(tau = i) = h_i prod_{j > i} (1 - h_j), which is far less noisy than
    # the single draw above when B is small.
    exp_tau = None
    if algo == "block":
        h = bv.bv_verify_ex(*a)[2]["h"].double().clamp(0.0, 1.0)
        tail = torch.ones_like(h[:, 0])
        e = torch.zeros_like(tail)
        for i in range(w.gamma, 0, -1):
            e = e + i * h[:, i] * tail
            tail = tail * (1.0 - h[:, i])
        exp_tau = float(e.mean().item())
    return {"B": w.B, "gamma": w.gamma, "sigma": w.draft_sigma, "algo": algo, "ms": med, "ms_min": min(ms), "expected_tau": exp_tau,
            "verifications_per_s": w.B * w.gamma / (med * 1e-3),
            "frac_hbm": w.logit_bytes / (med * 1e-3) / 1e9 / hbm_peak_gbs(), "mean_tau": tau,
            "flushed": need_flush}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--algos", default="block,token")
    ap.add_argument("--batches", default=",".join(str(b) for b in wl.SWEEP_B))
    ap.add_argument("--gammas", default=",".join(str(g) for g in wl.SWEEP_GAMMA))
    ap.add_argument("--sigmas", default=",".join(str(s) for s in wl.SWEEP_SIGMA))
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args()
    bv.load_library()
    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device; there is no CPU fallback")
    flush = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device="cuda")
    rows = []
    for B in (int(x) for x in args.batches.split(",")):
        for g in (int(x) for x in args.gammas.split(",")):
            for s in (float(x) for x in args.sigmas.split(",")):
                for algo in args.algos.split(","):
                    rows.append(time_cell(wl.sweep_cell(B, g, s), algo, args.calls, flush))
                    if not args.markdown:
                        print(json.dumps(rows[-1]), flush=True)
    if args.markdown:
        print("| B | gamma | sigma | algo | ms / call (median) | verifications/s | logits bytes / time, of HBM copy peak | mean tau | E[tau] given the blocks |")
        print("|---|---|---|---|---|---|---|---|---|")
        for r in rows:
            print("| %d | %d | %g | %s | %.4f | %.3g | %.3f | %.2f | %s |" % (
                r["B"], r["gamma"], r["sigma"], r["algo"], r["ms"], r["verifications_per_s"], r["frac_hbm"], r["mean_tau"],
                "%.2f" % r["expected_tau"] if r["expected_tau"] is not None else "-"))


if __name__ == "__main__":
    main()
