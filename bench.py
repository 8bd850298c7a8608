#!/usr/bin/env python
"""Benchmark of the draft-verification hot path.

A "step" is one Block Verification call (every stage: normalisers, drafted-token
probabilities, prefix recursion, residual masses, acceptance weights, selection
of tau, residual sample) over one batch of synthetic logits.  The default
workload is B=256, gamma=8, V=256000, bf16 (2.2 GB of logits, far larger than
L2, so nothing is served from cache between steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c1|c2|c3|c4] [--algo block|token|sample|block_lse|token_lse|greedy|block_probs|token_probs]

Prints one JSON line.  With N > 1 (launched by torch.distributed.run) every rank
verifies its own batch of the same shape (weak scaling, no collective on the
data path); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2403_10444_b200 import workloads as wl  # noqa: E402
from paper_2403_10444_b200 import sharding  # noqa: E402

METRIC = "verifications/s (B*gamma logit rows)"
UNIT = "verifications/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        # NCCL's own account of the communicator (topology, transports) goes to a file in the system's
        # temporary directory, not to stdout, where the one JSON line must stay alone
        if "NCCL_DEBUG" not in os.environ:
            import tempfile
            os.environ["NCCL_DEBUG"] = "INFO"
            os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "bv_bench_nccl_%h_%p.log"))
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return rank, world, local, dist
    return 0, 1, 0, None


class OracleRun:
    """The CPU oracle, as it stands, on a bounded sample of the workload.

    The sample (the first n sequences, n sized from one probe pass so that a pass over it takes about
    ``pass_s`` seconds) is generated once; every call of :meth:`one_pass` verifies it again.
    """

    def __init__(self, w, algo_name: str, pass_s: float):
        import oracle
        self.oracle, self.w, self.algo_name = oracle, w, algo_name
        self.algo = {"block": oracle.BLOCK_VERIFY, "block_lse": oracle.BLOCK_VERIFY, "block_probs": oracle.BLOCK_VERIFY,
                     "greedy": oracle.GREEDY_BLOCK_VERIFY}.get(algo_name, oracle.TOKEN_VERIFY)
        self.probs = algo_name.endswith("_probs")
        self.cores = oracle.threads()
        probe = self._prepare(wl.make_inputs(wl.scaled(w, B=max(1, min(w.B, self.cores))), "cpu"))
        per_seq = self._run(probe) / probe["B"]
        n = int(max(1, min(w.B, pass_s / max(per_seq, 1e-9))))
        self.n = max(min(n, w.B), min(w.B, self.cores))
        self.sample = probe if self.n == probe["B"] else self._prepare(wl.make_inputs(wl.scaled(w, B=self.n), "cpu"))

    def _prepare(self, inp):
        import numpy as np
        t, d = inp["target_logits"], inp["draft_logits"]
        if self.probs:      # (the distributions handed over as probabilities in the storage type, as on the GPU)
            t = torch.softmax(t.float() / inp["temperature"], -1).to(t.dtype)
            d = torch.softmax(d.float() / inp["temperature"], -1).to(d.dtype)
        if t.dtype == torch.bfloat16:
            t = t.view(torch.int16).numpy().view(np.uint16); d = d.view(torch.int16).numpy().view(np.uint16)
        else:
            t = t.numpy(); d = d.numpy()
        g = inp["draft_tokens"].shape[1]
        p = {"t": t, "d": d, "x": inp["draft_tokens"].numpy(), "u": inp["uniforms"].numpy(),
             "T": inp["temperature"], "B": inp["draft_tokens"].shape[0]}
        if self.algo_name.endswith("_lse"):
            p["lse"] = torch.logsumexp(inp["draft_logits"].double() / inp["temperature"], -1).float().numpy()
        if self.algo_name == "sample":
            p["rows"] = d.reshape(-1, d.shape[-1])
            p["u_rows"] = p["u"][:, :g].reshape(-1).copy()
        return p

    def _run(self, p) -> float:
        o = self.oracle
        t0 = time.perf_counter()
        if self.algo_name == "sample":
            o.sample_rows(p["rows"], p["u_rows"], p["T"])
        elif self.probs:
            o.verify_probs(self.algo, p["t"], p["d"], p["x"], p["u"])
        elif self.algo_name.endswith("_lse"):
            o.verify(self.algo, p["t"], p["d"], p["x"], p["u"], p["T"], draft_lse=p["lse"])
        else:
            o.verify(self.algo, p["t"], p["d"], p["x"], p["u"], p["T"])
        return time.perf_counter() - t0

    def one_pass(self) -> float:
        """Seconds the oracle takes for the sample."""
        return self._run(self.sample)

    def describe(self, passes: int, seconds: float) -> str:
        what = "drafting step" if self.algo_name == "sample" else \
            self.algo_name.replace("_lse", " with supplied draft normalisers").replace("_probs", " on probabilities") + " verify"
        return "first %d of %d sequences of workload %s (%s), %d passes of %.2f s" % (
            self.n, self.w.B, self.w.name, what, passes, seconds)


def time_oracle(w, algo_name: str, budget_s: float = 20.0):
    """cpu_baseline record: the oracle goes through a whole workload in about a second on a many-core
    host, so the sample is repeated until about half the budget is spent (not one noisy second)."""
    run = OracleRun(w, algo_name, budget_s)
    dt, reps = 0.0, 0
    while reps == 0 or (dt < 0.5 * budget_s and reps < 64):
        dt += run.one_pass()
        reps += 1
    dt /= reps
    return {"value": run.n * w.gamma / dt, "unit": UNIT, "cores": run.cores, "kind": "oracle",
            "sample": run.describe(reps, dt)}


def reference_arm(args, w):
    """The oracle on the host cores, one pass over its bounded sample per step; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    steps, warmup = args.steps, args.warmup
    run = OracleRun(w, args.algo, max(0.5, min(10.0, 120.0 / max(1, steps + warmup))))
    times = [run.one_pass() for _ in range(warmup + steps)][warmup:]
    ms = 1e3 * sum(times) / len(times)
    value = run.n * w.gamma / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "gamma": w.gamma, "V": w.V, "storage": w.dtype,
                       "algo": args.algo, "step": "%d sequences per step (bounded sample)" % run.n},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": run.cores, "kind": "oracle",
                             "sample": run.describe(steps, ms * 1e-3)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(wl.CONFIGS))
    ap.add_argument("--algo", default="block", choices=["block", "token", "sample", "block_lse", "token_lse", "greedy", "block_probs", "token_probs"],
                    help="block / token verification, the drafting step (sampling the draft rows), block "
                         "verification with the draft normalisers that the drafting step leaves, or one "
                         "iteration of greedy block verification (Algorithm 4); block_probs / token_probs: the "
                         "two verifications on the workload's distributions given as probabilities")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override B (profiling on a smaller case)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="library tuning option set before the run (bv_set_option), may be repeated")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = wl.CONFIGS[args.workload]
    if args.batch > 0:
        w = wl.scaled(w, B=args.batch, name="%s_B%d" % (w.name, args.batch))

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain program: become the launcher of one rank per GPU (each rank runs this file again)
        sys.exit(sharding.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if args.impl == "reference":
        reference_arm(args, w)
        return

    import paper_2403_10444_b200 as bv
    bv.load_library()  # fails loudly if the CUDA library was not built
    for o in args.option:
        name, _, val = o.partition("=")
        bv.bv_set_option(name, int(val))
    rank, world, local, dist = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    # weak scaling: every rank draws its own batch of the same shape
    inp = wl.make_inputs(wl.scaled(w, seed=w.seed + 1000 * rank), dev)
    fn = bv.bv_verify if args.algo == "block" else bv.tv_verify
    a = (inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"], inp["temperature"])
    if args.algo == "sample":
        # the drafting step on the same draft rows: B gamma rows of V logits, one uniform each
        rows2d = inp["draft_logits"].view(w.B * w.gamma, w.V)
        u_rows = inp["uniforms"][:, : w.gamma].contiguous().view(-1)
        fn = lambda *_: bv.bv_sample_draft(rows2d, u_rows, inp["temperature"])
        args.e2e_steps = 0          # (no host-buffer form of this entry point)
    if args.algo in ("block_lse", "token_lse"):
        # normalisers as the drafting step leaves them, computed once outside the timed region
        lse = bv.bv_sample_draft(inp["draft_logits"].view(w.B * w.gamma, w.V),
                                 inp["uniforms"][:, : w.gamma].contiguous().view(-1), inp["temperature"])[1]
        lse = lse.view(w.B, w.gamma).contiguous()
        lfn = bv.bv_verify_lse if args.algo == "block_lse" else bv.tv_verify_lse
        fn = lambda *_: lfn(*a[:4], lse, a[4])
        args.e2e_steps = 0
    if args.algo == "greedy":
        fn = bv.gbv_verify
        args.e2e_steps = 0          # (no host-buffer form of this entry point)
    if args.algo in ("block_probs", "token_probs"):
        # the same distributions, handed over as probabilities in the storage type (formed outside the timed region)
        pt = torch.empty_like(inp["target_logits"]); pd = torch.empty_like(inp["draft_logits"])
        for b0 in range(0, w.B, 16):
            pt[b0:b0 + 16] = torch.softmax(inp["target_logits"][b0:b0 + 16].float() / inp["temperature"], -1).to(pt.dtype)
            pd[b0:b0 + 16] = torch.softmax(inp["draft_logits"][b0:b0 + 16].float() / inp["temperature"], -1).to(pd.dtype)
        pfn = bv.bv_verify_probs if args.algo == "block_probs" else bv.tv_verify_probs
        fn = lambda *_: pfn(pt, pd, a[2], a[3])
        args.e2e_steps = 0

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        fn(*a)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    launches = 0
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.profiler.start()      # (a profiler started with capture off sees exactly the timed steps)
    start.record()
    for i in range(args.steps):
        evs[i][0].record()
        out = fn(*a)
        evs[i][1].record()
        launches += 1 if args.algo == "sample" else bv.bv_last_launch_count()
    args.kernel_code = bv.bv_last_kernel()
    stop.record()
    barrier()
    torch.cuda.profiler.stop()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = start.elapsed_time(stop)
    kernel_ms = [e0.elapsed_time(e1) for e0, e1 in evs]
    total_ms = sharding.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = sharding.whole_job_rate(w.B * w.gamma, ms_per_step)

    # ---- for the record: the same call with every position evaluated in full (diagnostic entry) ----
    full_ms = None
    if args.algo == "block":
        for _ in range(2):
            bv.bv_verify_ex(*a)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(5):
            bv.bv_verify_ex(*a)
        f1.record()
        f1.synchronize()
        full_ms = f0.elapsed_time(f1) / 5
    args.full_ms = full_ms
    # ---- Algorithm 1 on the same batch (the baseline the paper compares with), same timing rules ----
    args.token = None
    if args.algo == "block":
        n_tok = max(3, min(args.steps, 10))
        for _ in range(3):
            tok_out = bv.tv_verify(*a)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n_tok):
            tok_out = bv.tv_verify(*a)
        t1.record()
        t1.synchronize()
        tok_ms = sharding.max_over_ranks(t0.elapsed_time(t1) / n_tok, dev)
        args.token = (tok_ms, n_tok, tok_out)

    # ---- end to end: host buffers through the C-ABI host entry, copies inside the timed region ----
    e2e = None
    if args.e2e_steps > 0:
        e2e = end_to_end(args, w, inp, out, bv, barrier, dist, dev, world)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    finish(args, w, world, value, ms_per_step, kernel_ms, clocks, e2e, launches, out, dist)


def end_to_end(args, w, inp, out, bv, barrier, dist, dev, world):
    host = {k: (v.cpu().pin_memory() if torch.is_tensor(v) else v) for k, v in inp.items()}
    hfn = bv.bv_verify_host if args.algo == "block" else bv.tv_verify_host
    ha = (host["target_logits"], host["draft_logits"], host["draft_tokens"], host["uniforms"], host["temperature"])
    ot = torch.empty((w.B, w.gamma + 1), dtype=torch.int32).pin_memory()
    ol = torch.empty((w.B,), dtype=torch.int32).pin_memory()
    hfn(*ha, out_tokens=ot, out_len=ol)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        hfn(*ha, out_tokens=ot, out_len=ol)
    e2e_s = (time.perf_counter() - t0) / args.e2e_steps
    e2e_s = sharding.max_over_ranks(e2e_s, dev)
    h2d = sum(host[k].numel() * host[k].element_size()
              for k in ("target_logits", "draft_logits", "draft_tokens", "uniforms"))
    d2h = ot.numel() * 4 + ol.numel() * 4
    assert torch.equal(ot, out[0].cpu()) and torch.equal(ol, out[1].cpu()), "host and device entry points disagree"
    return {"value": world * w.B * w.gamma / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}


def token_bytes(w, out_len) -> int:
    """Algorithm 1 stops at the first rejection: a sequence that emits n tokens needs the row pairs
    0 .. min(n, gamma) - 1 and, when all gamma tokens were accepted, target row gamma."""
    n = out_len.long().clamp(min=0)
    rows = 2 * n.clamp(max=w.gamma) + (n == w.gamma + 1).long()
    return int(rows.sum().item()) * w.V * (4 if w.dtype == "f32" else 2)


def finish(args, w, world, value, ms_per_step, kernel_ms, clocks, e2e, launches, out, dist):
    peak, peak_src = measured_peak()
    k_ms = statistics.mean(kernel_ms)
    mean_len = float(out[1].float().mean().item()) if args.algo != "sample" else None
    esz = 4 if w.dtype == "f32" else 2
    if args.algo == "sample":
        algo_bytes = w.B * w.gamma * w.V * esz
        kernel = "sample_rows_kernel"
    elif args.algo == "block_lse":
        # what must be read at least: every target row, and one draft row per block for the residual
        algo_bytes = w.B * (w.gamma + 2) * w.V * esz
        kernel = "verify_flow_kernel"
    elif args.algo == "token_lse":
        # Algorithm 1 with supplied draft normalisers: target rows 0 .. min(n, gamma) - 1 for the tests, the target
        # row at tau (already among them unless every token was accepted) and the draft row at tau for the residual
        n = out[1].long().clamp(min=0)
        algo_bytes = int((n.clamp(max=w.gamma) + 1).sum().item()) * w.V * esz
        kernel = "verify_flow_kernel"
    elif args.algo in ("block_probs", "token_probs"):
        # given probabilities, what must be read is the row pair at the selected position (or the last
        # target row) of every sequence, besides the 2 gamma entries of its drafted tokens
        n = out[1].long().clamp(min=0)
        algo_bytes = int((2 * (n <= w.gamma).long() + (n == w.gamma + 1).long()).sum().item()) * w.V * esz
        kernel = "verify_flow_kernel"
    elif args.algo in ("block", "greedy"):
        # Algorithms 2 and 4 need every row: B (2 gamma + 1) V elements
        algo_bytes = w.logit_bytes
        kernel = "verify_flow_kernel"
    else:
        algo_bytes = token_bytes(w, out[1])
        kernel = "verify_flow_kernel"
    if args.algo != "sample":      # (the library says which of its verification kernels the shape got)
        kernel = {1: "verify_flow_kernel", 2: "verify_cluster_kernel", 3: "verify_stream_kernel",
                  4: "verify_small_kernel"}.get(getattr(args, "kernel_code", 0), kernel)
    achieved = algo_bytes / (k_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "gamma": w.gamma, "V": w.V, "storage": w.dtype,
                   "temperature": w.temperature, "algo": args.algo, "parallelism": "batch-sharded x%d" % world,
                   "options": args.option or None,
                   "l2": "inputs (%.2f GB per step) exceed L2" % (w.logit_bytes / 1e9),
                   "mean_emitted_len": mean_len,
                   # Algorithm 2's residual masses are evaluated only for positions that can be the selected
                   # one (h_i <= p_i), with identical outputs; the time with all of them evaluated:
                   "all_positions_ms_per_step": getattr(args, "full_ms", None)},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": TRAFFIC_BYTES.get((w.name, args.algo, kernel)),
                     "peak_source": peak_src, "kernel": kernel, "kernel_ms": k_ms,
                     "algorithmic_bytes": algo_bytes, "frac_of_8TBps": achieved / 8000.0},
        "sequences_per_s": world * w.B / (ms_per_step * 1e-3),
    }
    if getattr(args, "token", None):
        tok_ms, n_tok, tok_out = args.token
        tb = token_bytes(w, tok_out[1])
        rejected = int((tok_out[1] <= w.gamma).sum().item())
        line["token"] = {
            "algo": "token (Algorithm 1), same batch, same kernel machinery", "ms_per_step": tok_ms, "steps": n_tok,
            "value": world * w.B * w.gamma / (tok_ms * 1e-3), "unit": UNIT,
            "mean_emitted_len": float(tok_out[1].float().mean().item()),
            # bytes Algorithm 1 needs when nothing is read twice; the kernel reads the row pair at the
            # stopping position a second time for the residual sample
            "algorithmic_bytes": tb, "achieved": tb / (tok_ms * 1e-3) / 1e9, "frac": tb / (tok_ms * 1e-3) / 1e9 / peak,
            "second_sweep_bytes": rejected * 2 * w.V * esz,
            "block_over_token_time": ms_per_step / tok_ms}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = time_oracle(w, args.algo)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the one-pass
# ncu capture of this command at full size that profiles/ summarises; None for a workload or
# kernel with no capture.
TRAFFIC_BYTES = {
    ("c4", "block", "verify_flow_kernel"): 2544254464,
    ("c4", "token", "verify_flow_kernel"): 826027264,
    ("c4", "greedy", "verify_flow_kernel"): 2567559424,
    ("c4", "block_lse", "verify_flow_kernel"): 1486017536,
    ("c4", "sample", "sample_rows_kernel"): 1058338048,
    ("c4", "block_probs", "verify_flow_kernel"): 350525696,
    ("c4", "token_probs", "verify_flow_kernel"): 264830208,
}


if __name__ == "__main__":
    main()
