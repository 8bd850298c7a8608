"""The outer loop of speculative decoding (Algorithm 3) around the library's kernels, for synthetic
models whose next-token logits depend on the last token only (two [V, V] tables of logits).

    python -m paper_2403_10444_b200.specdec [--V 32768] [--B 64] [--gammas 2,4,8] [--iterations 32]

Each iteration drafts gamma tokens autoregressively with ``bv_draft_chain`` (one launch; or gamma calls of
``bv_sample_draft``), which also leaves every draft row's log-normaliser, looks up the target rows along the drafted path (the stand-in for the
parallel scoring pass of the large model), and verifies the block with ``bv_verify_lse`` (Block
Verification, Algorithm 2), ``bv_verify``, ``tv_verify`` (Token Verification, Algorithm 1) or ``tv_verify_lse``.  The
accepted tokens and the correction token extend every sequence, whose last token is the context of the
next iteration.  Table look-ups and the bookkeeping of sequence positions are torch indexing; sampling
and verification run in the CUDA library.  All random numbers are inputs.

Reported: block efficiency (tokens generated per iteration, the paper's measure) and the law of the
number of accepted tokens tau.  Greedy block verification is not offered here: across iterations it
needs the modified model of Algorithm 5.
"""
from __future__ import annotations

import argparse
import json
import time
from typing import Dict

import torch

from . import binding as bv
from . import workloads as wl

ALGOS = ("block_lse", "block", "token", "token_lse")


def run(target_table: torch.Tensor, draft_table: torch.Tensor, first_tokens: torch.Tensor,
        u_draft: torch.Tensor, u_verify: torch.Tensor, gamma: int, temperature: float = 1.0,
        algo: str = "block_lse", graph: bool = False, chain: bool = True) -> Dict[str, torch.Tensor]:
    """Run ``u_draft.shape[0]`` iterations of Algorithm 3 for ``first_tokens.shape[0]`` sequences.

    target_table, draft_table: CUDA [V, V] float32 or bfloat16 (row t = logits after token t; -inf
    entries, as a top-k / top-p mask leaves them, are allowed); first_tokens: CUDA int32 [B], the
    last token of each context; u_draft [N, gamma, B] and u_verify [N, B, gamma+2]: CUDA float32
    uniforms.  Returns ``tokens`` int32 [B, N (gamma+1)] (generated tokens, then -1), ``lengths``
    int64 [B], ``tau`` int32 [N, B] (accepted draft tokens per iteration) and ``drafted`` int32
    [N, B, gamma].

    Every step of an iteration has fixed shapes and runs on the device without a host round trip
    (the iteration number lives in a device counter), so with ``graph=True`` one iteration is
    captured in a CUDA graph and replayed: the launches of an iteration then cost one graph launch
    instead of one driver call each.  Data faults are looked for once, after the last iteration.
    ``chain``: the gamma drafted tokens of an iteration come from one launch of ``bv_draft_chain``
    (default) instead of gamma calls of ``bv_sample_draft`` with their look-ups and copies.
    """
    if algo not in ALGOS:
        raise ValueError("algo must be one of %s" % (ALGOS,))
    V = target_table.shape[0]
    if tuple(target_table.shape) != (V, V) or tuple(draft_table.shape) != (V, V):
        raise ValueError("the model tables must be [V, V]")
    N, B = u_draft.shape[0], first_tokens.shape[0]
    if tuple(u_draft.shape) != (N, gamma, B) or tuple(u_verify.shape) != (N, B, gamma + 2):
        raise ValueError("u_draft must be [N, gamma, B] and u_verify [N, B, gamma+2]")
    dev = target_table.device
    width = N * (gamma + 1)
    # state of the loop, updated in place (column `width` of seq takes what is not kept)
    seq = torch.full((B, width + 1), -1, dtype=torch.int32, device=dev)
    pos = torch.zeros((B,), dtype=torch.int64, device=dev)
    taus = torch.empty((N, B), dtype=torch.int32, device=dev)
    drafted = torch.empty((N, B, gamma), dtype=torch.int32, device=dev)
    cur = first_tokens.to(torch.int64).clone()
    it = torch.zeros((1,), dtype=torch.int64, device=dev)          # the iteration number, on the device
    fault = torch.zeros((1,), dtype=torch.int32, device=dev)
    draft_logits = torch.empty((B, gamma, V), dtype=draft_table.dtype, device=dev)
    target_logits = torch.empty((B, gamma + 1, V), dtype=target_table.dtype, device=dev)
    lse = torch.empty((B, gamma), dtype=torch.float32, device=dev)
    toks = torch.empty((B, gamma), dtype=torch.int32, device=dev)
    col = torch.arange(gamma + 1, device=dev)
    trash = torch.full((1,), width, dtype=torch.int64, device=dev)

    def iteration():
        ud = u_draft.index_select(0, it)[0]                        # [gamma, B]
        uv = u_verify.index_select(0, it)[0]                       # [B, gamma+2]
        # drafting step: X_1..X_gamma ~ M_s autoregressively, keeping the conditional rows
        if chain:
            # (one launch for the whole chain; the rows it went through are gathered afterwards)
            tok, row_lse = bv.bv_draft_chain(draft_table, cur.to(torch.int32), ud.contiguous(), temperature)
            toks.copy_(tok)
            lse.copy_(row_lse)
            path = torch.cat([cur[:, None], toks.to(torch.int64)], dim=1)
            torch.index_select(draft_table, 0, path[:, :gamma].reshape(-1), out=draft_logits.view(B * gamma, V))
        else:
            last = cur
            for i in range(gamma):
                rows = draft_table.index_select(0, last)
                tok, row_lse = bv.bv_sample_draft(rows, ud[i], temperature)
                draft_logits[:, i] = rows
                lse[:, i] = row_lse
                toks[:, i] = tok
                last = tok.to(torch.int64)
            path = torch.cat([cur[:, None], toks.to(torch.int64)], dim=1)
        # the large model's conditional rows along the drafted path, gamma + 1 of them
        torch.index_select(target_table, 0, path.reshape(-1), out=target_logits.view(B * (gamma + 1), V))
        if algo == "block_lse":
            out, out_len = bv.bv_verify_lse(target_logits, draft_logits, toks, uv, lse, temperature)
        elif algo == "token_lse":
            out, out_len = bv.tv_verify_lse(target_logits, draft_logits, toks, uv, lse, temperature)
        elif algo == "block":
            out, out_len = bv.bv_verify(target_logits, draft_logits, toks, uv, temperature)
        else:
            out, out_len = bv.tv_verify(target_logits, draft_logits, toks, uv, temperature)
        fault.add_((out_len < 1).any().to(torch.int32))
        n_out = out_len.to(torch.int64).clamp_(min=1)
        keep = col[None, :] < n_out[:, None]
        seq.scatter_(1, torch.where(keep, pos[:, None] + col[None, :], trash), out)
        cur.copy_(out.gather(1, (n_out - 1)[:, None]).squeeze(1))
        pos.add_(n_out)
        taus.index_copy_(0, it, (out_len - 1)[None, :])
        drafted.index_copy_(0, it, toks[None])
        it.add_(1)

    if graph and N > 1:
        # the first iteration runs eagerly on the side stream (the library sizes its workspace for
        # that stream, torch its caches); the second is captured, and replayed for the rest
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            iteration()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            iteration()
        # (capturing has not run anything: replay it for iterations 1 .. N-1)
        torch.cuda.current_stream(dev).wait_stream(side)
        for _ in range(N - 1):
            g.replay()
    else:
        for _ in range(N):
            iteration()
    if int(fault.item()) != 0:
        raise RuntimeError("a sequence reported a data fault (out_len = -1)")
    return dict(tokens=seq[:, :width].contiguous(), lengths=pos, tau=taus, drafted=drafted)


def block_efficiency(result) -> float:
    """Tokens generated per iteration (accepted draft tokens + the correction token), averaged."""
    return float(result["tau"].float().mean().item()) + 1.0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--V", type=int, default=32768)
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--gammas", default="2,4,8")
    ap.add_argument("--iterations", type=int, default=32)
    ap.add_argument("--draft-sigma", type=float, default=1.0)
    ap.add_argument("--temperature", type=float, default=1.0)
    ap.add_argument("--seed", type=int, default=7)
    ap.add_argument("--top-p", type=float, default=0.0, help="mask both models' rows to their top-p nucleus")
    ap.add_argument("--graph", action="store_true", help="replay one captured iteration as a CUDA graph")
    ap.add_argument("--no-chain", action="store_true", help="draft with gamma sampler calls instead of one chain launch")
    args = ap.parse_args()
    bv.load_library()
    tt, dt = wl.markov_models(args.V, "bf16", args.seed, 2.0, args.draft_sigma, 1.1, "cuda")
    if args.top_p > 0:
        tt, dt = wl.top_p_mask(tt, args.top_p, args.temperature), wl.top_p_mask(dt, args.top_p, args.temperature)
    first = torch.zeros((args.B,), dtype=torch.int32, device="cuda")
    for gamma in [int(x) for x in args.gammas.split(",")]:
        ud, uv = wl.loop_uniforms(args.iterations, args.B, gamma, args.seed + gamma, "cuda")
        for algo in ALGOS:
            run(tt, dt, first, ud[:2], uv[:2], gamma, args.temperature, algo, args.graph, not args.no_chain)       # warm-up
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            res = run(tt, dt, first, ud, uv, gamma, args.temperature, algo, args.graph, not args.no_chain)
            torch.cuda.synchronize()
            dt_s = time.perf_counter() - t0
            print(json.dumps({"V": args.V, "B": args.B, "gamma": gamma, "algo": algo,
                              "iterations": args.iterations, "draft_sigma": args.draft_sigma,
                              "temperature": args.temperature, "top_p": args.top_p or None, "graph": args.graph, "chain": not args.no_chain,
                              "block_efficiency": round(block_efficiency(res), 4),
                              "tokens": int(res["lengths"].sum().item()),
                              "ms_per_iteration": round(dt_s / args.iterations * 1e3, 3),
                              "tokens_per_s": round(float(res["lengths"].sum().item()) / dt_s, 1)}), flush=True)


if __name__ == "__main__":
    main()
