"""Seeded synthetic inputs for draft verification: the five benchmark workloads.

This module only draws inputs (logits, drafted tokens, uniforms).  It holds
none of the verification arithmetic and is used by both the CUDA path's tests
and benchmark and by the CPU oracle's tests, which receive the same bits.

Recipe shared by every workload: target logits [B, gamma+1, V] are drawn in
fp32; draft logits [B, gamma, V] are the fp32 target rows 0..gamma-1 plus iid
Gaussian noise; both are then rounded to the storage dtype.  Drafted tokens are
drawn from softmax(stored draft logits / T) row by row (so X_i ~ Q_{i-1}
exactly as the verifier sees it); uniforms are iid U[0, 1) in fp32,
[B, gamma+2].  All draws come from one torch.Generator seeded per workload on
the device the tensors are created on, sequence by sequence.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    gamma: int
    V: int
    dtype: str            # "f32" | "bf16"
    temperature: float
    seed: int
    target_sigma: float   # std of the iid Gaussian part of the target logits
    zipf: float           # coefficient a of the -a * ln(rank) term under a random permutation (0: none)
    boost_tokens: int     # number of randomly chosen tokens per row raised by boost_value
    boost_value: float
    draft_sigma: float    # std of the noise added to the target to form the draft

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def logit_bytes(self) -> int:
        """Minimum bytes a verification must read: B (2 gamma + 1) V sizeof(dtype)."""
        return self.B * (2 * self.gamma + 1) * self.V * (4 if self.dtype == "f32" else 2)


CONFIGS: Dict[str, Workload] = {
    # small case the CPU oracle finishes in well under a second
    "c1": Workload("c1", 1, 4, 1024, "f32", 1.0, 0, 2.0, 0.0, 0, 0.0, 0.5),
    "c2": Workload("c2", 8, 8, 32000, "f32", 1.0, 1, 3.0, 0.0, 50, 8.0, 1.0),
    "c3": Workload("c3", 64, 8, 128256, "bf16", 0.8, 2, 0.3, 1.1, 0, 0.0, 0.7),
    # roofline headline
    "c4": Workload("c4", 256, 8, 256000, "bf16", 1.0, 3, 3.0, 1.1, 0, 0.0, 1.5),
}


def sweep_cell(B: int, gamma: int, draft_sigma: float) -> Workload:
    """One cell of the V = 152064 sweep (generated like c3, seed 4)."""
    return Workload("c5_B%d_g%d_s%g" % (B, gamma, draft_sigma), B, gamma, 152064, "bf16", 0.8, 4,
                    0.3, 1.1, 0, 0.0, draft_sigma)


SWEEP_B = (1, 16, 64, 256, 512)
SWEEP_GAMMA = (2, 4, 8, 16)
SWEEP_SIGMA = (0.1, 1.0, 3.0)


def scaled(w: Workload, **kw) -> Workload:
    """A smaller or larger copy of a workload (same recipe, different sizes)."""
    return replace(w, **kw)


def make_inputs(w: Workload, device="cpu") -> Dict[str, torch.Tensor]:
    """Draw the inputs of one workload on ``device``.

    Returns target_logits, draft_logits (storage dtype), draft_tokens (int32),
    uniforms (float32) and the temperature.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    g, V, B = w.gamma, w.V, w.B
    tgt = torch.empty((B, g + 1, V), dtype=w.torch_dtype, device=dev)
    drf = torch.empty((B, g, V), dtype=w.torch_dtype, device=dev)
    tok = torch.empty((B, g), dtype=torch.int32, device=dev)
    uni = torch.empty((B, g + 2), dtype=torch.float32, device=dev)
    log_rank = torch.log(torch.arange(1, V + 1, dtype=torch.float32, device=dev)) if w.zipf else None
    for b in range(B):
        t = torch.randn((g + 1, V), generator=gen, device=dev, dtype=torch.float32) * w.target_sigma
        if w.zipf:
            # rank_k under a random permutation per row
            perm = torch.rand((g + 1, V), generator=gen, device=dev).argsort(dim=1)
            t = t - w.zipf * log_rank[perm]
        if w.boost_tokens:
            idx = torch.rand((g + 1, V), generator=gen, device=dev).argsort(dim=1)[:, : w.boost_tokens]
            t.scatter_add_(1, idx, torch.full(idx.shape, w.boost_value, device=dev))
        d = t[:g] + torch.randn((g, V), generator=gen, device=dev, dtype=torch.float32) * w.draft_sigma
        tgt[b] = t.to(w.torch_dtype)
        drf[b] = d.to(w.torch_dtype)
        q = torch.softmax(drf[b].float() / w.temperature, dim=-1)
        tok[b] = torch.multinomial(q, 1, generator=gen).squeeze(1).to(torch.int32)
        uni[b] = torch.rand((g + 2,), generator=gen, device=dev, dtype=torch.float32)
    return dict(target_logits=tgt, draft_logits=drf, draft_tokens=tok, uniforms=uni,
                temperature=float(w.temperature))


def markov_models(V: int, dtype: str, seed: int, target_sigma: float = 2.0, draft_sigma: float = 1.0,
                  zipf: float = 0.0, device="cpu"):
    """Synthetic context-dependent models for the decoding loop: next-token logits depend on the last
    token only.  Returns (target_table, draft_table), each [V, V] in the storage dtype, row t = the
    logits after token t; the draft rows are the fp32 target rows plus iid Gaussian noise, drawn and
    rounded like the verification workloads above."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    t = torch.randn((V, V), generator=gen, device=dev, dtype=torch.float32) * target_sigma
    if zipf:
        perm = torch.rand((V, V), generator=gen, device=dev).argsort(dim=1)
        t = t - zipf * torch.log(torch.arange(1, V + 1, dtype=torch.float32, device=dev))[perm]
    d = t + torch.randn((V, V), generator=gen, device=dev, dtype=torch.float32) * draft_sigma
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    return t.to(td), d.to(td)


def top_p_mask(table: torch.Tensor, top_p: float, temperature: float = 1.0) -> torch.Tensor:
    """Nucleus masking of every row of a [V, V] table of logits: the tokens of a row are kept in
    order of decreasing probability under softmax(row / temperature) until their mass reaches
    ``top_p`` (the token that crosses it included), the others are set to -inf.  Same dtype."""
    z = table.float() / temperature
    order = z.argsort(dim=1, descending=True)
    prob = torch.softmax(z, dim=1).gather(1, order)
    before = prob.cumsum(dim=1) - prob                    # mass of the tokens ahead of each one
    drop_sorted = before >= top_p
    drop = torch.zeros_like(drop_sorted).scatter_(1, order, drop_sorted)
    return table.masked_fill(drop, float("-inf"))


def loop_uniforms(iterations: int, B: int, gamma: int, seed: int, device="cpu"):
    """The uniforms one run of the decoding loop consumes: u_draft [iterations, gamma, B] (one per
    drafted token) and u_verify [iterations, B, gamma+2] (the verification's), float32 in [0, 1)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    u_draft = torch.rand((iterations, gamma, B), generator=gen, device=dev, dtype=torch.float32)
    u_verify = torch.rand((iterations, B, gamma + 2), generator=gen, device=dev, dtype=torch.float32)
    return u_draft, u_verify
