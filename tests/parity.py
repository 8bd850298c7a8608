"""Comparison of the CUDA path with the CPU oracle on the same bits (used by the GPU tests,
the smoke check and nothing else).

Tolerances, from the arithmetic of the CUDA path (fp32 per element, fp64 combination):
  - log-normalisers: 3e-6 absolute (they are returned as fp32 and are near 16, where one
    fp32 ulp is 1.9e-6);
  - p_i: 1e-5 relative; h_i: 1e-5 h_i + 1e-7 (h_i inherits the conditioning of S_i);
  - S_i: 1e-5 relative literally where S_i >= 1e-2 p_i; below that the bound is
    1e-5 S_i + 1e-7 p_i, because S is then the small difference of sums whose own
    fp32 rounding is 6e-8 p_i; where the oracle has S_i = 0 the CUDA value must be 0;
  - tau and Y: bit-exact, except for trials in which a uniform lies within 1e-6 of
    the threshold it is compared with (oracle margins); those are counted.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import oracle

NEAR = 1e-6


def to_numpy_logits(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def run_oracle(algo: int, inp) -> "oracle.OracleResult":
    return oracle.verify(algo, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                         inp["draft_tokens"].cpu().numpy(), inp["uniforms"].cpu().numpy(),
                         inp["temperature"])


def to_device(inp, dev="cuda"):
    return {k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in inp.items()}


def run_cuda(algo: int, inp, diagnostics=True):
    import paper_2403_10444_b200 as bv
    d = to_device(inp)
    fn = {(oracle.BLOCK_VERIFY, True): bv.bv_verify_ex, (oracle.TOKEN_VERIFY, True): bv.tv_verify_ex,
          (oracle.BLOCK_VERIFY, False): bv.bv_verify, (oracle.TOKEN_VERIFY, False): bv.tv_verify}[(algo, diagnostics)]
    out = fn(d["target_logits"], d["draft_logits"], d["draft_tokens"], d["uniforms"], d["temperature"])
    torch.cuda.synchronize()
    return out


@dataclass
class ParityReport:
    trials: int
    near_threshold: int
    mismatches: int            # tau or Y differs (all of them, near-threshold or not)
    hard_mismatches: int       # differs although no uniform was near its threshold
    max_rel_S: float
    max_rel_S_conditioned: float  # over positions with S >= 1e-2 p
    S_floor_violations: int
    max_rel_h: float
    max_rel_p: float
    max_abs_lse: float

    def __str__(self):
        return ("trials=%d near=%d mismatch=%d hard=%d relS=%.2e relS(S>=.01p)=%.2e floorviol=%d "
                "relh=%.2e relp=%.2e abslse=%.2e" % (
                    self.trials, self.near_threshold, self.mismatches, self.hard_mismatches,
                    self.max_rel_S, self.max_rel_S_conditioned, self.S_floor_violations,
                    self.max_rel_h, self.max_rel_p, self.max_abs_lse))


def compare(algo: int, ref: "oracle.OracleResult", out_tokens, out_len, diag=None) -> ParityReport:
    ot = out_tokens.cpu().numpy()
    ol = out_len.cpu().numpy()
    B = ol.shape[0]
    same = (ol == ref.out_len) & np.all(ot == ref.out_tokens, axis=1)
    ok_rows = ref.out_len >= 0
    near = ok_rows & ((ref.margin_eta < NEAR) | (ref.margin_smp < NEAR))
    mism = ~same
    hard = mism & ~near
    rel_S = rel_Sc = rel_h = rel_p = abs_lse = 0.0
    floor_viol = 0
    if diag is not None:
        S = diag["S"].cpu().numpy().astype(np.float64)
        h = diag["h"].cpu().numpy().astype(np.float64)
        p = diag["p"].cpu().numpy().astype(np.float64)
        lt = diag["lse_t"].cpu().numpy().astype(np.float64)
        ld = diag["lse_d"].cpu().numpy().astype(np.float64)
        rows = ok_rows
        for got, want in ((lt, ref.lse_t), (ld, ref.lse_d)):
            m = rows[:, None] & ~np.isnan(want)
            assert not np.isnan(got[m]).any(), "CUDA path left a log-normaliser unset"
            if m.any():
                abs_lse = max(abs_lse, float(np.abs(got[m] - want[m]).max()))
        m = rows[:, None] & ~np.isnan(ref.h)
        assert not np.isnan(h[m]).any()
        if m.any():
            rel_h = float((np.abs(h[m] - ref.h[m]) / (np.abs(ref.h[m]) + 1e-2)).max())
        if algo == oracle.BLOCK_VERIFY:
            m = rows[:, None] & ~np.isnan(ref.p)
            rel_p = float((np.abs(p[m] - ref.p[m]) / np.maximum(ref.p[m], 1e-30)).max())
            pS = ref.p[:, :-1]
        else:
            pS = np.ones_like(ref.S)
        m = rows[:, None] & ~np.isnan(ref.S)
        assert not np.isnan(S[m]).any()
        zero = m & (ref.S == 0)
        assert np.all(S[zero] == 0), "CUDA S must be exactly 0 where the oracle's is"
        pos = m & (ref.S > 0)
        if pos.any():
            err = np.abs(S[pos] - ref.S[pos])
            rel = err / ref.S[pos]
            rel_S = float(rel.max())
            cond = ref.S[pos] >= 1e-2 * pS[pos]
            if cond.any():
                rel_Sc = float(rel[cond].max())
            floor_viol = int((err > 1e-5 * ref.S[pos] + 1e-7 * pS[pos]).sum())
    return ParityReport(B, int(near.sum()), int(mism.sum()), int(hard.sum()), rel_S, rel_Sc,
                        floor_viol, rel_h, rel_p, abs_lse)


def assert_parity(rep: ParityReport, check_diag=True):
    assert rep.hard_mismatches == 0, str(rep)
    assert rep.near_threshold <= max(1, int(np.ceil(1e-4 * rep.trials))), str(rep)
    if check_diag:
        assert rep.max_abs_lse <= 3e-6, str(rep)
        assert rep.max_rel_p <= 1e-5, str(rep)
        assert rep.max_rel_h <= 1e-5, str(rep)
        assert rep.max_rel_S_conditioned <= 1e-5, str(rep)
        assert rep.S_floor_violations == 0, str(rep)
