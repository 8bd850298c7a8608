"""Comparison of the CUDA path with the CPU oracle on the same bits (used by the GPU tests,
the smoke check and nothing else).

Tolerances, from the arithmetic of the CUDA path (fp32 per element, fp64 combination):
  - log-normalisers: 3e-6 absolute (they are returned as fp32 and are near 16, where one
    fp32 ulp is 1.9e-6);
  - p_i: 1e-5 relative; h_i: 1e-5 h_i + 1e-7 plus the largest change of h = S / (S + 1 - p) over the
    box that the S and p bounds span (h increases with both, so the corners give it exactly);
  - S_i: the bound is 1e-5 S_i + 2^-20 p_i + |error of p_i|, and 1e-5 relative literally where S_i is
    large enough for that to guarantee it.  Every term of S_i is a difference
    p_i P_i(x) - Q_i(x) = p_i A_x / Z_P - B_x / Z_Q of two ratios; each of the four ingredients carries
    the error of ex2.approx.ftz.f32, whose documented bound is 2^-22 relative (the normalisers as
    sums of such values), the terms that count have Q_i(x) <= p_i P_i(x), and the P_i(x) add up to
    at most one: 4 x 2^-22 p_i in the worst case (typical: 3e-8 p_i rms, unbiased; largest seen in
    the 60-cell sweep 1.7e-7 p_i, in random shapes with near-identical models about 3e-7 p_i).
    S_i is 1-Lipschitz in p_i, which carries the accumulated error of i ratios (bounded on its
    own), hence the last term, taken as measured.  Where the oracle has S_i = 0 the CUDA value must
    stay within the absolute part of the bound (and is exactly 0 when the two rows are
    bit-identical); the largest value seen there is part of the report;
  - Greedy Block Verification (Algorithm 4): the same bounds with the unclipped product in place
    of p_i; where that product is one or more the acceptance ratio is only required to be >= 1;
  - tau and Y: bit-exact, except for trials in which a uniform lies within 1e-6 of
    the threshold it is compared with: a differing tau needs an eta_i within 1e-6 of
    h_i (oracle margin); a differing Y needs the sampling uniform within 1e-6 of the
    CDF cell of the CUDA token (recomputed here in fp64).  Both are counted.  Differing taus
    must stay within 1e-4 of the trials (rounded up).  For Y the bound is
    trials (1e-4 + 2e-8 V): the kernels form every sum that decides a token in double, but each
    weight is an ex2.approx.ftz.f32 value with up to 2^-22 relative error, which displaces the
    CDF by a few 1e-9, and a uniform that close to one of the V cell edges changes cell: about
    1e-8 V of all trials (measured over the sweep at V = 152064: 3 of 2500 distinct trials).

Every report can be appended, as one JSON line, to the file named by BV_PARITY_LOG.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, asdict

import numpy as np
import torch

import oracle

NEAR = 1e-6
S_FLOOR = 2.0 ** -20      # four times the error bound of ex2.approx.ftz.f32 (see above): what S_i / p_i cannot be trusted below


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
          (oracle.BLOCK_VERIFY, False): bv.bv_verify, (oracle.TOKEN_VERIFY, False): bv.tv_verify,
          (oracle.GREEDY_BLOCK_VERIFY, True): bv.gbv_verify_ex,
          (oracle.GREEDY_BLOCK_VERIFY, False): bv.gbv_verify}[(algo, diagnostics)]
    out = fn(d["target_logits"], d["draft_logits"], d["draft_tokens"], d["uniforms"], d["temperature"])
    torch.cuda.synchronize()
    return out


@dataclass
class ParityReport:
    trials: int
    near_threshold: int        # trials with some deciding uniform within 1e-6 of its threshold
    mismatches: int            # tau or Y differs (all of them, excused or not)
    excused_tau: int           # tau differs and an eta_i was within 1e-6 of h_i
    excused_Y: int             # same tau, Y differs, and u is within 1e-6 of the CUDA token's CDF cell
    hard_mismatches: int       # differs with no such excuse
    max_rel_S: float
    max_rel_S_conditioned: float  # over positions with S >= 2.4e-2 p
    S_floor_violations: int
    max_h_err_over_tol: float
    max_rel_p: float
    max_abs_lse: float
    vocab: int = 0
    max_S_at_zero: float = 0.0   # largest CUDA S_i / p_i where the oracle's S_i is exactly 0

    def __str__(self):
        return ("trials=%d near=%d mismatch=%d excused_tau=%d excused_Y=%d hard=%d relS=%.2e "
                "relS(where 1e-5 is guaranteed)=%.2e floorviol=%d h_err/tol=%.2f relp=%.2e abslse=%.2e" % (
                    self.trials, self.near_threshold, self.mismatches, self.excused_tau,
                    self.excused_Y, self.hard_mismatches, self.max_rel_S,
                    self.max_rel_S_conditioned, self.S_floor_violations,
                    self.max_h_err_over_tol, self.max_rel_p, self.max_abs_lse))


def _widen(row: np.ndarray) -> np.ndarray:
    if row.dtype == np.uint16:
        return (row.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return row.astype(np.float64)


def token_is_valid(algo, ref, inp_np, b, y, probs=False) -> bool:
    """Is token y within 1e-6 (in probability) of the CDF cell the sampling uniform falls in,
    under the oracle's normalisers and p for sequence b?  (fp64, index order.)  ``probs``: the
    rows hold probabilities, used as stored."""
    tgt, drf, uni, T = inp_np
    g = drf.shape[1]
    tau = int(ref.out_len[b]) - 1
    T = float(np.float32(T))
    P = _widen(tgt[b, tau]) if probs else np.exp(_widen(tgt[b, tau]) / T - ref.lse_t[b, tau])
    if tau < g:
        p = ref.p[b, tau] if algo != oracle.TOKEN_VERIFY else 1.0   # (the unclipped product for Algorithm 4)
        Q = _widen(drf[b, tau]) if probs else np.exp(_widen(drf[b, tau]) / T - ref.lse_d[b, tau])
        w = np.maximum(p * P - Q, 0.0)
        if not w.sum() > 0:
            w = P
        u = float(uni[b, g])
    else:
        w, u = P, float(uni[b, g + 1])
    if y < 0 or y >= w.shape[0] or not w[y] > 0:
        return False
    C = np.cumsum(w)
    lo = (C[y] - w[y]) / C[-1]
    hi = C[y] / C[-1]
    return lo - NEAR <= u <= hi + NEAR


def compare(algo: int, ref: "oracle.OracleResult", out_tokens, out_len, diag=None, inp=None, probs=False) -> ParityReport:
    ot = out_tokens.cpu().numpy()
    ol = out_len.cpu().numpy()
    B = ol.shape[0]
    same = (ol == ref.out_len) & np.all(ot == ref.out_tokens, axis=1)
    ok_rows = ref.out_len >= 0
    near = ok_rows & ((ref.margin_eta < NEAR) | (ref.margin_smp < NEAR))
    mism = ~same
    excused_tau = excused_Y = hard = 0
    inp_np = None
    for b in np.nonzero(mism)[0]:
        if not ok_rows[b] or ol[b] < 0:
            hard += 1
        elif ol[b] != ref.out_len[b]:
            if ref.margin_eta[b] < NEAR:
                excused_tau += 1
            else:
                hard += 1
        else:
            tau = int(ol[b]) - 1
            prefix_same = np.array_equal(ot[b, :tau], ref.out_tokens[b, :tau]) and np.all(ot[b, tau + 1:] == -1)
            if inp is not None and inp_np is None:
                inp_np = (to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                          inp["uniforms"].cpu().numpy(), inp["temperature"])
            if prefix_same and inp_np is not None and token_is_valid(algo, ref, inp_np, b, int(ot[b, tau]), probs):
                excused_Y += 1
            else:
                hard += 1
    rel_S = rel_Sc = h_over = rel_p = abs_lse = S_at_zero = 0.0
    floor_viol = 0
    V = 0
    if diag is not None:
        S = diag["S"].cpu().numpy().astype(np.float64)
        h = diag["h"].cpu().numpy().astype(np.float64)
        p = diag["p"].cpu().numpy().astype(np.float64)
        rows = ok_rows
        # (the entry points on probabilities form no normalisers)
        pairs = [] if "lse_t" not in diag else [(diag["lse_t"].cpu().numpy().astype(np.float64), ref.lse_t),
                                                (diag["lse_d"].cpu().numpy().astype(np.float64), ref.lse_d)]
        for got, want in pairs:
            m = rows[:, None] & ~np.isnan(want)
            assert not np.isnan(got[m]).any(), "CUDA path left a log-normaliser unset"
            if m.any():
                abs_lse = max(abs_lse, float(np.abs(got[m] - want[m]).max()))
        if algo != oracle.TOKEN_VERIFY:
            m = rows[:, None] & ~np.isnan(ref.p)
            rel_p = float((np.abs(p[m] - ref.p[m]) / np.maximum(ref.p[m], 1e-30)).max())
            pS = ref.p[:, :-1]
            # h_i = S_i / (S_i + 1 - p_i), 1 <= i < gamma: propagate the S and p tolerances.
            # Positions with S_i = 0 are skipped: there h_i := 0 by convention and decides nothing.
            g = ref.S.shape[1]
            for i in range(1, g):
                Sr, pr, hr = ref.S[:, i], ref.p[:, i], ref.h[:, i]
                mm = rows & (Sr > 0)
                if algo == oracle.GREEDY_BLOCK_VERIFY:
                    # Algorithm 4's ratio with an unclipped product of one or more is at least one:
                    # the test passes whatever the uniform, and that is all the value says
                    sure = mm & (pr >= 1.0)
                    assert np.all(h[sure, i] >= 1.0), "a position with pt_i >= 1 must pass its test"
                    mm = mm & (pr < 1.0)
                if mm.any():
                    # h increases with S and with p: its largest deviation over the box |dS| <= eS, |dp| <= ep is at
                    # the corners (exact, where a first-order estimate breaks down as S + 1 - p gets small).
                    # ep: the error of p_i as measured (the diagnostic is a float: plus half an ulp);
                    # eS: the bound asserted for S_i below
                    ep = np.abs(p[mm, i] - pr[mm]) + 2.0 ** -24 * pr[mm]
                    eS = 1e-5 * Sr[mm] + S_FLOOR * pr[mm] + ep
                    one_p = 1.0 - pr[mm] if algo != oracle.GREEDY_BLOCK_VERIFY else np.maximum(1.0 - pr[mm], 0.0)
                    hi = (Sr[mm] + eS) / (Sr[mm] + eS + np.maximum(one_p - ep, 0.0))
                    lo_S = np.maximum(Sr[mm] - eS, 0.0)
                    lo = lo_S / np.maximum(lo_S + one_p + ep, 1e-300)
                    tol = np.maximum(hi - hr[mm], hr[mm] - lo) + 1e-5 * hr[mm] + 1e-7
                    h_over = max(h_over, float((np.abs(h[mm, i] - hr[mm]) / tol).max()))
            mm = rows
            if mm.any():
                tol = 1e-5 * ref.h[mm, g] + 1e-7
                h_over = max(h_over, float((np.abs(h[mm, g] - ref.h[mm, g]) / tol).max()))
        else:
            pS = np.ones_like(ref.S)
            m = rows[:, None] & ~np.isnan(ref.h)
            assert not np.isnan(h[m]).any()
            if m.any():
                h_over = float((np.abs(h[m] - ref.h[m]) / (1e-5 * ref.h[m] + 1e-7)).max())
        m = rows[:, None] & ~np.isnan(ref.S)
        assert not np.isnan(S[m]).any()
        # S_i is 1-Lipschitz in p_i (dS/dp = sum of P_i(x) over the tokens with a positive term <= 1), and p_i
        # carries the accumulated error of i ratios (bounded on its own, 1e-5 relative): the absolute part of
        # the S bound is the exponentials' floor plus the error of p_i as measured
        dp = np.abs(p[:, :-1] - ref.p[:, :-1]) if algo != oracle.TOKEN_VERIFY else np.zeros_like(ref.S)
        dp = np.where(np.isnan(dp), 0.0, dp)
        zero = m & (ref.S == 0)
        # an exactly empty residual: the CUDA value may differ from 0 only by the rounding
        # floor (it is exactly 0 for bit-identical rows, see test_draft_equals_target)
        assert np.all(S[zero] <= S_FLOOR * pS[zero] + dp[zero]), "CUDA S must vanish where the oracle's does"
        S_at_zero = float((S[zero] / np.maximum(pS[zero], 1e-300)).max()) if zero.any() else 0.0
        pos = m & (ref.S > 0)
        if pos.any():
            err = np.abs(S[pos] - ref.S[pos])
            rel = err / ref.S[pos]
            rel_S = float(rel.max())
            cond = ref.S[pos] >= (S_FLOOR * pS[pos] + dp[pos]) / 1e-5
            if cond.any():
                rel_Sc = float(rel[cond].max())
            floor_viol = int((err > 1e-5 * ref.S[pos] + S_FLOOR * pS[pos] + dp[pos]).sum())
    if inp is not None:
        V = int(inp["target_logits"].shape[-1])
    return ParityReport(B, int(near.sum()), int(mism.sum()), excused_tau, excused_Y, hard, rel_S,
                        rel_Sc, floor_viol, h_over, rel_p, abs_lse, V, S_at_zero)


def assert_parity(rep: ParityReport, check_diag=True):
    assert rep.hard_mismatches == 0, str(rep)
    # an eta within 1e-6 of h_i: at most 1e-4 of trials may differ for that reason
    assert rep.excused_tau <= int(np.ceil(1e-4 * rep.trials)), str(rep)
    # a sampling uniform within 1e-6 of an edge of the emitted token's CDF cell: the share of such
    # trials that the exponentials' own error can move across an edge grows with the number of edges
    assert rep.excused_Y <= int(np.ceil(rep.trials * (1e-4 + 2e-8 * rep.vocab))), str(rep)
    if check_diag:
        assert rep.max_abs_lse <= 3e-6, str(rep)
        assert rep.max_rel_p <= 1e-5, str(rep)
        assert rep.max_h_err_over_tol <= 1.0, str(rep)
        assert rep.max_rel_S_conditioned <= 1e-5, str(rep)
        assert rep.S_floor_violations == 0, str(rep)


def record(rep: ParityReport, label: str):
    """Appends the report to the file named by BV_PARITY_LOG (one JSON line), if that is set."""
    path = os.environ.get("BV_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(dict(case=label, **asdict(rep))) + "\n")
