"""The law of the number of accepted tokens through the library (GPU): the complementary CDF of tau
for the context-free two-token models of the paper's introduction with ten drafted tokens (the
figure that compares the two verifications), against the exact Pr(tau >= i) from the laws in
``oracle/exact.py``; and the low-temperature limit, where both verifications reduce to comparing
arg-max tokens and emit the same sequence."""
from fractions import Fraction as F

import numpy as np
import pytest
import torch

from oracle import exact
from helpers import all_blocks
from paper_2403_10444_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def exact_ccdf(P, Q, V, gamma, algo):
    """Pr(tau >= i), i = 0..gamma, over drafted blocks X^gamma ~ M_s^gamma and the algorithm's uniforms."""
    law = [F(0)] * (gamma + 1)
    for blk in all_blocks(V, gamma):
        if algo == "block":
            h = exact.block_quantities(P, Q, blk)[2]
            cond = exact.tau_law_block(h)
        else:
            cond = exact.tau_law_token(exact.token_quantities(P, Q, blk))
        w = exact.joint(Q, blk)
        for i in range(gamma + 1):
            law[i] += w * cond[i]
    return [float(sum(law[i:])) for i in range(gamma + 1)]


@pytest.mark.parametrize("entry", ["logits", "probs"])
def test_toy_ccdf_of_tau_with_ten_drafted_tokens(entry):
    import paper_2403_10444_b200 as bv
    gamma, V, N = 10, 8, 400_000           # (tokens 2..7 have probability zero: rows are whole vectors)
    P = lambda pre: [F(1, 3), F(2, 3)]
    Q = lambda pre: [F(2, 3), F(1, 3)]
    g = torch.Generator(device="cuda").manual_seed(10)
    p_row = torch.tensor([1 / 3, 2 / 3] + [0.0] * 6, device="cuda")
    q_row = torch.tensor([2 / 3, 1 / 3] + [0.0] * 6, device="cuda")
    tok = (torch.rand((N, gamma), generator=g, device="cuda") >= 2 / 3).to(torch.int32)     # X_i ~ M_s
    uni = torch.rand((N, gamma + 2), generator=g, device="cuda")
    tgt = p_row.expand(N, gamma + 1, V).contiguous()
    drf = q_row.expand(N, gamma, V).contiguous()
    if entry == "logits":
        tgt, drf = tgt.log(), drf.log()
        fns = {"block": lambda: bv.bv_verify(tgt, drf, tok, uni, 1.0), "token": lambda: bv.tv_verify(tgt, drf, tok, uni, 1.0)}
    else:
        fns = {"block": lambda: bv.bv_verify_probs(tgt, drf, tok, uni), "token": lambda: bv.tv_verify_probs(tgt, drf, tok, uni)}
    ccdf = {}
    for algo, fn in fns.items():
        out, out_len = fn()
        tau = (out_len - 1).cpu().numpy()
        assert tau.min() >= 0
        want = exact_ccdf(P, Q, 2, gamma, algo)
        got = [(tau >= i).mean() for i in range(gamma + 1)]
        for i in range(gamma + 1):
            se = np.sqrt(max(want[i] * (1 - want[i]), 1e-12) / N)
            assert abs(got[i] - want[i]) <= 4.5 * se + 1e-9, (algo, i, got[i], want[i])
        ccdf[algo] = got
        # generated tokens are a or b only
        o = out.cpu().numpy()
        assert o[o >= 0].max() <= 1
    # Block Verification accepts longer sub-blocks: its curve lies above Token Verification's
    assert all(ccdf["block"][i] >= ccdf["token"][i] - 1e-3 for i in range(gamma + 1))
    assert ccdf["block"][gamma] > ccdf["token"][gamma] * 1.5


def test_low_temperature_limit_both_verifications_emit_the_same_tokens():
    # T -> 0: softmax(z / T) tends to the arg-max token, every acceptance ratio to 0 or to at least 1,
    # p_i to 0 or 1, and the residual to the target's arg-max: Algorithms 1 and 2 both keep the drafted
    # tokens while they are the target's arg-max and then emit the target's arg-max
    import paper_2403_10444_b200 as bv
    w = wl.scaled(wl.CONFIGS["c3"], B=96, gamma=8, V=16384, draft_sigma=0.15)
    inp = wl.make_inputs(w, "cuda")
    T = 0.001
    tgt, drf = inp["target_logits"], inp["draft_logits"]
    tok = drf.float().argmax(-1).to(torch.int32)            # the draft model's samples in the limit
    top2 = tgt.float().topk(2, -1).values
    top2d = drf.float().topk(2, -1).values
    clear = ((top2[..., 0] - top2[..., 1]).min(1).values > 20 * T) & ((top2d[..., 0] - top2d[..., 1]).min(1).values > 20 * T)
    assert clear.sum() >= 32                                 # sequences without a near-tie at this temperature
    a = bv.bv_verify(tgt, drf, tok, inp["uniforms"], T)
    b = bv.tv_verify(tgt, drf, tok, inp["uniforms"], T)
    amax = tgt.float().argmax(-1).to(torch.int32)
    agree = (tok == amax[:, : w.gamma])
    n_acc = torch.where(agree.all(1), torch.full_like(agree[:, 0], w.gamma, dtype=torch.int64),
                        (~agree).to(torch.int64).argmax(1))
    idx = torch.nonzero(clear).flatten().cpu().tolist()
    for i in idx:
        k = int(n_acc[i])
        want = [int(x) for x in tok[i, :k]] + [int(amax[i, k])]
        assert int(a[1][i]) == k + 1 and int(b[1][i]) == k + 1, i
        assert [int(x) for x in a[0][i, : k + 1]] == want and [int(x) for x in b[0][i, : k + 1]] == want, i
    assert len({int(n_acc[i]) for i in idx}) >= 3            # several acceptance lengths occur
