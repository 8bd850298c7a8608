"""The drafting step (bv_sample_draft) through the C-ABI against the CPU oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle
from parity import to_numpy_logits

pytestmark = pytest.mark.gpu

NEAR = 1e-6


def check(logits, uniforms, T):
    import paper_2403_10444_b200 as bv
    want_tok, want_lse, margin = oracle.sample_rows(to_numpy_logits(logits), uniforms.numpy(), T)
    tok, lse = bv.bv_sample_draft(logits.cuda(), uniforms.cuda(), T)
    torch.cuda.synchronize()
    tok, lse = tok.cpu().numpy(), lse.cpu().numpy().astype(np.float64)
    rows, V = logits.shape
    bad = want_tok < 0
    assert np.array_equal(tok[bad], want_tok[bad]) and np.isnan(lse[bad]).all()
    ok = ~bad
    assert np.abs(lse[ok] - want_lse[ok]).max(initial=0.0) <= 3e-6
    diff = ok & (tok != want_tok)
    # a differing token is excused only if the uniform lies within 1e-6 (in probability) of the
    # edge of its CDF cell, and such cases must stay within 1e-4 + 2e-8 V of the rows (see parity.py)
    assert not (diff & ~(margin < NEAR)).any(), "token differs away from any threshold"
    assert diff.sum() <= int(np.ceil(rows * (1e-4 + 2e-8 * V)))
    # and the CUDA token must then be the neighbour cell with positive weight
    for r in np.nonzero(diff)[0]:
        z = to_numpy_logits(logits)[r]
        z = (z.astype(np.uint32) << 16).view(np.float32) if z.dtype == np.uint16 else z
        w = np.exp(z.astype(np.float64) / np.float32(T) - want_lse[r])
        C = np.cumsum(w)
        lo, hi = (C[tok[r]] - w[tok[r]]) / C[-1], C[tok[r]] / C[-1]
        assert w[tok[r]] > 0 and lo - NEAR <= float(uniforms[r]) <= hi + NEAR
    return int(diff.sum())


@pytest.mark.parametrize("rows,V,dtype,T", [(64, 256000, "bf16", 1.0), (300, 32000, "f32", 0.8),
                                            (40, 152064, "bf16", 0.8), (33, 8, "f32", 1.0),
                                            (500, 1024, "bf16", 2.5), (7, 4104, "f32", 0.3),
                                            (5, 1 << 21, "f32", 1.0), (3, (1 << 21) + 8, "bf16", 0.7)])
def test_sampler_matches_the_oracle(rows, V, dtype, T):
    g = torch.Generator().manual_seed(rows + V)
    z = torch.randn((rows, V), generator=g) * 3.0
    z = z - 1.1 * torch.log(torch.rand((rows, V), generator=g).argsort(dim=1).float() + 1.0)
    logits = z.bfloat16() if dtype == "bf16" else z
    u = torch.rand((rows,), generator=g)
    check(logits, u, T)


def test_sampler_frequencies_on_a_tiny_vocabulary():
    # 200000 uniforms on one row of 8 logits: the token frequencies are the softmax
    import paper_2403_10444_b200 as bv
    from scipy import stats
    z = torch.tensor([0.3, -1.0, 2.0, float("-inf"), 0.0, 1.5, -0.5, 0.7])
    n = 200_000
    u = torch.rand((n,), generator=torch.Generator().manual_seed(1))
    tok, _ = bv.bv_sample_draft(z.repeat(n, 1).cuda(), u.cuda(), 0.9)
    cnt = np.bincount(tok.cpu().numpy(), minlength=8).astype(np.float64)
    p = torch.softmax(z.double() / 0.9, 0).numpy()
    assert cnt[3] == 0
    keep = p > 0
    chi = ((cnt[keep] - n * p[keep]) ** 2 / (n * p[keep])).sum()
    assert chi < stats.chi2.isf(1e-6, keep.sum() - 1)


def test_sampler_domain_errors_and_refusals():
    import paper_2403_10444_b200 as bv
    z = torch.zeros((4, 16))
    z[0, 5] = float("nan")
    z[1, :] = float("-inf")
    z[2, 7] = float("inf")
    u = torch.full((4,), 0.5)
    tok, lse = bv.bv_sample_draft(z.cuda(), u.cuda(), 1.0)
    tok, lse = tok.cpu(), lse.cpu()
    assert tok[:3].tolist() == [-1, -1, -1] and torch.isnan(lse[:3]).all()
    assert tok[3].item() == 8 and abs(lse[3].item() - np.log(16)) < 1e-6
    with pytest.raises(bv.BVError):            # rows that are not whole 16-byte vectors
        bv.bv_sample_draft(torch.zeros((2, 5)).cuda(), u[:2].cuda(), 1.0)
    with pytest.raises(bv.BVError):
        bv.bv_sample_draft(z.cuda(), u.cuda(), 0.0)
