"""Randomly drawn shapes through every kernel that admits them, all three algorithms, with and without
diagnostics, against the oracle by the rules of tests/parity.py (GPU).  The draws are seeded: the same
cases every run.  (A ten-minute run of the same loop over 58 000 calls found no disagreement and no
wait that ran out.)"""
import random

import pytest

import oracle
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle, run_cuda, compare, assert_parity, record

pytestmark = pytest.mark.gpu

KERNELS = {"default": 0, "flow": 1, "small": 4}


def draw(rnd):
    while True:
        B = rnd.choice([1, 2, 3, 5, 8, 13, 16, 17, 31, 32, 33, 40, 64, 100, 257, 400])
        g = rnd.choice([1, 2, 3, 4, 5, 8, 11, 16, 20])
        V = rnd.choice([8, 16, 24, 64, 1000, 1024, 4096, 4104, 10000, 32000, 50304])
        dtype = rnd.choice(["f32", "bf16"])
        if B * (2 * g + 1) * V > 1.5e8 or (dtype == "bf16" and V % 8):
            continue
        return wl.Workload("rs", B, g, V, dtype, rnd.choice([0.5, 0.8, 1.0, 1.7]), rnd.randrange(1 << 30), 2.0,
                           rnd.choice([0.0, 1.1]), 0, 0.0, rnd.choice([0.05, 0.3, 1.0, 2.5]))


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes(seed, bv_options):
    import paper_2403_10444_b200 as bv
    rnd = random.Random(1000 + seed)
    for _ in range(8):
        w = draw(rnd)
        inp = wl.make_inputs(w, "cpu")
        fits_small = w.B <= 32 and w.B * (2 * w.gamma + 1) <= 1056 and w.B * (w.gamma + 1) <= 560
        for algo in (oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY, oracle.GREEDY_BLOCK_VERIFY):
            ref = run_oracle(algo, inp)
            for name, code in KERNELS.items():
                if name == "small" and not fits_small:
                    continue
                bv_options("kernel", code)
                for diag in (True, False):
                    out = run_cuda(algo, inp, diagnostics=diag)
                    rep = compare(algo, ref, out[0], out[1], out[2] if diag else None, inp)
                    record(rep, "random shape B=%d gamma=%d V=%d %s T=%g sigma=%g algo %d kernel %s %s" % (
                        w.B, w.gamma, w.V, w.dtype, w.temperature, w.draft_sigma, algo, name, "diagnostics" if diag else "plain"))
                    assert_parity(rep, diag), (w, algo, name, diag)
                    assert bv.bv_stream_status() == 0


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_other_entry_points(seed, bv_options):
    """The entry points on probabilities, with supplied draft normalisers, and the drafting step."""
    import numpy as np
    import torch
    import paper_2403_10444_b200 as bv
    from parity import to_numpy_logits
    rnd = random.Random(2000 + seed)
    for _ in range(6):
        w = draw(rnd)
        inp = wl.make_inputs(w, "cpu")
        T, g, V = w.temperature, w.gamma, w.V
        fits_small = w.B <= 32 and w.B * (2 * g + 1) <= 1056 and w.B * (g + 1) <= 560
        kernels = [c for n, c in KERNELS.items() if n != "small" or fits_small]
        pin = dict(inp)
        for k in ("target_logits", "draft_logits"):
            pin[k] = torch.softmax(inp[k].double() / T, -1).to(inp[k].dtype).contiguous()
        a = tuple(pin[k].cuda() for k in ("target_logits", "draft_logits", "draft_tokens", "uniforms"))
        for algo, fn in ((oracle.BLOCK_VERIFY, bv.bv_verify_probs), (oracle.TOKEN_VERIFY, bv.tv_verify_probs)):
            ref = oracle.verify_probs(algo, to_numpy_logits(pin["target_logits"]), to_numpy_logits(pin["draft_logits"]),
                                      pin["draft_tokens"].numpy(), pin["uniforms"].numpy())
            for code in kernels:
                bv_options("kernel", code)
                for diag in (True, False):
                    out = fn(*a, diagnostics=diag)
                    assert_parity(compare(algo, ref, out[0], out[1], out[2] if diag else None, pin, probs=True), diag)
        lse = torch.logsumexp(inp["draft_logits"].double() / np.float32(T), -1).float()
        d = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
        for algo, fn in ((oracle.BLOCK_VERIFY, bv.bv_verify_lse), (oracle.TOKEN_VERIFY, bv.tv_verify_lse)):
            ref = oracle.verify(algo, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                                inp["draft_tokens"].numpy(), inp["uniforms"].numpy(), T, draft_lse=lse.numpy())
            for code in kernels:
                bv_options("kernel", code)
                for diag in (True, False):
                    out = fn(d["target_logits"], d["draft_logits"], d["draft_tokens"], d["uniforms"], lse.cuda(), T,
                             diagnostics=diag)
                    assert_parity(compare(algo, ref, out[0], out[1], out[2] if diag else None, inp), diag)
        assert bv.bv_stream_status() == 0
        rows = inp["draft_logits"].reshape(-1, V).contiguous()
        u = inp["uniforms"][:, :g].reshape(-1).contiguous()
        want_tok, want_lse, margin = oracle.sample_rows(to_numpy_logits(rows), u.numpy(), T)
        tok, l = bv.bv_sample_draft(rows.cuda(), u.cuda(), T)
        tok, l = tok.cpu().numpy(), l.cpu().numpy().astype(np.float64)
        assert not ((tok != want_tok) & ~(margin < 1e-6)).any()
        assert np.abs(l - want_lse).max() <= 3e-6
