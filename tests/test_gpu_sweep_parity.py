"""GPU parity over the whole sweep: every cell of B x gamma x draft noise at V = 152064, both
algorithms, against the CPU oracle on the same bits.

The CUDA calls run on the full cell, in the launch shape the benchmark and the sweep time; the
oracle checks every sequence of cells with B <= 64 and the first 64 sequences of larger ones.  Per
cell the rules of parity.assert_parity apply; over all cells the trials whose tau differs with an
excuse (a uniform within 1e-6 of its threshold) must stay within 1e-4 of all trials, those whose
token differs within 1e-4 + 2e-8 V of them (see parity.py).
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle, run_cuda, compare, assert_parity, record

pytestmark = pytest.mark.gpu

CHECKED = 64
TOTALS = {"trials": 0, "excused_tau": 0, "excused_Y": 0, "near": 0, "cells": 0}


def _head(inp, n):
    return {k: (v[:n] if torch.is_tensor(v) else v) for k, v in inp.items()}


@pytest.mark.parametrize("B", wl.SWEEP_B)
@pytest.mark.parametrize("gamma", wl.SWEEP_GAMMA)
def test_sweep_cells_match_the_oracle(B, gamma):
    for sigma in wl.SWEEP_SIGMA:
        inp = wl.make_inputs(wl.sweep_cell(B, gamma, sigma), "cuda")
        n = min(B, CHECKED)
        head = _head(inp, n)
        for algo in (oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY):
            ref = run_oracle(algo, head)
            ot, ol, diag = run_cuda(algo, inp)                      # every position, with diagnostics
            rep = compare(algo, ref, ot[:n], ol[:n], {k: v[:n] for k, v in diag.items()}, head)
            ot2, ol2 = run_cuda(algo, inp, diagnostics=False)[:2]   # the call a server makes
            rep2 = compare(algo, ref, ot2[:n], ol2[:n], None, head)
            for r, kind in ((rep, "diagnostics"), (rep2, "plain")):
                label = "c5 B=%d gamma=%d sigma=%g %s %s" % (B, gamma, sigma, "block" if algo == oracle.BLOCK_VERIFY else "token", kind)
                record(r, label)
                assert_parity(r, kind == "diagnostics")
                TOTALS["trials"] += r.trials
                TOTALS["excused_tau"] += r.excused_tau
                TOTALS["excused_Y"] += r.excused_Y
                TOTALS["near"] += r.near_threshold
            TOTALS["cells"] += 1
        del inp, head
        torch.cuda.empty_cache()


def test_sweep_totals():
    # runs after the cells (same module, file order): the excuses of all of them together
    if TOTALS["cells"] == 0:
        pytest.skip("the cells did not run in this process")
    print("sweep parity: %(cells)d cell x algorithm cases, %(trials)d trials, %(near)d near a threshold, "
          "%(excused_tau)d taus and %(excused_Y)d tokens differing with an excuse" % TOTALS)
    assert TOTALS["excused_tau"] <= 1e-4 * TOTALS["trials"], TOTALS
    assert TOTALS["excused_Y"] <= (1e-4 + 2e-8 * 152064) * TOTALS["trials"], TOTALS
