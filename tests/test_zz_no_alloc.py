"""The entry point that allocates nothing, checked against the ordinary one (GPU).

bv_verify_noalloc() is for programs that embed this library where a device allocation at
call time is not allowed: an inference server whose memory pool owns the whole GPU, code
that may be recording a stream capture, a process with allocator hooks.  It keeps its
scratch in a fixed 8 MiB array inside the library, shared by all calls, which holds
whatever the previous call left there.  So the test calls it twice in a row on different
inputs: a second call that trips over stale counters, or a first call that only works on
fresh memory, shows up as a difference from bv_verify().

This file sorts after the other test files on purpose: a run that stops at the first
failure has then already run everything else.  It also passes when run alone in a fresh
process, because it needs nothing the other tests set up.
"""
import ctypes

import pytest
import torch

import oracle
import paper_2403_10444_b200 as bv
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle, compare, assert_parity

pytestmark = pytest.mark.gpu


def _inputs(B, gamma, V, dtype, seed):
    w = wl.Workload("na", B, gamma, V, dtype, 1.0, seed, 2.0, 0.0, 0, 0.0, 1.0)
    return wl.make_inputs(w, "cuda")


def _call_noalloc(lib, inp, out_tokens, out_len):
    """Straight through the C ABI: raw pointers, caller-owned outputs, torch's current stream."""
    t, d, x, u = inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"]
    B, g1, V = t.shape
    code = 0 if t.dtype == torch.float32 else 1
    return lib.bv_verify_noalloc(t.data_ptr(), d.data_ptr(), x.data_ptr(), u.data_ptr(), B, g1 - 1, V, code,
                                 ctypes.c_float(inp["temperature"]), out_tokens.data_ptr(), out_len.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)


def _flow_kernel_with_default_shapes(bv_options):
    # the entry point without allocations always runs the flow kernel with the work-item shape chosen by
    # problem size: the call it is compared with must do the same, whatever the environment set
    bv_options("kernel", 1)
    for name in ("flow_chunks", "flow_pieces", "flow_ctas", "flow_depth", "flow_keep_l2", "flow_fine"):
        bv_options(name, 0)


def test_two_calls_in_a_row_match_the_allocating_entry_point(bv_options):
    _flow_kernel_with_default_shapes(bv_options)
    lib = bv.load_library()
    # the second problem is smaller and of another dtype, so leftovers of the first would matter
    cases = [_inputs(48, 6, 32768, "bf16", seed=101), _inputs(19, 3, 8192, "f32", seed=102)]
    outs = []
    for inp in cases:
        B, g1, _ = inp["target_logits"].shape
        ot = torch.full((B, g1), -7, dtype=torch.int32, device="cuda")
        ol = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        assert _call_noalloc(lib, inp, ot, ol) == 0
        outs.append((ot, ol))
    torch.cuda.synchronize()
    for inp, (ot, ol) in zip(cases, outs):
        want_tokens, want_len = bv.bv_verify(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"],
                                             inp["uniforms"], inp["temperature"])
        torch.cuda.synchronize()
        # same kernel, same chunking, deterministic sums: integer outputs agree bit for bit,
        # which is the tolerance the other GPU tests use for tau and the emitted token
        assert torch.equal(ol, want_len)
        assert torch.equal(ot, want_tokens)
        # and against the CPU oracle, by the rules of the other parity tests
        ref = run_oracle(oracle.BLOCK_VERIFY, inp)
        assert_parity(compare(oracle.BLOCK_VERIFY, ref, ot, ol, None, inp), False)


def test_problem_beyond_the_fixed_scratch_is_refused():
    lib = bv.load_library()
    # nothing is read before the size check, so small buffers stand in for the huge problem
    inp = _inputs(2, 2, 1024, "f32", seed=103)
    ot = torch.full((2, 3), -7, dtype=torch.int32, device="cuda")
    ol = torch.full((2,), -7, dtype=torch.int32, device="cuda")
    t = inp["target_logits"]
    rc = lib.bv_verify_noalloc(t.data_ptr(), inp["draft_logits"].data_ptr(), inp["draft_tokens"].data_ptr(),
                               inp["uniforms"].data_ptr(), 1 << 20, 8, 256000, 1, ctypes.c_float(1.0),
                               ot.data_ptr(), ol.data_ptr(), None)
    assert rc == -5
    assert "scratch" in bv.bv_status_string(rc)
    torch.cuda.synchronize()
    assert torch.all(ot == -7) and torch.all(ol == -7)      # nothing was launched
    # rows that are not whole 16-byte vectors are not served by this entry point
    rc = lib.bv_verify_noalloc(t.data_ptr(), inp["draft_logits"].data_ptr(), inp["draft_tokens"].data_ptr(),
                               inp["uniforms"].data_ptr(), 2, 2, 1022, 0, ctypes.c_float(1.0),
                               ot.data_ptr(), ol.data_ptr(), None)
    assert rc == -2


def test_the_largest_benchmark_workload_fits(bv_options):
    # B = 256, gamma = 8, V = 256000 needs 5 MB of the 8 MiB array
    _flow_kernel_with_default_shapes(bv_options)
    lib = bv.load_library()
    inp = wl.make_inputs(wl.CONFIGS["c4"], "cuda")
    B, g1, _ = inp["target_logits"].shape
    ot = torch.full((B, g1), -7, dtype=torch.int32, device="cuda")
    ol = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    assert _call_noalloc(lib, inp, ot, ol) == 0
    want_tokens, want_len = bv.bv_verify(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"],
                                         inp["uniforms"], inp["temperature"])
    torch.cuda.synchronize()
    assert torch.equal(ol, want_len) and torch.equal(ot, want_tokens)
