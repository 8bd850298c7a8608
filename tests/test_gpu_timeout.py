"""A bounded device-side wait that runs out ends the call with BV_ERR_TIMEOUT and harms nothing (GPU).

Every wait inside the kernels has a limit; when one gives up, the kernel records it and returns.
The failure is made on purpose here without faulting or hanging anything: the library's test
option "never_signal" makes the flow kernel's worker warps stop reporting their items as swept,
and "wait_limit" shortens the limits to a few thousand polls, on a grid of two CTAs and a tiny
problem.  The waits of the other warps then run out within a fraction of a millisecond."""
import numpy as np
import pytest
import torch

import oracle
import paper_2403_10444_b200 as bv
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle

pytestmark = pytest.mark.gpu


def _tiny(seed):
    return wl.make_inputs(wl.Workload("to", 3, 2, 4096, "bf16", 1.0, seed, 2.0, 0.0, 0, 0.0, 1.0), "cpu")


@pytest.mark.parametrize("kernel", [1, 4])      # the flow kernel; the small-batch kernel (a CTA stays away from its grid barrier)
def test_wait_that_runs_out_is_reported_and_the_next_call_works(kernel, bv_options):
    inp = _tiny(5)
    bv_options("kernel", kernel)
    pinned = {k: (v.pin_memory() if torch.is_tensor(v) else v) for k, v in inp.items()}
    dev = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
    args = lambda d: (d["target_logits"], d["draft_logits"], d["draft_tokens"], d["uniforms"], d["temperature"])
    bv.bv_verify(*args(dev))                       # workspace set-up with everything in order
    assert bv.bv_stream_status() == 0

    bv_options("flow_ctas", 2)
    bv_options("wait_limit", 2000)
    bv_options("never_signal", 1)
    # host-buffer entry point: synchronises, so it reports the failure itself
    with pytest.raises(bv.BVError) as err:
        bv.bv_verify_host(*args(pinned))
    assert err.value.status == -4
    # device entry point: returns at once; the stream's status tells
    bv.bv_verify(*args(dev))
    assert bv.bv_stream_status() == -4
    assert bv.bv_stream_status() == 0              # the report clears the record

    bv_options("never_signal", 0)
    bv_options("wait_limit", 0)
    bv_options("flow_ctas", 0)
    ref = run_oracle(oracle.BLOCK_VERIFY, inp)
    ot, ol = bv.bv_verify_host(*args(pinned))
    assert np.array_equal(ol.numpy(), ref.out_len) and np.array_equal(ot.numpy(), ref.out_tokens)
    ot, ol = bv.bv_verify(*args(dev))
    assert bv.bv_stream_status() == 0
    assert np.array_equal(ol.cpu().numpy(), ref.out_len) and np.array_equal(ot.cpu().numpy(), ref.out_tokens)
