"""A bounded device-side wait that really runs out: the kernel gives up by itself, reports
QBLORA_ERR_TIMEOUT through the workspace status word, and the library is usable afterwards."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import gate_strict, qweight_to_dev, to_bf16_dev, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("direction", ["fwd", "bwd"])
def test_a_wait_that_runs_out_sets_the_status_word_and_the_kernel_returns(direction):
    from paper_2407_17029_b200 import binding as qb
    # Two token tiles by two row tiles, eight K-blocks: the producers of every CTA leave out the copy of their
    # fourth K-block (the bytes are announced to the stage's barrier and never arrive).  With the wait limit set to
    # 2 * 10^6 cycles (about a millisecond) the MMA issuer, the dequant warps, the producers and the epilogue warps
    # each run into the limit, the pair frees its tensor memory and the kernel ends on its own: no trap, no fault,
    # no endless loop.  The call itself returns OK (the launch succeeded); the status word says what happened.
    T, d_out, d_in = 300, 512, 512
    W = synth.normal(81, "timeout/W", (d_out, d_in), 0.02)
    X = synth.round_to_bf16(synth.normal(81, "timeout/X", (T, d_in)))
    dY = synth.round_to_bf16(synth.normal(81, "timeout/dY", (T, d_out)))
    qw = oracle.quantize_blockwise(W, 64, 1, 0)
    dq, Xd, dYd = qweight_to_dev(qw), to_bf16_dev(X), to_bf16_dev(dY)
    op = qb.OP_LINEAR_FWD if direction == "fwd" else qb.OP_LINEAR_BWD
    ws = qb.alloc_workspace(op, dq, None, T)

    def call():
        if direction == "fwd":
            return qb.linear_fwd(dq, None, Xd, torch.float32, ws=ws)
        return qb.linear_bwd(dq, None, None, dYd, torch.float32, ws=ws)[0]

    good = call()
    assert qb.device_status(ws) == qb.OK
    try:
        qb.debug_set_wait_limit(2_000_000)
        qb.debug_drop_load(3)
        call()
        assert qb.device_status(ws) == qb.ERR_TIMEOUT          # synchronises: the kernel has returned
    finally:
        qb.debug_drop_load(-1)
        qb.debug_set_wait_limit(0)
    # the next ordinary call on the same workspace is clean and right
    again = call()
    assert qb.device_status(ws) == qb.OK
    assert torch.equal(again, good)
    Wt = oracle.dequantize(qw)
    ref = oracle.linear_fwd(Wt, None, X) if direction == "fwd" else oracle.linear_bwd(Wt, None, X, dY)[0]
    gate_strict(to_np64(again), ref, f"{direction} after a timed-out call")
