"""A bounded device-side wait that really runs out: the kernel gives up by itself, reports
QBLORA_ERR_TIMEOUT through the workspace status word, and the library is usable afterwards."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import gate_strict, qweight_to_dev, to_bf16_dev, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("direction,T,d_out,d_in", [("fwd", 300, 512, 512), ("bwd", 300, 512, 512),
                                                    ("fwd", 2100, 4864, 256), ("bwd", 2100, 256, 4864)])
def test_a_wait_that_runs_out_sets_the_status_word_and_the_kernel_returns(direction, T, d_out, d_in):
    from paper_2407_17029_b200 import binding as qb
    # Two token tiles by two row tiles, eight K-blocks: the producers of every CTA leave out the copy of their
    # fourth K-block (the bytes are announced to the stage's barrier and never arrive).  With the wait limit set to
    # 2 * 10^6 cycles (about a millisecond) the MMA issuer, the dequant warps, the producers and the epilogue warps
    # each run into the limit, the pair frees its tensor memory and the kernel ends on its own: no trap, no fault,
    # no endless loop.  The call itself returns OK (the launch succeeded); the status word says what happened.
    # The two larger shapes (19 row tiles x 5 token tiles of 512, four K-blocks) run the 256 x 512 tile form of
    # the kernel, with its four-stage ring and eight epilogue warps.
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


@pytest.mark.parametrize("d_out,d_in", [(4864, 256), (256, 4864)])
def test_a_producer_held_up_before_the_adapter_blocks_changes_nothing(d_out, d_in):
    from paper_2407_17029_b200 import binding as qb
    # 19 row tiles x 5 token tiles = 95 tiles on 74 CTA pairs, rank 256 = four adapter K-blocks = one whole turn
    # of the four-stage ring.  While a pair's producer idles in front of its first adapter K-block (what a long
    # wait for the adapter's compressed activation amounts to), the dequant warps can build all four adapter
    # tiles without it and reach the first weight K-blocks of the pair's next tile; they must not take the
    # barrier phases of the previous turn of the ring for the ones they wait for (they once did, and built those
    # weight tiles from the previous turn's codes).  (4864, 256) lays the forward's row tiles out this way,
    # (256, 4864) the backward's; the held call has to reproduce the ordinary one bit for bit.
    T, r = 2100, 256
    W = synth.normal(85, "hold/W", (d_out, d_in), 0.02)
    X = synth.round_to_bf16(synth.normal(85, "hold/X", (T, d_in)))
    dY = synth.round_to_bf16(synth.normal(85, "hold/dY", (T, d_out)))
    A = synth.round_to_bf16(synth.normal(85, "hold/A", (d_in // 64, r), 0.3))
    B = synth.round_to_bf16(synth.normal(85, "hold/B", (r, d_out // 8), 0.3))
    dq = qb.quantize_blockwise(torch.from_numpy(W).to("cuda:0"), 64, 1, qb.FMT_AFFINE_MINMAX)
    ad = qb.Adapter(64, 8, r, 1.0, to_bf16_dev(A), to_bf16_dev(B))
    Xd, dYd = to_bf16_dev(X), to_bf16_dev(dY)
    wsf = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, ad, T)
    wsb = qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, ad, T)
    Y = qb.linear_fwd(dq, ad, Xd, torch.float32, ws=wsf)
    dX = qb.linear_bwd(dq, ad, Xd, dYd, torch.float32, need_da=False, need_db=False, ws=wsb)[0]
    try:
        qb.debug_hold_producer(400_000)            # about 0.2 ms: several K-blocks' worth of everybody else's time
        Yh = qb.linear_fwd(dq, ad, Xd, torch.float32, ws=wsf)
        qb.debug_hold_producer(400_000)
        dXh = qb.linear_bwd(dq, ad, Xd, dYd, torch.float32, need_da=False, need_db=False, ws=wsb)[0]
    finally:
        qb.debug_hold_producer(0)
    assert qb.device_status(wsf) == qb.OK and qb.device_status(wsb) == qb.OK
    assert torch.equal(Yh, Y)
    assert torch.equal(dXh, dX)
