"""qablora_merge_noalloc: the merge for callers that cannot hand the library a workspace.

Some users of this library may not allocate device memory at the moment they need a merge (a serving
process whose memory is fully committed when an adapter is swapped in, code running inside another
framework's stream-ordered pipeline).  For them the library keeps the merge's scratch in a fixed
2 MiB array inside the library image.  This test calls that entry point through the C ABI twice in a
row, with different adapters, and requires the new beta to equal what the ordinary, workspace-based
qablora_merge produces -- bit for bit, the bar the merge tests use -- and checks that an adapter
too large for the fixed array is refused with a clear status instead of being attempted.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import DEV, adapter_to_dev, qweight_to_dev

pytestmark = pytest.mark.gpu


def _case(seed, d_out, d_in, r, scaling):
    W = synth.normal(seed, "na/W", (d_out, d_in), 0.02)
    A = synth.round_to_bf16(synth.normal(seed, "na/A", (d_in // 64, r), 0.02))
    B = synth.round_to_bf16(synth.normal(seed, "na/B", (r, d_out // 8), 0.02))
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    return qw, oracle.Adapter(64, 8, r, scaling, A, B)


def test_noalloc_merge_matches_workspace_merge_twice_in_a_row():
    from paper_2407_17029_b200 import binding as qb
    # two different problems back to back: the second must not see anything of the first in the scratch
    for seed, d_out, d_in, r, s in [(71, 640, 1024, 64, 3.0), (72, 320, 448, 48, 0.5)]:
        qw, ad = _case(seed, d_out, d_in, r, s)
        dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
        ref = qb.merge(dq, da)                                   # existing entry point (caller's workspace)
        out = torch.full_like(dq.beta, float("nan"))
        got = qb.merge_noalloc(dq, da, out)
        torch.cuda.synchronize()
        assert torch.equal(got.beta.view(torch.int32), ref.beta.view(torch.int32))
        assert np.array_equal(out.cpu().numpy().view(np.uint32), oracle.merge(qw, ad).beta.view(np.uint32))
        assert got.codes.data_ptr() == dq.codes.data_ptr() and got.alpha.data_ptr() == dq.alpha.data_ptr()


def test_noalloc_merge_refuses_what_does_not_fit():
    from paper_2407_17029_b200 import binding as qb
    # (d_in/64) * (d_out/8) = 64 * 4608 = 294912 > 262144 entries
    d_out, d_in, r = 36864, 4096, 8
    codes = torch.zeros((d_out, d_in // 2), dtype=torch.uint8, device=DEV)
    alpha = torch.ones((d_out, d_in // 64), dtype=torch.float32, device=DEV)
    beta = torch.zeros_like(alpha)
    dq = qb.QWeight(d_out, d_in, 64, 1, qb.FMT_AFFINE_MINMAX, [0.0] * 16, codes, alpha, beta)
    A = torch.zeros((d_in // 64, r), dtype=torch.bfloat16, device=DEV)
    B = torch.zeros((r, d_out // 8), dtype=torch.bfloat16, device=DEV)
    out = torch.full_like(beta, 7.0)
    with pytest.raises(qb.QbloraError) as e:
        qb.merge_noalloc(dq, qb.Adapter(64, 8, r, 1.0, A, B), out)
    assert e.value.status == qb.ERR_TOO_LARGE
    assert "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())                              # refused before anything ran
    qb.merge(dq, qb.Adapter(64, 8, r, 1.0, A, B))               # the workspace-based call still takes it
