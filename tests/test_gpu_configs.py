"""GPU parity at the full sizes of the five benchmark configurations, in the launch configuration
the benchmark times.  The oracle computes a seeded sample of token rows (each row in full) for Y
and dX, and dA / dB over all tokens (they do not involve the base weight)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import (adapter_to_dev, gate_bf16, gate_strict, qweight_to_dev, sample_rows, to_bf16_dev,
                           to_dev, to_np64, visible_scaling)

pytestmark = pytest.mark.gpu

N_ROWS = {"C1": 256, "C2": 96, "C3": 48, "C4": 32, "C5": 32}


@pytest.fixture(scope="module")
def qb():
    from paper_2407_17029_b200 import binding
    return binding


def cases():
    out = []
    for name in ("C1", "C2", "C3", "C4"):
        wl = synth.WORKLOADS[name]
        for spec in wl.linears:
            if name == "C4" and spec.name in ("k", "v", "o", "up"):
                continue                      # same shapes as q / gate; the benchmark still runs them
            geoms = (synth.GEOM_A, synth.GEOM_B) if name in ("C1", "C2") else (synth.GEOM_A,)
            for g in geoms:
                out.append(pytest.param(name, spec, g, id=f"{name}-{spec.name}-{g.name}"))
    return out


@pytest.mark.parametrize("name,spec,geom", cases())
def test_finetune_config_fwd_bwd(qb, name, spec, geom):
    wl = synth.WORKLOADS[name]
    li = synth.make_linear_inputs(wl, spec, geom, seed=0)
    T = wl.tokens
    qw = oracle.quantize_blockwise(li.W, wl.block_in, 1, wl.qfmt)
    # full-size quantizer parity, bit for bit
    dq = qb.quantize_blockwise(to_dev(li.W), wl.block_in, 1, wl.qfmt)
    assert np.array_equal(dq.codes.cpu().numpy(), qw.codes)
    assert np.array_equal(dq.alpha.cpu().numpy().view(np.uint32), qw.alpha.view(np.uint32))
    del li.W
    Wt = oracle.dequantize(qw)
    rows = sample_rows(7, T, N_ROWS[name])
    Xs, dYs = li.X[rows], li.dY[rows]
    Xd, dYd = to_bf16_dev(li.X), to_bf16_dev(li.dY)
    for visible in (False, True):
        ad = oracle.Adapter(geom.lambda_in, geom.lambda_out, li.rank, li.scaling, li.A, li.B)
        if visible:
            ad.scaling = visible_scaling(Wt, ad, Xs)
        da = adapter_to_dev(ad)
        refY = oracle.linear_fwd(Wt, ad, Xs)
        Y = qb.linear_fwd(dq, da, Xd, torch.bfloat16)
        gate_bf16(to_np64(Y[torch.from_numpy(rows).to(Y.device)]), refY, f"{name}/{spec.name} Y visible={visible}")
        refdX, _, _ = oracle.linear_bwd(Wt, ad, Xs, dYs, want_da=False, want_db=False)
        _, refdA, refdB = oracle.linear_bwd(None, ad, li.X, li.dY, want_dx=False)
        dX, dA, dB = qb.linear_bwd(dq, da, Xd, dYd, torch.bfloat16)
        gate_bf16(to_np64(dX[torch.from_numpy(rows).to(dX.device)]), refdX, f"{name}/{spec.name} dX visible={visible}")
        gate_strict(to_np64(dA), refdA, f"{name}/{spec.name} dA", per_row=False)
        gate_strict(to_np64(dB), refdB, f"{name}/{spec.name} dB", per_row=False)


@pytest.mark.parametrize("spec", synth.WORKLOADS["C5"].linears, ids=lambda s: s.name)
def test_deploy_config_merge_and_lowbit(qb, spec):
    wl = synth.WORKLOADS["C5"]
    li = synth.make_linear_inputs(wl, spec, synth.GEOM_A, seed=0, tokens=2048)
    qw = oracle.quantize_blockwise(li.W, wl.block_in, 1, oracle.FMT_AFFINE_MINMAX)
    dq = qb.quantize_blockwise(to_dev(li.W), wl.block_in, 1, qb.FMT_AFFINE_MINMAX)
    assert np.array_equal(dq.codes.cpu().numpy(), qw.codes)
    assert np.array_equal(dq.alpha.cpu().numpy().view(np.uint32), qw.alpha.view(np.uint32))
    assert np.array_equal(dq.beta.cpu().numpy().view(np.uint32), qw.beta.view(np.uint32))
    del li.W
    Wt = oracle.dequantize(qw)
    rows = sample_rows(9, 2048, N_ROWS["C5"])
    ad = oracle.Adapter(64, 8, li.rank, 1.0, li.A, li.B)
    ad.scaling = visible_scaling(Wt, ad, li.X[rows])           # make the merged shift matter
    merged_ref = oracle.merge(qw, ad)
    merged = qb.merge(dq, adapter_to_dev(ad))
    assert np.array_equal(merged.beta.cpu().numpy().view(np.uint32), merged_ref.beta.view(np.uint32))
    assert torch.equal(merged.codes, dq.codes) and torch.equal(merged.alpha, dq.alpha)
    unmerged = oracle.linear_fwd(Wt, ad, li.X[rows])            # the paper's merge identity as the target
    for T in wl.lowbit_tokens:
        sel = rows[:T] if T < len(rows) else rows
        Xd = to_bf16_dev(li.X[:T] if T < 2048 else li.X)
        Y = qb.lowbit_gemm(merged, Xd, torch.bfloat16)
        if T < 2048:
            ref = oracle.linear_fwd(Wt, ad, li.X[:T])
            gate_bf16(to_np64(Y), ref, f"C5/{spec.name} lowbit T={T}")
        else:
            gate_bf16(to_np64(Y[torch.from_numpy(sel).to(Y.device)]), unmerged, f"C5/{spec.name} lowbit T=2048")
