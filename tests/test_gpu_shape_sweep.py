"""Random shapes: the tensor-core path against the general CUDA-core path of the same library (no oracle needed, so
the shapes can be large and many), twice per shape, some with the producers of the fused contraction held up in front
of their adapter K-blocks.  Both paths are gated against the oracle elsewhere; what this sweep looks for is what a
handful of hand-picked shapes can miss: a tile schedule, a ragged edge or a barrier phase that goes wrong only for
some combination of row tiles, token tiles, K-blocks, rank and timing.  The two paths differ by the bf16 rounding of
the weight operand (rms 1.7e-3 of the output, maxima just under 1e-2 of a token row's RMS), so whole wrong tiles or
stale operands stand out by two orders of magnitude."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _err(a, b):
    a, b = a.double(), b.double()
    row = b.pow(2).mean(dim=1, keepdim=True).sqrt().clamp_min(1e-30)
    return float(((a - b).abs() / row).max()), float((a - b).pow(2).mean().sqrt() / b.pow(2).mean().sqrt().clamp_min(1e-30))


@pytest.mark.parametrize("seed", range(6))
def test_tensor_core_path_against_general_path_on_random_shapes(seed, monkeypatch):
    from paper_2407_17029_b200 import binding as qb
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(1000 + seed)
    gen = torch.Generator(device=dev).manual_seed(1000 + seed)
    for case in range(40):
        big = rng.random() < 0.5
        if rng.random() < 0.5:      # many row tiles in the forward
            d_out, d_in = int(rng.integers(1, 100 if big else 12)) * 64, int(rng.integers(1, 12 if big else 20)) * 64
        else:                       # many row tiles in the backward
            d_in, d_out = int(rng.integers(1, 100 if big else 20)) * 64, int(rng.integers(1, 12)) * 64
        T = int(rng.integers(1, 3300 if big else 600))
        qfmt = int(rng.integers(0, 2))
        r = int(rng.choice([0, 8, 16, 48, 64, 136, 256]))
        hold = int(rng.choice([0, 0, 100_000, 400_000]))
        W = torch.randn(d_out, d_in, device=dev, generator=gen) * 0.02
        dq = qb.quantize_blockwise(W, 64, 1, qfmt)
        X = torch.randn(T, d_in, device=dev, generator=gen).to(torch.bfloat16)
        dY = torch.randn(T, d_out, device=dev, generator=gen).to(torch.bfloat16)
        ad = None
        if r:
            A = (torch.randn(d_in // 64, r, device=dev, generator=gen) * 0.3).to(torch.bfloat16)
            B = (torch.randn(r, d_out // 8, device=dev, generator=gen) * 0.3).to(torch.bfloat16)
            ad = qb.Adapter(64, 8, r, float(rng.choice([1.0, 0.05])), A, B)

        def run(ws_f=None, ws_b=None):
            Y = qb.linear_fwd(dq, ad, X, torch.float32, ws=ws_f)
            if ad is None:
                return Y, qb.linear_bwd(dq, None, None, dY, torch.float32, ws=ws_b)[0], None, None
            return (Y,) + tuple(qb.linear_bwd(dq, ad, X, dY, torch.float32, ws=ws_b))

        monkeypatch.setenv("QBLORA_FORCE_GENERAL", "1")
        ref = run()
        monkeypatch.delenv("QBLORA_FORCE_GENERAL")
        wsf, wsb = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, ad, T), qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, ad, T)
        what = f"seed {seed} case {case}: T={T} d_out={d_out} d_in={d_in} fmt={qfmt} r={r} hold={hold}"
        outs = []
        try:
            for rep in range(2):
                if ad is not None and hold:
                    qb.debug_hold_producer(hold)        # consumed by the forward's contraction
                Y = qb.linear_fwd(dq, ad, X, torch.float32, ws=wsf)
                if ad is not None and hold:
                    qb.debug_hold_producer(hold)        # ... and by the backward's
                rest = (qb.linear_bwd(dq, None, None, dY, torch.float32, ws=wsb)[0], None, None) if ad is None \
                    else tuple(qb.linear_bwd(dq, ad, X, dY, torch.float32, ws=wsb))
                outs.append((Y,) + rest)
        finally:
            qb.debug_hold_producer(0)
        assert qb.device_status(wsf) == qb.OK and qb.device_status(wsb) == qb.OK, what
        for a, b in zip(outs[0], outs[1]):
            assert a is None or torch.equal(a, b), what + " (second call differs from the first)"
        for name, got, want in (("Y", outs[0][0], ref[0]), ("dX", outs[0][1], ref[1])):
            mx, rm = _err(got, want)
            assert mx <= 3e-2 and rm <= 5e-3, f"{what}: {name} max/row-rms {mx:.3e}, rms/rms {rm:.3e}"
        if ad is not None:
            for name, got, want in (("dA", outs[0][2], ref[2]), ("dB", outs[0][3], ref[3])):
                e = float((got - want).abs().max() / want.pow(2).mean().sqrt().clamp_min(1e-30))
                assert e <= 1e-2, f"{what}: {name} max/rms {e:.3e}"


@pytest.mark.parametrize("seed", range(3))
def test_low_bit_product_against_general_path_on_random_shapes(seed, monkeypatch):
    # the merged layer's product at every kind of token count: the one-token and K-outer decode kernels (1..16),
    # the fused contraction with its offset-term K-blocks in both tile forms (17 and up)
    from paper_2407_17029_b200 import binding as qb
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(2000 + seed)
    gen = torch.Generator(device=dev).manual_seed(2000 + seed)
    for case in range(40):
        d_out, d_in = int(rng.integers(1, 120)) * 64, int(rng.integers(1, 60)) * 64
        T = int(rng.choice([1, 2, 3, 5, 8, 9, 12, 16, 17, 40, 200, 257, 600, 1500, 2600]))
        W = torch.randn(d_out, d_in, device=dev, generator=gen) * 0.02
        dq = qb.quantize_blockwise(W, 64, 1, qb.FMT_AFFINE_MINMAX)
        A = (torch.randn(d_in // 64, 64, device=dev, generator=gen) * 0.3).to(torch.bfloat16)
        B = (torch.randn(64, d_out // 8, device=dev, generator=gen) * 0.3).to(torch.bfloat16)
        merged = qb.merge(dq, qb.Adapter(64, 8, 64, float(rng.choice([1.0, 20.0])), A, B))
        X = torch.randn(T, d_in, device=dev, generator=gen).to(torch.bfloat16)
        monkeypatch.setenv("QBLORA_FORCE_GENERAL", "1")
        ref = qb.lowbit_gemm(merged, X, torch.float32)
        monkeypatch.delenv("QBLORA_FORCE_GENERAL")
        ws = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, merged, None, T)
        Y1 = qb.lowbit_gemm(merged, X, torch.float32, ws=ws)
        Y2 = qb.lowbit_gemm(merged, X, torch.float32, ws=ws)
        what = f"seed {seed} case {case}: T={T} d_out={d_out} d_in={d_in}"
        assert qb.device_status(ws) == qb.OK, what
        assert torch.equal(Y1, Y2), what + " (second call differs from the first)"
        mx, rm = _err(Y1, ref)
        assert mx <= 3e-2 and rm <= 5e-3, f"{what}: max/row-rms {mx:.3e}, rms/rms {rm:.3e}"
