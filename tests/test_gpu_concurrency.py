"""Host-side concurrency through the C ABI: CUDA-graph replay of the 256 x 512 tile form, and two host threads
calling the library at the same time on their own streams and workspaces (the library's cached per-device state is
atomic and its backward side stream is per thread; callers only have to keep one workspace to one call at a time)."""
import threading

import pytest
import torch

pytestmark = pytest.mark.gpu


def _problem(qb, seed, T, d_out, d_in, r):
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev).manual_seed(seed)
    W = torch.randn(d_out, d_in, device=dev, generator=gen) * 0.02
    dq = qb.quantize_blockwise(W, 64, 1, seed & 1)
    A = (torch.randn(d_in // 64, r, device=dev, generator=gen) * 0.2).to(torch.bfloat16)
    B = (torch.randn(r, d_out // 8, device=dev, generator=gen) * 0.2).to(torch.bfloat16)
    ad = qb.Adapter(64, 8, r, 1.0, A, B)
    X = torch.randn(T, d_in, device=dev, generator=gen).to(torch.bfloat16)
    dY = torch.randn(T, d_out, device=dev, generator=gen).to(torch.bfloat16)
    return dq, ad, X, dY


def test_cuda_graph_replay_of_wide_tiles_equals_eager_calls():
    from paper_2407_17029_b200 import binding as qb
    # 19 row tiles x 5 token tiles of 512 on 74 CTA pairs, forward and backward (the backward's row tiles come from
    # the second problem, whose d_in is the large side)
    for T, d_out, d_in in ((2100, 4864, 256), (2100, 256, 4864)):
        dq, ad, X0, dY0 = _problem(qb, 11, T, d_out, d_in, 64)
        _, _, X1, dY1 = _problem(qb, 12, T, d_out, d_in, 64)
        wf = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, ad, T)
        wb = qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, ad, T)
        eager = []
        for X, dY in ((X0, dY0), (X1, dY1)):
            Y = qb.linear_fwd(dq, ad, X, ws=wf)
            dX, dA, dB = qb.linear_bwd(dq, ad, X, dY, ws=wb)
            torch.cuda.synchronize()
            eager.append((Y.clone(), dX.clone(), dA.clone(), dB.clone()))
        Xs, dYs = torch.empty_like(X0), torch.empty_like(dY0)
        Y, dX = torch.empty_like(eager[0][0]), torch.empty_like(eager[0][1])
        dA, dB = torch.empty_like(eager[0][2]), torch.empty_like(eager[0][3])
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            Xs.copy_(X0); dYs.copy_(dY0)
            qb.linear_fwd(dq, ad, Xs, ws=wf, out=Y)
            qb.linear_bwd(dq, ad, Xs, dYs, ws=wb, outs=(dX, dA, dB))
            st.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                qb.linear_fwd(dq, ad, Xs, ws=wf, out=Y)
                qb.linear_bwd(dq, ad, Xs, dYs, ws=wb, outs=(dX, dA, dB))
            for it in range(10):
                k = it & 1
                Xs.copy_((X0, X1)[k]); dYs.copy_((dY0, dY1)[k])
                g.replay()
                st.synchronize()
                assert torch.equal(Y, eager[k][0]) and torch.equal(dX, eager[k][1]), f"replay {it}"
                assert torch.equal(dA, eager[k][2]) and torch.equal(dB, eager[k][3]), f"replay {it}"
        assert qb.device_status(wf) == qb.OK and qb.device_status(wb) == qb.OK


def test_two_host_threads_on_their_own_streams():
    from paper_2407_17029_b200 import binding as qb
    shapes = ((1100, 2560, 512, 64), (700, 512, 2304, 136))
    problems, refs = [], []
    for i, (T, d_out, d_in, r) in enumerate(shapes):
        dq, ad, X, dY = _problem(qb, 21 + i, T, d_out, d_in, r)
        wf = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, ad, T)
        wb = qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, ad, T)
        Y = qb.linear_fwd(dq, ad, X, ws=wf)
        dX, dA, dB = qb.linear_bwd(dq, ad, X, dY, ws=wb)
        torch.cuda.synchronize()
        problems.append((dq, ad, X, dY, wf, wb))
        refs.append((Y.clone(), dX.clone(), dA.clone(), dB.clone()))
    errors = []
    start = threading.Barrier(2)

    def worker(i):
        try:
            torch.cuda.set_device(0)
            dq, ad, X, dY, wf, wb = problems[i]
            st = torch.cuda.Stream()
            start.wait()
            with torch.cuda.stream(st):
                for it in range(40):
                    Y = qb.linear_fwd(dq, ad, X, ws=wf)
                    dX, dA, dB = qb.linear_bwd(dq, ad, X, dY, ws=wb)
                    if it % 8 == 7:
                        st.synchronize()
                        same = all(torch.equal(a, b) for a, b in zip((Y, dX, dA, dB), refs[i]))
                        if not same or qb.device_status(wf, st) != qb.OK or qb.device_status(wb, st) != qb.OK:
                            errors.append(f"thread {i} iteration {it}")
                st.synchronize()
        except Exception as ex:      # surface in the main thread
            errors.append(f"thread {i}: {ex!r}")

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
