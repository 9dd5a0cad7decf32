"""The library's calls can be recorded into a CUDA graph and replayed: they allocate nothing, never
synchronise and take all data-dependent quantities (scales, statistics) from device memory.  A chain
of calls is run eagerly, captured, replayed on fresh inputs, and must reproduce the eager results bit
for bit."""
import numpy as np
import pytest
import torch

import paper_2407_17353_b200 as sc

pytestmark = pytest.mark.gpu


def build_chain(seed_scale):
    dev = torch.device("cuda")
    g = torch.Generator(device=dev).manual_seed(7)
    M, N, K = 512, 768, 256
    t = {}
    t["a"] = torch.randn((M, K), device=dev, generator=g)
    t["b"] = torch.randn((N, K), device=dev, generator=g)
    A = sc.ScaledTensor.make((t["a"] * seed_scale).to(torch.float8_e4m3fn), 1.0)
    B = sc.ScaledTensor.make(t["b"].to(torch.float8_e4m3fn), 2.0 ** -6)
    Y = sc.ScaledTensor.empty((M, N), torch.bfloat16)
    Yq = sc.ScaledTensor.empty((M, N), torch.float8_e4m3fn)
    R = sc.ScaledTensor.make(torch.randn((M, N), device=dev, generator=g).to(torch.bfloat16), 1.0)
    S = sc.ScaledTensor.empty((M, N), torch.bfloat16)
    S8 = sc.ScaledTensor.empty((M, N), torch.float8_e4m3fn)
    gamma = sc.ScaledTensor.make(torch.ones(N, device=dev).to(torch.bfloat16), 1.0)
    beta = sc.ScaledTensor.make(torch.zeros(N, device=dev).to(torch.bfloat16), 1.0)
    L = sc.ScaledTensor.empty((M, N), torch.float8_e4m3fn)
    mean = torch.empty(M, dtype=torch.float32, device=dev)
    rinv = torch.empty(M, dtype=torch.float32, device=dev)
    Am, Bm = sc.MxTensor(M, N), sc.MxTensor(N, N)
    W2 = sc.ScaledTensor.make(torch.randn((N, N), device=dev, generator=g).to(torch.bfloat16), 2.0 ** -5)
    Y2 = sc.ScaledTensor.empty((M, N), torch.bfloat16)
    H = N // 64
    O = sc.ScaledTensor(torch.empty((M, N), dtype=torch.bfloat16, device=dev).view(M, H, 64).permute(1, 0, 2),
                        torch.zeros(1, device=dev))
    ws_mm = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    ws_rs = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, M * N))
    heads = lambda X: sc.ScaledTensor(X.data.view(M, H, 64).permute(1, 0, 2), X.scale)

    def chain():
        sc.scalify_scaled_matmul(A, B, Y, ws_mm, transB=True, stat=sc.STAT_AMAX, Yq=Yq)   # GEMM + pass 2
        sc.scalify_scaled_add(Y, R, S)
        sc.scalify_rescale(S, S8, stat=sc.STAT_AMAX, ws=ws_rs)                             # one-launch rescale
        sc.scalify_scaled_layernorm(S, gamma, beta, L, eps=1e-5, mean=mean, rinv=rinv)
        sc.scalify_mx_quantize(S, Am)
        sc.scalify_mx_quantize(W2, Bm)
        sc.scalify_mx_matmul(Am, Bm, Y2, ws_mm)
        sc.scalify_scaled_attention(heads(L), heads(S8), heads(Yq), O, sm_scale=0.125, causal=True)

    outputs = lambda: [x.data.contiguous().view(torch.uint8).cpu().numpy().copy() for x in (Yq, S8, L, Y2, O)] + \
                      [np.array([x.scale_value() for x in (Yq, S8, L, Y2, O)])]
    return A, t, chain, outputs


def test_chain_of_calls_replays_from_a_cuda_graph():
    A, t, chain, outputs = build_chain(1.0)
    set_input = lambda f: A.data.copy_((t["a"] * f).to(torch.float8_e4m3fn))
    # eager results for a small and a large input (the statistics and scales differ, all on the device);
    # these runs also do the one-time host work (function attributes, the tensor-map entry point)
    want = {}
    for f in (0.25, 3.0):
        set_input(f)
        chain()
        torch.cuda.synchronize()
        want[f] = outputs()
    assert not np.array_equal(want[0.25][-1], want[3.0][-1])   # the propagated scales do differ
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            chain()
    # replays in both orders: a replay must not see anything a previous replay left behind (a larger
    # statistic of an earlier input, a stale scale word)
    for f in (3.0, 0.25, 0.25, 3.0):
        set_input(f)
        graph.replay()
        torch.cuda.synchronize()
        got = outputs()
        for g, w in zip(got, want[f]):
            assert np.array_equal(g, w), f
    # and eager calls still work after replays
    set_input(0.25)
    chain()
    torch.cuda.synchronize()
    for g, w in zip(outputs(), want[0.25]):
        assert np.array_equal(g, w)
