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
    Yq2 = sc.ScaledTensor.empty((M, N), torch.float8_e4m3fn)
    hint = torch.zeros(1, dtype=torch.float32, device=dev)   # carries over from call to call, whatever its value
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
    Pd = sc.ScaledTensor(torch.zeros((H, M, M), dtype=torch.uint8, device=dev).view(torch.float8_e4m3fn),
                         torch.ones(1, device=dev))
    dO8 = sc.ScaledTensor.make(torch.randn((M, N), device=dev, generator=g).to(torch.float8_e5m2), 2.0 ** -9)
    dS = sc.ScaledTensor.empty((H, M, M), torch.float8_e5m2)
    dQ, dK, dV = (sc.ScaledTensor(torch.empty((M, N), dtype=torch.bfloat16, device=dev).view(M, H, 64).permute(1, 0, 2),
                                  torch.zeros(1, device=dev)) for _ in range(3))
    ws_mm = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    ws_rs = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, M * N))
    heads = lambda X: sc.ScaledTensor(X.data.view(M, H, 64).permute(1, 0, 2), X.scale)

    def chain():
        sc.scalify_scaled_matmul(A, B, Y, ws_mm, transB=True, stat=sc.STAT_AMAX, Yq=Yq)   # GEMM + pass 2
        sc.scalify_scaled_matmul_speculative(A, B, Y, Yq2, hint, ws_mm, transB=True)       # predicted rescale
        sc.scalify_scaled_add(Y, R, S)
        sc.scalify_rescale(S, S8, stat=sc.STAT_AMAX, ws=ws_rs)                             # one-launch rescale
        sc.scalify_scaled_layernorm(S, gamma, beta, L, eps=1e-5, mean=mean, rinv=rinv)
        sc.scalify_mx_quantize(S, Am)
        sc.scalify_mx_quantize(W2, Bm)
        sc.scalify_mx_matmul(Am, Bm, Y2, ws_mm)
        sc.scalify_scaled_attention(heads(L), heads(S8), heads(Yq), O, sm_scale=0.125, causal=True, P_dump=Pd)
        sc.scalify_scaled_attention_bwd(heads(L), heads(S8), heads(Yq), Pd, heads(dO8), dS, dQ, dK, dV,
                                        sm_scale=0.125, causal=True)

    outs = (Yq, Yq2, S8, L, Y2, O, dQ, dK, dV)
    outputs = lambda: [x.data.contiguous().view(torch.uint8).cpu().numpy().copy() for x in outs] + \
                      [np.array([x.scale_value() for x in outs])]
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


def test_training_style_chain_with_state_replays_from_a_cuda_graph():
    """Calls that carry state from one call to the next (the delayed-rescale statistic, Adam's moments and
    weights with their scales) plus the backward and support kernels: two eager steps from a saved initial
    state must equal two replays of one recorded step from the same state."""
    dev = torch.device("cuda")
    g = torch.Generator(device=dev).manual_seed(11)
    rnd = lambda shape, dt, std=1.0: (torch.randn(shape, device=dev, generator=g) * std).to(dt)
    R, D, V, T = 256, 512, 1000, 64
    VP = 1008
    ids = torch.randint(0, V, (R,), device=dev, generator=g, dtype=torch.int64)
    targets = torch.randint(0, V, (R,), device=dev, generator=g, dtype=torch.int64)
    wte = sc.ScaledTensor.make(rnd((VP, D), torch.bfloat16, 0.02 * 64), 2.0 ** -6)
    wpe = sc.ScaledTensor.make(rnd((T, D), torch.bfloat16, 0.02 * 64), 2.0 ** -6)
    X = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    gamma = sc.ScaledTensor.make(rnd((D,), torch.bfloat16) * 0.1 + 1.0, 1.0)
    beta = sc.ScaledTensor.make(rnd((D,), torch.bfloat16, 0.1), 1.0)
    H8 = sc.ScaledTensor.empty((R, D), torch.float8_e4m3fn)
    mean = torch.empty(R, dtype=torch.float32, device=dev)
    rinv = torch.empty(R, dtype=torch.float32, device=dev)
    W8 = sc.ScaledTensor.make(rnd((VP, D), torch.float8_e4m3fn), 2.0 ** -6)
    stat_state = torch.full((1,), 2.0, dtype=torch.float32, device=dev)
    logits = sc.ScaledTensor.empty((R, VP), torch.bfloat16)
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    dlogits = sc.ScaledTensor.empty((R, VP), torch.float8_e5m2)
    dH = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    Gx = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    Ga = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    act = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    dX = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    dXq = sc.ScaledTensor.empty((R, D), torch.float8_e5m2)
    dgam = sc.ScaledTensor.empty((D,), torch.float32)
    dbet = sc.ScaledTensor.empty((D,), torch.float32)
    S = sc.ScaledTensor.make(rnd((4, T, T), torch.bfloat16, 2.0), 0.5)
    P = sc.ScaledTensor.empty((4, T, T), torch.float8_e4m3fn)
    dP = sc.ScaledTensor.make(rnd((4, T, T), torch.bfloat16), 2.0 ** -8)
    dS = sc.ScaledTensor.empty((4, T, T), torch.bfloat16)
    dwte = sc.ScaledTensor.empty((VP, D), torch.float32)
    dwpe = sc.ScaledTensor.empty((T, D), torch.float32)
    n = 4096 + 5
    ag = sc.ScaledTensor.make(rnd((n,), torch.float8_e5m2), 2.0 ** -12)
    am = sc.ScaledTensor.make(rnd((n,), torch.float16, 1.6), 2.0 ** -16)
    av = sc.ScaledTensor.make((rnd((n,), torch.float32) ** 2).to(torch.float16), 2.0 ** -24)
    aw = sc.ScaledTensor.make(rnd((n,), torch.float16, 1.28), 2.0 ** -6)
    awc = sc.ScaledTensor.make(torch.zeros(n, dtype=torch.uint8, device=dev).view(torch.float8_e4m3fn), 1.0)
    adam, wc = sc.AdamTensors([ag], [am], [av], [aw]), [awc]
    ws_mm = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, R, VP))
    ws_ln = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, D))
    ws_ce = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_CROSS_ENTROPY, R))
    ws_ad = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1))
    # delayed rescale of the LayerNorm gradient: the statistic word of its own workspace IS the state
    ws_lnd = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, D))
    ln_state = ws_lnd.statistic()
    ln_state.fill_(2.0 ** -9)
    dXd = sc.ScaledTensor.empty((R, D), torch.float8_e5m2)
    # the exact rescales that predict their power of two from the statistic their workspace saw last: the
    # prediction word is state too (the first step starts without one and takes the repair path)
    ws_ln1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, D))
    ws_rs1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, R * D, 0))
    dXq1 = sc.ScaledTensor.empty((R, D), torch.float8_e5m2)
    act8 = sc.ScaledTensor.empty((R, D), torch.float8_e4m3fn)
    state = [stat_state, ln_state, am.data, am.scale, av.data, av.scale, aw.data, aw.scale, ws_ln1.prediction(),
             ws_rs1.prediction()]
    saved = [x.clone() for x in state]

    def reset():
        for x, s in zip(state, saved):
            x.copy_(s)

    def step():
        sc.scalify_scaled_embedding(ids, T, wte, wpe, X)
        sc.scalify_scaled_layernorm(X, gamma, beta, H8, eps=1e-5, mean=mean, rinv=rinv)
        sc.scalify_scaled_matmul_delayed(H8, W8, stat_state, logits, ws_mm, transB=True, stat=sc.STAT_AMAX,
                                         stat_out=stat_state)
        sc.scalify_scaled_cross_entropy(logits, V, targets, loss, dlogits, ws_ce)
        sc.scalify_scaled_matmul(dlogits, W8, dH, ws_mm)
        sc.scalify_scaled_gelu(X, act)
        sc.scalify_scaled_gelu_bwd(dH, X, Ga)
        sc.scalify_scaled_layernorm_bwd(dH, X, gamma, mean, rinv, dX, ws_ln, eps=1e-5, stat_dx=sc.STAT_L2, dXq=dXq,
                                        dgamma=dgam, dbeta=dbet)
        sc.scalify_scaled_layernorm_bwd_delayed(dH, X, gamma, mean, rinv, ln_state, dXd, ws_lnd, eps=1e-5,
                                                stat_dx=sc.STAT_L2)
        sc.scalify_scaled_layernorm_bwd(dH, X, gamma, mean, rinv, None, ws_ln1, eps=1e-5, stat_dx=sc.STAT_L2, dXq=dXq1)
        sc.scalify_rescale(act, act8, stat=sc.STAT_AMAX, ws=ws_rs1)
        sc.scalify_scaled_softmax(S, P, causal=True)
        sc.scalify_scaled_softmax_bwd(dP, P, dS)
        sc.scalify_scaled_embedding_bwd(ids, T, dX, dwte, dwpe)
        sc.scalify_scaled_adam_step_cast(adam, wc, ws_ad, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=3)

    outs = [logits, dlogits, dH, act, Ga, dX, dXq, dXd, dXq1, act8, dgam, dbet, P, dS, am, av, aw, awc]
    atomics = [dwte, dwpe]   # scatter-adds with fp32 atomics: the order of the addends is not fixed

    def snapshot():
        torch.cuda.synchronize()
        return [x.data.contiguous().view(torch.uint8).cpu().numpy().copy() for x in outs] + \
               [np.array([x.scale_value() for x in outs] + [float(loss.item()), float(stat_state.item()), float(ln_state.item())])]

    reset()
    step()
    first = snapshot()
    first_atomics = [x.data.float().cpu().numpy().copy() for x in atomics]
    step()
    second = snapshot()
    assert not np.array_equal(first[-1], second[-1])     # the state did move between the steps
    reset()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            step()
    reset()
    graph.replay()
    for a, b in zip(snapshot(), first):
        assert np.array_equal(a, b)
    for x, w in zip(atomics, first_atomics):
        assert np.allclose(x.data.float().cpu().numpy(), w, rtol=1e-5, atol=1e-6)
    graph.replay()
    for a, b in zip(snapshot(), second):
        assert np.array_equal(a, b)
    # the one-pass rescale of the LayerNorm gradient gave the two-pass call's bits in every one of these runs
    assert torch.equal(dXq1.data.view(torch.uint8), dXq.data.view(torch.uint8)) and dXq1.scale_value() == dXq.scale_value()
