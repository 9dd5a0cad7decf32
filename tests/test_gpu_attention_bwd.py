"""GPU parity of the fused attention backward against the oracle's composition of the calls it replaces
(scaled matmul -> softmax backward on the data components -> three scaled matmuls), stage by stage:
  dP       (optional copy) within 1 ulp of BF16 (or the 1e-5 * sum|a*b| accumulation bar) of the oracle's dO V^T,
  dS       against the oracle's softmax backward of the kernel's own dP: within 1 ulp of E5M2, or half an
           ulp plus 1e-5 * P (|dP| + sum|dP P|) (the row sum is accumulated in fp32); exactly 0 where P is 0,
  dQ       within 1 ulp (or the accumulation bar) of the oracle's matmul of the kernel's own dS with K,
  dK, dV   the same with dS^T Q and P^T dO,
  scales   bit-exact: dS_s = dO_s V_s kf(hd) c, dQ_s = dS_s K_s kf(Tk), dK_s = dS_s Q_s kf(Tq), dV_s = dO_s kf(Tq).
The probabilities fed in are the oracle's own (scores -> causal softmax -> E4M3), with exact zeros where the
mask hides a key."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu

HD = 64


def oracle_probabilities(q, q_dt, qs, k, ks, c, causal):
    H = q.shape[0]
    out = []
    for h in range(H):
        So, s_scale = orc.scaled_matmul(q[h], q_dt, qs, k[h], orc.E4M3, ks, orc.BF16, transB=True)[:2]
        Po, _ = orc.softmax_fwd(So[None], orc.BF16, s_scale * c, causal, orc.E4M3)
        out.append(Po[0])
    return np.stack(out)


def run_case(H, Tq, Tk, causal, merged_layout=False, q_dt=orc.E4M3, do_dt=orc.E5M2, g_dt=orc.BF16, seed=1,
             check_heads=None, HD=HD):
    qs, ks, vs, dos, c = 2.0 ** -1, 2.0 ** 1, 2.0 ** -3, 2.0 ** -9, 0.125
    q = si.to_bits(si.normal(seed, 1, (H, Tq, HD), 1.0), q_dt)
    k = si.to_bits(si.normal(seed, 2, (H, Tk, HD), 1.0), orc.E4M3)
    v = si.to_bits(si.normal(seed, 3, (H, Tk, HD), 1.0), orc.E4M3)
    do = si.to_bits(si.normal(seed, 4, (H, Tq, HD), 1.0), do_dt)
    P = oracle_probabilities(q, q_dt, qs, k, ks, c, causal)

    def dev_heads(x, dt, T):
        if not merged_layout:
            return to_dev(x, dt)
        buf = torch.zeros((T, H * HD), dtype=torch.uint8, device="cuda").view(sc.TORCH_DTYPE[dt])
        view = buf.view(T, H, HD).permute(1, 0, 2)      # [H, T, HD] view of a [T, H*HD] buffer
        view.copy_(to_dev(x, dt))
        return view

    def out_heads(T):
        if merged_layout:
            buf = torch.zeros((T, H * HD), dtype=sc.TORCH_DTYPE[g_dt], device="cuda")
            return sc.ScaledTensor(buf.view(T, H, HD).permute(1, 0, 2), torch.zeros(1, device="cuda"))
        return sc.ScaledTensor.empty((H, T, HD), sc.TORCH_DTYPE[g_dt])
    Q = sc.ScaledTensor.make(dev_heads(q, q_dt, Tq), qs)
    K = sc.ScaledTensor.make(dev_heads(k, orc.E4M3, Tk), ks)
    V = sc.ScaledTensor.make(dev_heads(v, orc.E4M3, Tk), vs)
    dO = sc.ScaledTensor.make(dev_heads(do, do_dt, Tq), dos)
    Pd = sc.ScaledTensor(to_dev(P, orc.E4M3), None)
    dS = sc.ScaledTensor(torch.full((H, Tq, Tk), 0x55, dtype=torch.uint8, device="cuda").view(torch.float8_e5m2),
                         torch.zeros(1, device="cuda"))
    dQ, dK, dV = out_heads(Tq), out_heads(Tk), out_heads(Tk)
    dPd = sc.ScaledTensor(torch.zeros((H, Tq, Tk), dtype=torch.bfloat16, device="cuda"), None)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_scaled_attention_bwd(Q, K, V, Pd, dO, dS, dQ, dK, dV, sm_scale=c, causal=causal, dP_dump=dPd,
                                    status=status)
    assert int(status.item()) == 0
    kf_hd, kf_tk, kf_tq = orc.kf(HD), orc.kf(Tk), orc.kf(Tq)
    ds_scale = dos * vs * kf_hd * c
    assert dS.scale_value() == ds_scale
    assert dQ.scale_value() == ds_scale * ks * kf_tk
    assert dK.scale_value() == ds_scale * qs * kf_tq
    assert dV.scale_value() == dos * kf_tq
    dP_gpu = to_bits(dPd.data, orc.BF16)
    dS_gpu = to_bits(dS.data, orc.E5M2)
    dQ_gpu = to_bits(dQ.data.contiguous(), g_dt)
    dK_gpu = to_bits(dK.data.contiguous(), g_dt)
    dV_gpu = to_bits(dV.data.contiguous(), g_dt)
    # blocks of 128 x 128 the kernel visits: all without a mask, else those not wholly above the diagonal
    ii, jj = np.meshgrid(np.arange(Tq), np.arange(Tk), indexing="ij")
    if causal:
        last_q_of_block = np.minimum((ii // 128) * 128 + 127, 10 ** 9)
        visited = (jj // 128) * 128 <= last_q_of_block + (Tk - Tq)
        visible = jj <= ii + (Tk - Tq)
    else:
        visited = np.ones((Tq, Tk), dtype=bool)
        visible = visited
    for h in (range(H) if check_heads is None else check_heads):
        assert np.all(P[h][~visible] == 0)
        # dP
        dPo, dp_scale, acc, sab = orc.scaled_matmul(do[h], do_dt, dos, v[h], orc.E4M3, vs, orc.BF16, transB=True,
                                                    want_acc=True)
        assert dp_scale == dos * vs * kf_hd
        ok = within(dP_gpu[h][visited], dPo[visited], orc.BF16, acc[visited], sab[visited], 1e-5)
        assert ok.all(), (h, int((~ok).sum()))
        # dS from the kernel's own dP
        dP_in = np.where(visited, dP_gpu[h], 0).astype(np.uint16)
        dSo, ss = orc.softmax_bwd(dP_in, orc.BF16, dp_scale, P[h], orc.E4M3, 1.0, orc.E5M2)
        pv = orc.decode(P[h], orc.E4M3)
        gv = orc.decode(dP_in, orc.BF16)
        dot = (pv * gv).sum(axis=1, keepdims=True)
        mag = pv * (np.abs(gv) + np.abs(pv * gv).sum(axis=1, keepdims=True))
        ok = within(dS_gpu[h][visited], dSo[visited], orc.E5M2, (pv * (gv - dot))[visited], mag[visited], 1e-5)
        assert ok.all(), (h, int((~ok).sum()))
        assert np.all((dS_gpu[h][visited & ~visible] & 0x7F) == 0)
        assert np.all(dS_gpu[h][~visited] == 0x55)           # untouched
        dS_in = np.where(visited, dS_gpu[h], 0).astype(np.uint8)
        # dQ = dS K
        Qo, s1, a1, b1 = orc.scaled_matmul(dS_in, orc.E5M2, ds_scale, k[h], orc.E4M3, ks, g_dt, want_acc=True)
        assert s1 == ds_scale * ks * kf_tk
        ok = within(dQ_gpu[h], Qo, g_dt, a1, b1, 1e-5)
        assert ok.all(), ("dQ", h, int((~ok).sum()))
        # dK = dS^T Q
        Ko, s2, a2, b2 = orc.scaled_matmul(dS_in, orc.E5M2, ds_scale, q[h], q_dt, qs, g_dt, transA=True, want_acc=True)
        assert s2 == ds_scale * qs * kf_tq
        ok = within(dK_gpu[h], Ko, g_dt, a2, b2, 1e-5)
        assert ok.all(), ("dK", h, int((~ok).sum()))
        # dV = P^T dO
        Vo, s3, a3, b3 = orc.scaled_matmul(P[h], orc.E4M3, 1.0, do[h], do_dt, dos, g_dt, transA=True, want_acc=True)
        assert s3 == dos * kf_tq
        ok = within(dV_gpu[h], Vo, g_dt, a3, b3, 1e-5)
        assert ok.all(), ("dV", h, int((~ok).sum()))


@pytest.mark.parametrize("H,T", [(2, 128), (3, 256), (2, 1024)])
def test_causal_self_attention_backward(H, T):
    run_case(H, T, T, True)


def test_backward_benchmark_shape_96_heads_of_1024_tokens_sampled_heads():
    run_case(96, 1024, 1024, True, seed=11, check_heads=[0, 1, 37, 73, 94, 95])


def test_full_attention_backward_with_more_keys_than_queries():
    run_case(2, 128, 384, False)


def test_ragged_lengths_and_shifted_causal_mask_backward():
    run_case(2, 200, 224, True)


@pytest.mark.parametrize("H,Tq,Tk,causal", [(1, 96, 32, False), (2, 320, 320, True), (1, 40, 2048, True),
                                            (1, 2048, 2048, True), (3, 64, 64, True)])
def test_backward_edge_shapes(H, Tq, Tk, causal):
    # a single partial key block; a length that ends in the middle of a 128-query block (one 64-query ring
    # slot of the dK/dV launch is empty past the end); few queries against many keys; 16 key blocks
    run_case(H, Tq, Tk, causal, seed=7)


@pytest.mark.parametrize("H,Tq,Tk,causal", [(2, 128, 128, True), (3, 384, 384, True), (2, 200, 224, True),
                                            (2, 128, 384, False), (1, 1024, 1024, True), (1, 96, 32, False)])
def test_backward_head_dimension_128(H, Tq, Tk, causal):
    """Rows of 128 elements travel as two 64-byte column halves per tile: dP accumulates over both, dQ, dK and dV
    have 64 columns per half."""
    run_case(H, Tq, Tk, causal, HD=128)


def test_backward_head_dimension_128_at_48_heads_of_1024_tokens_sampled_heads():
    run_case(48, 1024, 1024, True, seed=13, check_heads=[0, 17, 47], HD=128)


def test_backward_head_dimension_128_inside_a_token_major_buffer_and_mixed_formats():
    run_case(3, 256, 256, True, merged_layout=True, q_dt=orc.E5M2, do_dt=orc.E4M3, g_dt=orc.F16, HD=128)


def test_backward_of_a_single_head_given_as_2d_arrays():
    T = 256
    q = si.to_bits(si.normal(9, 1, (1, T, HD), 1.0), orc.E4M3)
    k = si.to_bits(si.normal(9, 2, (1, T, HD), 1.0), orc.E4M3)
    v = si.to_bits(si.normal(9, 3, (1, T, HD), 1.0), orc.E4M3)
    do = si.to_bits(si.normal(9, 4, (1, T, HD), 1.0), orc.E5M2)
    P = oracle_probabilities(q, orc.E4M3, 1.0, k, 1.0, 0.125, True)
    mk = lambda x, dt, s: sc.ScaledTensor.make(to_dev(x[0], dt), s)
    Q, K, V, dO = mk(q, orc.E4M3, 1.0), mk(k, orc.E4M3, 1.0), mk(v, orc.E4M3, 1.0), mk(do, orc.E5M2, 1.0)
    Pd = sc.ScaledTensor(to_dev(P, orc.E4M3), None)
    dS = sc.ScaledTensor.empty((1, T, T), torch.float8_e5m2)
    out2, out3 = [], []
    for shape, outs in (((T, HD), out2), ((1, T, HD), out3)):
        dQ, dK, dV = (sc.ScaledTensor.empty(shape, torch.float32) for _ in range(3))
        a = (Q, K, V, Pd, dO) if len(shape) == 2 else tuple(
            sc.ScaledTensor(t.data.reshape((1,) + tuple(t.data.shape)), t.scale) if t is not Pd else t
            for t in (Q, K, V, Pd, dO))
        sc.scalify_scaled_attention_bwd(*a, dS, dQ, dK, dV, sm_scale=0.125, causal=True)
        outs.extend(to_bits(t.data, orc.F32).reshape(-1) for t in (dQ, dK, dV))
    for x, y in zip(out2, out3):
        assert np.array_equal(x, y)


def test_backward_heads_inside_a_token_major_buffer_and_mixed_formats():
    run_case(4, 256, 256, True, merged_layout=True, q_dt=orc.E5M2, do_dt=orc.E4M3, g_dt=orc.F16)


def test_backward_argument_checks():
    H, T = 2, 128
    f8 = lambda *s: sc.ScaledTensor.make(torch.zeros(s, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn), 1.0)
    Q, K, V, dO = f8(H, T, 64), f8(H, T, 64), f8(H, T, 64), f8(H, T, 64)
    P = f8(H, T, T)
    dS = sc.ScaledTensor(torch.zeros((H, T, T), dtype=torch.uint8, device="cuda").view(torch.float8_e5m2),
                         torch.zeros(1, device="cuda"))
    dQ, dK, dV = (sc.ScaledTensor.empty((H, T, 64), torch.bfloat16) for _ in range(3))
    with pytest.raises(sc.ScalifyError):
        sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, dS, dQ, dK, dV, sm_scale=0.1)    # not a power of two
    with pytest.raises(sc.ScalifyError):
        no_scale = sc.ScaledTensor(dS.data, None)
        sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, no_scale, dQ, dK, dV, sm_scale=0.125)
    with pytest.raises(sc.ScalifyError):
        dV16 = sc.ScaledTensor.empty((H, T, 64), torch.float16)
        sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, dS, dQ, dK, dV16, sm_scale=0.125)   # mixed gradient dtypes
    sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, dS, dQ, dK, dV, sm_scale=0.125)
