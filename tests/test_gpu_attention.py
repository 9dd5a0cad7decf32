"""GPU parity of the fused attention forward against the oracle's composition of the calls it replaces
(scaled matmul -> softmax on values -> scaled matmul), stage by stage through the kernel's optional
copies of the scores and the probabilities:
  scores   within 1 ulp of BF16 (or the 1e-5 * sum|a*b| accumulation bar) of the oracle's Q K^T,
  P        within 1 ulp of E4M3 of the oracle's softmax of the kernel's own scores (exactly 0 where masked),
  O        within 1 ulp (or the accumulation bar) of the oracle's matmul of the kernel's own P with V,
  O scale  bit-exact (V_s * kf(Tk))."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu

HD = 64


def run_case(H, Tq, Tk, causal, merged_layout=False, q_dt=orc.E4M3, v_dt=orc.E4M3, o_dt=orc.BF16, seed=1,
             check_heads=None, c=0.125, HD=HD):
    qs, ks, vs = 2.0 ** -1, 2.0 ** 1, 2.0 ** -3
    q = si.to_bits(si.normal(seed, 1, (H, Tq, HD), 1.0), q_dt)
    k = si.to_bits(si.normal(seed, 2, (H, Tk, HD), 1.0), orc.E4M3)
    v = si.to_bits(si.normal(seed, 3, (H, Tk, HD), 1.0), v_dt)

    def dev_heads(x, dt, T):
        if not merged_layout:
            return to_dev(x, dt)
        buf = torch.zeros((T, H * HD), dtype=torch.uint8, device="cuda").view(sc.TORCH_DTYPE[dt])
        view = buf.view(T, H, HD).permute(1, 0, 2)      # [H, T, HD] view of a [T, H*HD] buffer
        view.copy_(to_dev(x, dt))
        return view
    Q = sc.ScaledTensor.make(dev_heads(q, q_dt, Tq), qs)
    K = sc.ScaledTensor.make(dev_heads(k, orc.E4M3, Tk), ks)
    V = sc.ScaledTensor.make(dev_heads(v, v_dt, Tk), vs)
    if merged_layout:
        obuf = torch.zeros((Tq, H * HD), dtype=sc.TORCH_DTYPE[o_dt], device="cuda")
        O = sc.ScaledTensor(obuf.view(Tq, H, HD).permute(1, 0, 2), torch.zeros(1, device="cuda"))
    else:
        O = sc.ScaledTensor.empty((H, Tq, HD), sc.TORCH_DTYPE[o_dt])
    Sd = sc.ScaledTensor(torch.zeros((H, Tq, Tk), dtype=torch.bfloat16, device="cuda"), None)
    Pd = sc.ScaledTensor(torch.zeros((H, Tq, Tk), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn), None)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_scaled_attention(Q, K, V, O, sm_scale=c, causal=causal, S_dump=Sd, P_dump=Pd, status=status)
    assert int(status.item()) == 0
    kf_hd, kf_tk = orc.kf(HD), orc.kf(Tk)
    assert O.scale_value() == vs * kf_tk
    S_gpu = to_bits(Sd.data, orc.BF16)
    P_gpu = to_bits(Pd.data, orc.E4M3)
    O_gpu = to_bits(O.data.contiguous(), o_dt)
    ii, jj = np.meshgrid(np.arange(Tq), np.arange(Tk), indexing="ij")
    visible = (jj <= ii + (Tk - Tq)) if causal else np.ones((Tq, Tk), dtype=bool)
    for h in (range(H) if check_heads is None else check_heads):
        # scores
        So, s_scale, acc, sab = orc.scaled_matmul(q[h], q_dt, qs, k[h], orc.E4M3, ks, orc.BF16, transB=True,
                                                  want_acc=True)
        assert s_scale == qs * ks * kf_hd
        ok = within(S_gpu[h][visible], So[visible], orc.BF16, acc[visible], sab[visible], 1e-5)
        assert ok.all(), (h, int((~ok).sum()))
        # probabilities from the kernel's own scores
        S_in = np.where(visible, S_gpu[h], 0).astype(np.uint16)
        Po, ps = orc.softmax_fwd(S_in[None], orc.BF16, s_scale * c, causal, orc.E4M3)
        assert ps == 1.0
        assert ulp_diff(P_gpu[h][visible], Po[0][visible], orc.E4M3).max() <= 1, h
        assert np.all(P_gpu[h][~visible] == 0)
        # output from the kernel's own probabilities
        Oo, o_scale, oacc, osab = orc.scaled_matmul(P_gpu[h], orc.E4M3, 1.0, v[h], v_dt, vs, o_dt, want_acc=True)
        assert o_scale == vs * kf_tk
        ok = within(O_gpu[h], Oo, o_dt, oacc, osab, 1e-5)
        assert ok.all(), (h, int((~ok).sum()))
    return O


@pytest.mark.parametrize("H,T", [(2, 128), (3, 256), (2, 1024)])
def test_causal_self_attention(H, T):
    run_case(H, T, T, True)


def test_full_attention_with_more_keys_than_queries():
    run_case(2, 128, 384, False)


def test_ragged_lengths_and_shifted_causal_mask():
    run_case(2, 200, 224, True)


@pytest.mark.parametrize("c", [-0.125, 0.3, 1.0])
def test_other_softmax_scales(c):
    """A positive scale takes the kernel's short form (scale folded into the multiply-add that subtracts the row
    maximum, 1/l folded into the exponent); a negative one the general form, in which the largest score is not
    the largest scaled score."""
    run_case(2, 200, 224, True, c=c)
    run_case(1, 128, 256, False, c=c, seed=5)


def test_heads_inside_a_token_major_buffer_and_mixed_formats():
    run_case(4, 256, 256, True, merged_layout=True, q_dt=orc.E5M2, v_dt=orc.E5M2, o_dt=orc.F16)


@pytest.mark.parametrize("H,Tq,Tk,causal", [(2, 128, 128, True), (3, 384, 384, True), (2, 200, 224, True),
                                            (2, 128, 384, False), (1, 1024, 1024, True)])
def test_head_dimension_128(H, Tq, Tk, causal):
    """Rows of 128 elements travel as two 64-byte column halves per tile: the scores accumulate over both, the
    output has 64 columns per half."""
    run_case(H, Tq, Tk, causal, HD=128, c=2.0 ** -3.5 if Tq == 200 else 0.125)


def test_head_dimension_128_at_48_heads_of_1024_tokens_sampled_heads():
    """8 sequences x 6 heads of 128: the model width of the benchmark's shape with the wider heads."""
    run_case(48, 1024, 1024, True, seed=13, check_heads=[0, 17, 47], HD=128)


def test_head_dimension_128_inside_a_token_major_buffer_and_mixed_formats():
    run_case(3, 256, 256, True, merged_layout=True, q_dt=orc.E5M2, v_dt=orc.E5M2, o_dt=orc.F16, HD=128)


def test_benchmark_shape_96_heads_of_1024_tokens_sampled_heads():
    """The shape the benchmark times (8 sequences x 12 heads): the first, the last and some middle heads
    against the oracle, and the launch without the debug copies gives the same output bit for bit."""
    H, T = 96, 1024
    O = run_case(H, T, T, True, seed=11, check_heads=[0, 1, 37, 73, 94, 95])
    q = si.to_bits(si.normal(11, 1, (H, T, HD), 1.0), orc.E4M3)
    k = si.to_bits(si.normal(11, 2, (H, T, HD), 1.0), orc.E4M3)
    v = si.to_bits(si.normal(11, 3, (H, T, HD), 1.0), orc.E4M3)
    Q, K, V = (sc.ScaledTensor.make(to_dev(x, orc.E4M3), s) for x, s in ((q, 0.5), (k, 2.0), (v, 0.125)))
    O2 = sc.ScaledTensor.empty((H, T, HD), torch.bfloat16)
    sc.scalify_scaled_attention(Q, K, V, O2, sm_scale=0.125, causal=True)
    assert O2.scale_value() == O.scale_value()
    assert torch.equal(O2.data.view(torch.int16), O.data.view(torch.int16))


def test_probabilities_sum_to_one_and_without_copies():
    H, T = 2, 384
    q = si.to_bits(si.normal(5, 1, (H, T, HD), 1.0), orc.E4M3)
    k = si.to_bits(si.normal(5, 2, (H, T, HD), 1.0), orc.E4M3)
    ones = si.to_bits(np.ones((H, T, HD), dtype=np.float32), orc.E4M3)
    Q, K, V = (sc.ScaledTensor.make(to_dev(x, orc.E4M3), 1.0) for x in (q, k, ones))
    O = sc.ScaledTensor.empty((H, T, HD), torch.float32)
    sc.scalify_scaled_attention(Q, K, V, O, sm_scale=0.125, causal=True)
    # V = 1 everywhere: O values = sum of the (E4M3-rounded) probabilities of each row, about 1
    vals = O.data.float().cpu().numpy() * O.scale_value()
    assert np.all(np.abs(vals - 1.0) < 0.08)


def test_argument_checks():
    Q = sc.ScaledTensor.make(torch.zeros((2, 128, 32), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn), 1.0)
    O = sc.ScaledTensor.empty((2, 128, 32), torch.bfloat16)
    with pytest.raises(sc.ScalifyError):
        sc.scalify_scaled_attention(Q, Q, Q, O, sm_scale=0.125)   # head dimension 32 is not built
    Q = sc.ScaledTensor.make(torch.zeros((2, 256, 64), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn), 1.0)
    K = sc.ScaledTensor.make(torch.zeros((2, 128, 64), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn), 1.0)
    O = sc.ScaledTensor.empty((2, 256, 64), torch.bfloat16)
    with pytest.raises(sc.ScalifyError):
        sc.scalify_scaled_attention(Q, K, K, O, sm_scale=0.125, causal=True)   # causal with fewer keys than queries


def test_batch_of_sequences_as_a_4d_view_equals_one_call_per_sequence():
    """[batch, heads, T, 64] views of token-major buffers [batch * T, heads * 64] (the layout the QKV projection
    writes): one call over the 4-D views must reproduce, bit for bit, one call per sequence; forward and backward."""
    B, H, T = 3, 4, 256
    d = H * HD
    g = torch.Generator(device="cuda").manual_seed(3)
    rnd = lambda dt: torch.randn((B * T, d), device="cuda", generator=g).to(dt)
    q, k, v, do = rnd(torch.float8_e4m3fn), rnd(torch.float8_e4m3fn), rnd(torch.float8_e4m3fn), rnd(torch.float8_e5m2)
    scales = (0.5, 2.0, 0.125, 2.0 ** -9)

    def views(x, b=None):   # [B, H, T, HD] view, or [H, T, HD] of sequence b
        x4 = x.view(B, T, H, HD).permute(0, 2, 1, 3)
        return x4 if b is None else x4[b]

    def run(batched):
        out = {n: torch.zeros((B * T, d), dtype=torch.bfloat16, device="cuda") for n in ("o", "dq", "dk", "dv")}
        sw = {n: torch.zeros(1, device="cuda") for n in ("o", "ds", "dq", "dk", "dv")}
        P = torch.zeros((B, H, T, T), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
        dS = torch.zeros((B, H, T, T), dtype=torch.uint8, device="cuda").view(torch.float8_e5m2)
        ones = torch.ones(1, device="cuda")
        for b in ([None] if batched else range(B)):
            Q, K, V, dO = (sc.ScaledTensor.make(views(x, b), s) for x, s in zip((q, k, v, do), scales))
            O, dQ, dK, dV = (sc.ScaledTensor(views(out[n], b), sw[n]) for n in ("o", "dq", "dk", "dv"))
            Pb = sc.ScaledTensor(P if b is None else P[b], ones)
            dSb = sc.ScaledTensor(dS if b is None else dS[b], sw["ds"])
            sc.scalify_scaled_attention(Q, K, V, O, sm_scale=0.125, causal=True, P_dump=Pb)
            sc.scalify_scaled_attention_bwd(Q, K, V, Pb, dO, dSb, dQ, dK, dV, sm_scale=0.125, causal=True)
        torch.cuda.synchronize()
        return ([out[n].view(torch.int16).cpu().numpy() for n in out] + [P.view(torch.uint8).cpu().numpy(),
                dS.view(torch.uint8).cpu().numpy()], [float(sw[n].item()) for n in sw])
    one, s_one = run(True)
    per, s_per = run(False)
    assert s_one == s_per
    for a, b in zip(one, per):
        assert np.array_equal(a, b)


def test_fp32_pipe_bf16_rounding_is_round_to_nearest_even():
    """The attention kernels round the scores (and dP) to BF16 with three fp32 operations instead of a
    conversion.  That routine against the definition (torch's CPU cast): every upper half-word with the tie
    pattern and its two neighbours below it, and sixteen million random bit patterns (normal numbers below 2^111,
    zero included; the products of FP8 operands are far inside that range)."""
    g = torch.Generator().manual_seed(7)
    upper = torch.arange(65536, dtype=torch.int64) << 16
    pats = [upper | low for low in (0x8000, 0x7FFF, 0x8001, 0x0000, 0xFFFF, 0x0001)]
    pats.append(torch.randint(0, 2 ** 32, (1 << 24,), generator=g, dtype=torch.int64))
    bits = torch.cat(pats)
    e = (bits >> 23) & 0xFF
    bits = bits[((e > 0) & (e < 0xFF - 20)) | ((bits & 0x7FFFFFFF) == 0)]
    x = (bits & 0xFFFFFFFF).to(torch.uint32).view(torch.float32).contiguous()
    want = x.to(torch.bfloat16).to(torch.float32)
    xd = x.cuda()
    for two_wide in (False, True):   # the scalar routine and the one on two-wide instructions (elements in pairs)
        yd = torch.empty_like(xd)
        sc.scalify_debug_bf16_round(xd, yd, two_wide=two_wide)
        got = yd.cpu()
        assert torch.equal(got.view(torch.int32), want.view(torch.int32)), two_wide
