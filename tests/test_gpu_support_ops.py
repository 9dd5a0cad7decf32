"""GPU parity of the support kernels of a GPT-style step (embedding, causal softmax, cross-entropy)
against the oracle.  fp32 on the GPU, fp64 in the oracle: outputs within 1 ulp of the output format,
or, for sums that cancel, within half an ulp plus a small multiple of the magnitude of the terms."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu


def ST(bits, dt, scale):
    return sc.ScaledTensor.make(to_dev(bits, dt), scale)


@pytest.mark.parametrize("V,T,d,B", [(50, 8, 16, 3), (1000, 64, 768, 4), (50257, 128, 768, 2)])
@pytest.mark.parametrize("w_dt,y_dt", [(orc.F16, orc.BF16), (orc.BF16, orc.BF16), (orc.F32, orc.F32)])
def test_embedding_forward(V, T, d, B, w_dt, y_dt):
    n = B * T
    ids = si.uniform_int(71, 1, (n,), V)
    wte = si.to_bits(si.normal(71, 2, (V, d), 0.02 * 64), w_dt)
    wpe = si.to_bits(si.normal(71, 3, (T, d), 0.02 * 64), w_dt)
    Y = sc.ScaledTensor.empty((n, d), sc.TORCH_DTYPE[y_dt])
    sc.scalify_scaled_embedding(torch.from_numpy(ids).cuda(), T, ST(wte, w_dt, 2.0 ** -6), ST(wpe, w_dt, 2.0 ** -7), Y)
    yo, ys = orc.embedding_fwd(ids, T, wte, w_dt, 2.0 ** -6, wpe, w_dt, 2.0 ** -7, y_dt)
    assert Y.scale_value() == ys
    assert ulp_diff(to_bits(Y.data, y_dt), yo, y_dt).max() <= 1
    # without positions, and an out-of-range id is reported
    Y2 = sc.ScaledTensor.empty((n, d), sc.TORCH_DTYPE[y_dt])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad = ids.copy()
    bad[0] = V + 5
    sc.scalify_scaled_embedding(torch.from_numpy(bad).cuda(), T, ST(wte, w_dt, 2.0 ** -6), None, Y2, status=status)
    assert int(status.item()) == sc.DEV_BAD_INDEX
    yo2, ys2 = orc.embedding_fwd(ids[1:], 1, wte, w_dt, 2.0 ** -6, None, 0, 1.0, y_dt)
    assert Y2.scale_value() == ys2 and np.array_equal(to_bits(Y2.data, y_dt)[1:], yo2)


@pytest.mark.parametrize("V,T,d,B", [(50, 8, 16, 3), (997, 64, 768, 4)])
def test_embedding_backward(V, T, d, B):
    n = B * T
    ids = si.uniform_int(72, 1, (n,), V)
    ids[: n // 4] = 7  # a heavily repeated token
    dY = si.scaled_normal(72, 2, (n, d), orc.BF16)
    dwte = sc.ScaledTensor.empty((V, d), torch.float32)
    dwpe = sc.ScaledTensor.empty((T, d), torch.float32)
    dwte.data.fill_(123.0)  # the call overwrites the whole table
    sc.scalify_scaled_embedding_bwd(torch.from_numpy(ids).cuda(), T, ST(dY, orc.BF16, 2.0 ** -10), dwte, dwpe)
    to, s1, po, s2 = orc.embedding_bwd(ids, T, V, dY, orc.BF16, 2.0 ** -10, orc.F32)
    assert dwte.scale_value() == s1 and dwpe.scale_value() == s2
    g = np.abs(orc.decode(dY, orc.BF16))
    mag_t = np.zeros((V, d))
    np.add.at(mag_t, ids, g)
    got_t = orc.decode(to_bits(dwte.data, orc.F32), orc.F32)
    assert np.all(np.abs(got_t - orc.decode(to, orc.F32)) <= 2e-6 * mag_t + 1e-30)
    got_p = orc.decode(to_bits(dwpe.data, orc.F32), orc.F32)
    mag_p = g.reshape(B, T, d).sum(0) / orc.kf(B)
    assert np.all(np.abs(got_p - orc.decode(po, orc.F32)) <= 2e-6 * mag_p + 1e-30)


@pytest.mark.parametrize("shape", [(3, 12, 16), (2, 128, 128), (5, 64, 1024), (1, 4, 48)])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("s_dt,p_dt", [(orc.BF16, orc.E4M3), (orc.BF16, orc.BF16), (orc.F32, orc.F32)])
def test_softmax_forward(shape, causal, s_dt, p_dt):
    S = si.scaled_normal(73, 1, shape, s_dt, 2.0)
    P = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[p_dt])
    sc.scalify_scaled_softmax(ST(S, s_dt, 2.0 ** -1), P, causal=causal)
    po, ps = orc.softmax_fwd(S, s_dt, 2.0 ** -1, causal, p_dt)
    assert P.scale_value() == ps == 1.0
    got = to_bits(P.data, p_dt)
    if p_dt == orc.F32:
        g, w = orc.decode(got, p_dt), orc.decode(po, p_dt)
        assert np.all(np.abs(g - w) <= 4e-6 * w + 1e-12)
    else:
        assert ulp_diff(got, po, p_dt).max() <= 1
    if causal:
        Tq, Tk = shape[-2], shape[-1]
        mask = np.triu(np.ones((Tq, Tk), dtype=bool), Tk - Tq + 1)
        assert np.all(orc.decode(got, p_dt)[..., mask] == 0.0)


@pytest.mark.parametrize("shape", [(3, 12, 16), (2, 128, 128), (2, 64, 1024)])
@pytest.mark.parametrize("p_dt,o_dt", [(orc.E4M3, orc.BF16), (orc.BF16, orc.BF16), (orc.BF16, orc.E5M2)])
def test_softmax_backward(shape, p_dt, o_dt):
    S = si.scaled_normal(74, 1, shape, orc.BF16, 2.0)
    po, _ = orc.softmax_fwd(S, orc.BF16, 1.0, True, p_dt)
    dP = si.scaled_normal(74, 2, shape, orc.BF16)
    dS = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[o_dt])
    sc.scalify_scaled_softmax_bwd(ST(dP, orc.BF16, 2.0 ** -10), ST(po, p_dt, 1.0), dS)
    so, ss = orc.softmax_bwd(dP, orc.BF16, 2.0 ** -10, po, p_dt, 1.0, o_dt)
    assert dS.scale_value() == ss == 2.0 ** -10
    pv, gv = orc.decode(po, p_dt), orc.decode(dP, orc.BF16)
    dot = (pv * gv).sum(-1, keepdims=True)
    exact = pv * (gv - dot)
    mag = pv * (np.abs(gv) + np.abs(pv * gv).sum(-1, keepdims=True))
    assert within(to_bits(dS.data, o_dt), so, o_dt, exact, mag, 4e-6).all()


@pytest.mark.parametrize("n,V,ld", [(16, 37, 48), (12, 1000, 1008), (64, 50257, 50304), (700, 1000, 1008),
                                    (901, 4099, 4112)])
@pytest.mark.parametrize("g_dt", [orc.BF16, orc.E5M2, orc.F32])
def test_cross_entropy_and_gradient(n, V, ld, g_dt):
    # (the last two cases give every block several rows: the next row is copied in behind the current one)
    logits = si.scaled_normal(75, 1, (n, ld), orc.BF16, 3.0)
    tgt = si.uniform_int(75, 2, (n,), V)
    L = ST(logits, orc.BF16, 2.0 ** -1)
    G = sc.ScaledTensor.empty((n, ld), sc.TORCH_DTYPE[g_dt])
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_CROSS_ENTROPY, n))
    sc.scalify_scaled_cross_entropy(L, V, torch.from_numpy(tgt).cuda(), loss, G, ws)
    assert ws.check_status() == 0
    lo, go, gs = orc.cross_entropy(logits, orc.BF16, 2.0 ** -1, V, tgt, g_dt)
    assert abs(float(loss.item()) - lo) <= 2e-6 * abs(lo) + 1e-6
    assert G.scale_value() == gs
    got = to_bits(G.data, g_dt)
    exact64, _, _ = (None, None, None)
    _, g64, _ = orc.cross_entropy(logits, orc.BF16, 2.0 ** -1, V, tgt, orc.F32)
    exact = orc.decode(g64, orc.F32)
    assert within(got, go, g_dt, exact, np.abs(exact) + 1e-6, 8e-6).all()
    assert np.all(orc.decode(got, g_dt)[:, V:] == 0.0)
    # the loss alone (no gradient written) is the same number
    loss2 = torch.zeros(1, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_cross_entropy(L, V, torch.from_numpy(tgt).cuda(), loss2, None, ws)
    assert ws.check_status() == 0 and float(loss2.item()) == float(loss.item())
    # out-of-range target is reported
    bad = tgt.copy()
    bad[1] = V
    sc.scalify_scaled_cross_entropy(L, V, torch.from_numpy(bad).cuda(), loss, None, ws)
    assert ws.check_status() == sc.DEV_BAD_INDEX


@pytest.mark.parametrize("R,N,x_dt,y_dt", [(8192, 768, orc.E5M2, orc.BF16), (8192, 3072, orc.E5M2, orc.F32),
                                          (1000, 50, orc.BF16, orc.BF16), (37, 1030, orc.E4M3, orc.F16),
                                          (5, 24, orc.F32, orc.F32), (70000, 64, orc.F16, orc.F32)])
def test_column_sums(R, N, x_dt, y_dt):
    """The reduce-sum rule is the matmul rule with a ones operand and K = R: the oracle's scaled matmul of
    [1, R] ones with X is the definition.  Bar: 1 ulp of the output format, or half an ulp plus
    1e-5 * sum|x| (fp32 partial sums)."""
    ld = (N // 16 + 2) * 16                                          # a padded, 16-byte-aligned row stride
    full = si.to_bits(si.normal(91, R, (R, ld), 1.0), x_dt)
    x = np.ascontiguousarray(full[:, :N])
    X = sc.ScaledTensor.make(to_dev(full, x_dt)[:, :N], 2.0 ** -7)
    Y = sc.ScaledTensor.empty((N,), sc.TORCH_DTYPE[y_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N))
    sc.scalify_scaled_colsum(X, Y, ws)
    assert ws.check_status() == 0
    xv = orc.decode(x, x_dt)
    kf = orc.kf(R)
    exact = xv.sum(axis=0) / kf
    mag = np.abs(xv).sum(axis=0) / kf
    want = orc.encode(exact, y_dt)
    assert Y.scale_value() == 2.0 ** -7 * kf
    ok = within(to_bits(Y.data, y_dt), want, y_dt, exact, mag, 1e-5)
    assert ok.all(), int((~ok).sum())
    if x_dt in (orc.E4M3, orc.E5M2) and R <= 8192:
        # the same numbers from the oracle's matmul with a ones operand
        ones = si.to_bits(np.ones((1, R), dtype=np.float32), orc.E4M3)
        yo, ys = orc.scaled_matmul(ones, orc.E4M3, 1.0, x, x_dt, 2.0 ** -7, y_dt)[:2]
        assert ys == 2.0 ** -7 * kf and np.array_equal(yo.reshape(-1), want)
    # deterministic: a second call gives the same bits
    Y2 = sc.ScaledTensor.empty((N,), sc.TORCH_DTYPE[y_dt])
    sc.scalify_scaled_colsum(X, Y2, ws)
    assert np.array_equal(to_bits(Y2.data, y_dt), to_bits(Y.data, y_dt))


@pytest.mark.parametrize("R,N,x_dt,c_dt,y_dt", [(8192, 768, orc.BF16, orc.E5M2, orc.BF16), (8192, 3072, orc.BF16, orc.E5M2, orc.F32),
                                               (1000, 50, orc.F16, orc.E4M3, orc.BF16), (37, 1030, orc.BF16, orc.E4M3, orc.F16),
                                               (5, 24, orc.BF16, orc.E5M2, orc.F32), (70000, 64, orc.F16, orc.E5M2, orc.F32)])
def test_cast_fused_with_column_sums(R, N, x_dt, c_dt, y_dt):
    """One pass over a 16-bit gradient: its FP8 cast (the oracle's encoding of every element, scale unchanged)
    and the column sums of the CAST values by the reduce-sum rule - against the oracle, and bit for bit what the
    plain cast followed by the column sums of its output gives."""
    ld = (N // 16 + 2) * 16
    spread = 40.0 if c_dt == orc.E5M2 else 4.0
    full = si.to_bits(si.normal(93, R, (R, ld), spread), x_dt)
    x = np.ascontiguousarray(full[:, :N])
    X = sc.ScaledTensor.make(to_dev(full, x_dt)[:, :N], 2.0 ** -9)
    cbuf = torch.zeros((R, ld), dtype=torch.uint8, device="cuda").view(sc.TORCH_DTYPE[c_dt])
    cbuf.view(torch.uint8).fill_(0x55)
    C = sc.ScaledTensor(cbuf[:, :N], torch.zeros(1, device="cuda"))
    Y = sc.ScaledTensor.empty((N,), sc.TORCH_DTYPE[y_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N))
    sc.scalify_scaled_cast_colsum(X, C, Y, ws)
    assert ws.check_status() == 0
    # the cast: every element the oracle's encoding, the padding columns untouched
    want_c = orc.encode(orc.decode(x, x_dt), c_dt)
    got_c = to_bits(cbuf, c_dt)
    assert np.array_equal(got_c[:, :N], want_c) and np.all(got_c[:, N:] == 0x55)
    assert C.scale_value() == 2.0 ** -9
    # the sums: of the cast values
    cv = orc.decode(want_c, c_dt)
    kf = orc.kf(R)
    exact, mag = cv.sum(axis=0) / kf, np.abs(cv).sum(axis=0) / kf
    assert Y.scale_value() == 2.0 ** -9 * kf
    ok = within(to_bits(Y.data, y_dt), orc.encode(exact, y_dt), y_dt, exact, mag, 1e-5)
    assert ok.all(), int((~ok).sum())
    # the same bits as the two separate calls
    Xc = sc.ScaledTensor.make(to_dev(x, x_dt), 2.0 ** -9)
    Cc = sc.ScaledTensor.empty((R, N), sc.TORCH_DTYPE[c_dt]) if N % 16 == 0 else None
    if Cc is not None:
        sc.scalify_rescale(Xc, Cc)
        Y2 = sc.ScaledTensor.empty((N,), sc.TORCH_DTYPE[y_dt])
        sc.scalify_scaled_colsum(Cc, Y2, ws)
        assert np.array_equal(to_bits(Cc.data, c_dt), want_c)
        assert Y2.scale_value() == Y.scale_value()
        assert np.array_equal(to_bits(Y2.data, y_dt), to_bits(Y.data, y_dt))


def test_cast_colsum_argument_checks():
    R, N = 64, 128
    X = sc.ScaledTensor.make(torch.zeros((R, N), dtype=torch.bfloat16, device="cuda"), 1.0)
    C = sc.ScaledTensor.empty((R, N), torch.float8_e5m2)
    Y = sc.ScaledTensor.empty((N,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N))
    sc.scalify_scaled_cast_colsum(X, C, Y, ws)
    with pytest.raises(sc.ScalifyError):   # the input is a 16-bit gradient
        sc.scalify_scaled_cast_colsum(sc.ScaledTensor.make(torch.zeros((R, N), device="cuda"), 1.0), C, Y, ws)
    with pytest.raises(sc.ScalifyError):   # the cast goes to FP8
        sc.scalify_scaled_cast_colsum(X, sc.ScaledTensor.empty((R, N), torch.bfloat16), Y, ws)
    with pytest.raises(sc.ScalifyError):   # shapes
        sc.scalify_scaled_cast_colsum(X, sc.ScaledTensor.empty((R, N + 16), torch.float8_e5m2), Y, ws)
    with pytest.raises(sc.ScalifyError):   # a scale word of its own
        sc.scalify_scaled_cast_colsum(X, sc.ScaledTensor(C.data, X.scale), Y, ws)
