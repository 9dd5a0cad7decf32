"""GPU parity of the scaled LayerNorm forward / backward kernels against the oracle.

Forward outputs: within 1 ulp of the output format (fp32 arithmetic on the GPU,
fp64 in the oracle), or, where the affine sum n*gamma + beta cancels, within
half an ulp plus 2e-6 of the magnitude of the two terms.  Backward: dx is a difference of terms of size |ghat|*rinv,
so its fp32 error is bounded relative to that magnitude, not to the (possibly
tiny) result: |gpu - oracle| <= 1 ulp(result) or <= 2^-18 * max|ghat|*rinv of
the row.  The fused statistic and the rescaled gradient are checked
stage-isolated against the oracle's rescale of the library's own dX.
"""
import math

import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu


def st(bits, dt, scale=None):
    t = to_dev(bits, dt)
    return sc.ScaledTensor.make(t, scale) if scale is not None else sc.ScaledTensor(t, None)


SHAPES = [(1, 8), (37, 768), (300, 1024), (5, 4096), (129, 2048), (64, 80)]


@pytest.mark.parametrize("R,d", SHAPES)
@pytest.mark.parametrize("x_dt,y_dt", [(orc.BF16, orc.BF16), (orc.BF16, orc.E4M3), (orc.F16, orc.F16),
                                       (orc.F32, orc.F32), (orc.F32, orc.BF16)])
@pytest.mark.parametrize("eps_inside", [False, True])
def test_layernorm_forward(R, d, x_dt, y_dt, eps_inside):
    if x_dt == orc.F32 and d > 2048:
        pytest.skip("row longer than the supported 8 KiB")
    c = si.layernorm_case(R, d, seed=41, x_dtype=x_dt)
    gs, bs = 2.0 ** -1, 2.0 ** 1
    Y = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[y_dt])
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(st(c["X"], x_dt, 2.0 ** 4), st(c["gamma"], orc.BF16, gs), st(c["beta"], orc.BF16, bs),
                                Y, eps=1e-5, eps_inside_sqrt=eps_inside, mean=mean, rinv=rinv)
    yo, ys, mo, ro = orc.layernorm_fwd(c["X"], x_dt, c["gamma"], orc.BF16, gs, c["beta"], orc.BF16, bs, 1e-5,
                                       eps_inside, y_dt)
    assert Y.scale_value() == ys == 2.0
    got = to_bits(Y.data, y_dt)
    # y = n*gamma*fg + beta*fb evaluated in fp32: error relative to the magnitude of the two terms
    n32, _, _, _ = orc.layernorm_fwd(c["X"], x_dt, None, 0, 1.0, None, 0, 1.0, 1e-5, eps_inside, orc.F32)
    nv = orc.decode(n32, orc.F32)
    mag = np.abs(nv * orc.decode(c["gamma"], orc.BF16) * (gs / ys)) + np.abs(orc.decode(c["beta"], orc.BF16) * (bs / ys))
    exact = nv * orc.decode(c["gamma"], orc.BF16) * (gs / ys) + orc.decode(c["beta"], orc.BF16) * (bs / ys)
    ok = within(got, yo, y_dt, exact, mag + 1e-3, 2e-6)
    assert ok.all(), int((~ok).sum())
    assert np.allclose(mean.cpu().numpy(), mo, rtol=0, atol=2e-6)
    assert np.allclose(rinv.cpu().numpy(), ro, rtol=2e-6)


def test_layernorm_forward_without_affine_constant_rows_and_strided_input():
    R, d = 50, 256
    x = si.scaled_normal(42, 1, (R, d), orc.BF16)
    x[7, :] = si.to_bits(np.full(d, 3.0, dtype=np.float32), orc.BF16)  # zero-variance row
    buf = torch.zeros((R, d + 64), dtype=torch.bfloat16, device="cuda")
    buf[:, :d].copy_(to_dev(x, orc.BF16))
    X = sc.ScaledTensor(buf[:, :d], None)
    Y = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    sc.scalify_scaled_layernorm(X, None, None, Y, eps=1e-5)
    yo, ys, _, _ = orc.layernorm_fwd(x, orc.BF16, None, 0, 1.0, None, 0, 1.0, 1e-5, False, orc.BF16)
    assert Y.scale_value() == 1.0
    got = to_bits(Y.data, orc.BF16)
    assert ulp_diff(got, yo, orc.BF16).max() <= 1
    assert np.all(orc.decode(got[7], orc.BF16) == 0.0)


@pytest.mark.parametrize("R,d", [(1, 8), (37, 768), (300, 1024), (5, 4096), (1000, 768), (64, 80)])
@pytest.mark.parametrize("eps_inside", [False, True])
@pytest.mark.parametrize("stat", [sc.STAT_L2, sc.STAT_AMAX])
def test_layernorm_backward_with_gradient_rescale(R, d, eps_inside, stat):
    c = si.layernorm_case(R, d, seed=43)
    x_s, g_s, gam_s = 2.0 ** 2, 2.0 ** -10, 2.0 ** -1
    X, G, gamma = st(c["X"], orc.BF16, x_s), st(c["G"], orc.BF16, g_s), st(c["gamma"], orc.BF16, gam_s)
    Y = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, st(c["beta"], orc.BF16, 1.0), Y, eps=1e-5, eps_inside_sqrt=eps_inside,
                                mean=mean, rinv=rinv)
    dX = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    dXq = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
    dg = sc.ScaledTensor.empty((d,), torch.float32)
    db = sc.ScaledTensor.empty((d,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws, eps=1e-5, eps_inside_sqrt=eps_inside,
                                    stat_dx=stat, dXq=dXq, dgamma=dg, dbeta=db)
    assert ws.check_status() == 0
    o = orc.layernorm_bwd(c["G"], orc.BF16, g_s, c["X"], orc.BF16, x_s, c["gamma"], orc.BF16, gam_s, 1e-5,
                          eps_inside, orc.BF16, orc.F32, want_f64=True)
    assert dX.scale_value() == o["dX_scale"]
    assert dg.scale_value() == o["dgamma_scale"] and db.scale_value() == o["dbeta_scale"]
    got = to_bits(dX.data, orc.BF16)
    gv = orc.decode(c["G"], orc.BF16) * orc.decode(c["gamma"], orc.BF16)[None, :]
    _, _, _, ro = orc.layernorm_fwd(c["X"], orc.BF16, None, 0, 1.0, None, 0, 1.0, 1e-5, eps_inside, orc.BF16)
    row_mag = np.abs(gv).max(axis=1) * ro
    ok = within(got, o["dX"], orc.BF16, o["dx_f64"], row_mag[:, None], 2.0 ** -18)
    assert ok.all(), int((~ok).sum())
    # dgamma / dbeta: fp32 column sums, error relative to the sum of magnitudes
    n, _, _, _ = orc.layernorm_fwd(c["X"], orc.BF16, None, 0, 1.0, None, 0, 1.0, 1e-5, eps_inside, orc.F32)
    nv = orc.decode(n, orc.F32)
    Gd = orc.decode(c["G"], orc.BF16)
    f = orc.kf(R)
    mag_g = np.abs(Gd * nv).sum(axis=0) / f
    mag_b = np.abs(Gd).sum(axis=0) / f
    got_dg = orc.decode(to_bits(dg.data, orc.F32), orc.F32)
    got_db = orc.decode(to_bits(db.data, orc.F32), orc.F32)
    assert np.all(np.abs(got_dg - (Gd * nv).sum(axis=0) / f) <= 2e-5 * mag_g + 1e-30)
    assert np.all(np.abs(got_db - Gd.sum(axis=0) / f) <= 2e-5 * mag_b + 1e-30)
    # statistic and rescaled gradient, stage-isolated on the library's own dX
    so = orc.statistic(got, orc.BF16, stat)
    gstat = float(ws.statistic().item())
    if stat == sc.STAT_AMAX:
        assert gstat == so
    else:
        assert abs(gstat - so) <= 2e-6 * so
        if abs(math.log2(so) - round(math.log2(so))) < 1e-5:
            return
    qo, qs, _ = orc.rescale(got, orc.BF16, o["dX_scale"], stat, orc.E5M2)
    assert dXq.scale_value() == qs
    assert np.array_equal(to_bits(dXq.data, orc.E5M2), qo)


@pytest.mark.parametrize("R,d", [(1, 8), (37, 768), (300, 1024), (5, 4096), (1000, 768), (64, 80), (700, 4096)])
@pytest.mark.parametrize("dx_dt", [orc.E5M2, orc.E4M3, orc.BF16])
@pytest.mark.parametrize("stat,stat_in", [(sc.STAT_L2, 2.0 ** -7 * 1.3), (sc.STAT_AMAX, 0.011), (sc.STAT_AMAX, 0.0),
                                          (sc.STAT_L2, float("inf"))])
def test_layernorm_backward_with_delayed_rescale(R, d, dx_dt, stat, stat_in):
    """One pass: the gradient is written already divided by the power of two of an EARLIER statistic
    (Section 3.3), rounded once from fp32, and this step's statistic is that of the un-rebalanced values.
    Bar: the plain backward's bar (1 ulp of the output format, or half an ulp plus 2^-18 of the row's
    largest term), scale words exact, statistic 2e-6 relative (L2) or 2^-18 of the largest term (AMAX)."""
    from helpers import layernorm_bwd_delayed, ulp_of
    c = si.layernorm_case(R, d, seed=47)
    x_s, g_s, gam_s = 2.0 ** 2, 2.0 ** -10, 2.0 ** -1
    X, G, gamma = st(c["X"], orc.BF16, x_s), st(c["G"], orc.BF16, g_s), st(c["gamma"], orc.BF16, gam_s)
    Y = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, st(c["beta"], orc.BF16, 1.0), Y, eps=1e-5, mean=mean, rinv=rinv)
    dX = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[dx_dt])
    dg, db = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    # the earlier statistic sits in the word this call overwrites with its own (the state of a training loop)
    ws.statistic().fill_(stat_in)
    sc.scalify_scaled_layernorm_bwd_delayed(G, X, gamma, mean, rinv, ws.statistic(), dX, ws, eps=1e-5, stat_dx=stat,
                                            dgamma=dg, dbeta=db)
    assert ws.check_status() == 0
    o = layernorm_bwd_delayed(c["G"], orc.BF16, g_s, c["X"], orc.BF16, x_s, c["gamma"], orc.BF16, gam_s, 1e-5, False,
                              stat_in, stat, dx_dt, orc.F32)
    assert dX.scale_value() == o["dX_scale"]
    assert dg.scale_value() == o["dgamma_scale"] and db.scale_value() == o["dbeta_scale"]
    got = to_bits(dX.data, dx_dt)
    gv = orc.decode(c["G"], orc.BF16) * orc.decode(c["gamma"], orc.BF16)[None, :]
    _, _, _, ro = orc.layernorm_fwd(c["X"], orc.BF16, None, 0, 1.0, None, 0, 1.0, 1e-5, False, orc.BF16)
    row_mag = np.abs(gv).max(axis=1) * ro / o["r"]
    exact = o["dx_f64"] / o["r"]
    ok = within(got, o["dX"], dx_dt, exact, row_mag[:, None], 2.0 ** -18)
    assert ok.all(), int((~ok).sum())
    gstat = float(ws.statistic().item())
    if stat == sc.STAT_AMAX:
        assert abs(gstat - o["stat"]) <= 2.0 ** -18 * (row_mag.max() * o["r"])
    else:
        assert abs(gstat - o["stat"]) <= 2e-6 * o["stat"]
    # dgamma / dbeta do not depend on the rescale
    plain_dg, plain_db = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
    dX2 = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX2, ws, eps=1e-5, stat_dx=stat, dgamma=plain_dg,
                                    dbeta=plain_db)
    assert torch.equal(plain_dg.data, dg.data) and torch.equal(plain_db.data, db.data)


def test_layernorm_backward_delayed_argument_checks():
    R, d = 8, 64
    X = sc.ScaledTensor.make(torch.zeros((R, d), dtype=torch.bfloat16, device="cuda"), 1.0)
    dX = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
    mean = torch.zeros(R, device="cuda")
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    with pytest.raises(sc.ScalifyError):   # the plain call keeps a wide gradient
        sc.scalify_scaled_layernorm_bwd(X, X, None, mean, mean, dX, ws)
    with pytest.raises(sc.ScalifyError):   # no earlier statistic
        sc.scalify_scaled_layernorm_bwd_delayed(X, X, None, mean, mean, None, dX, ws)


@pytest.mark.parametrize("R,d", [(37, 768), (300, 1024), (3, 16)])
@pytest.mark.parametrize("x_dt,dx_dt", [(orc.F32, orc.E5M2), (orc.F32, orc.F32), (orc.F16, orc.E4M3), (orc.F16, orc.F16)])
def test_layernorm_backward_delayed_other_input_formats(R, d, x_dt, dx_dt):
    """fp32 and fp16 inputs (4 or 8 elements per 16-byte vector, so FP8 rows are written 4 or 8 bytes at a time)."""
    from helpers import layernorm_bwd_delayed, ulp_of
    Xb = si.scaled_normal(48, 1, (R, d), x_dt)
    Gb = si.scaled_normal(48, 4, (R, d), x_dt)
    gam = si.to_bits(1.0 + 0.1 * si.normal(48, 2, (d,)), orc.BF16)
    x_s, g_s, gam_s, stat_in = 2.0 ** -2, 2.0 ** -10, 1.0, 0.37
    X, G, gamma = st(Xb, x_dt, x_s), st(Gb, x_dt, g_s), st(gam, orc.BF16, gam_s)
    Y = sc.ScaledTensor.empty((R, d), torch.float32)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, None, Y, eps=1e-5, eps_inside_sqrt=True, mean=mean, rinv=rinv)
    dX = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[dx_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    state = torch.full((1,), stat_in, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm_bwd_delayed(G, X, gamma, mean, rinv, state, dX, ws, eps=1e-5, eps_inside_sqrt=True,
                                            stat_dx=sc.STAT_AMAX)
    assert ws.check_status() == 0 and float(state.item()) == np.float32(stat_in)   # a separate state word is only read
    o = layernorm_bwd_delayed(Gb, x_dt, g_s, Xb, x_dt, x_s, gam, orc.BF16, gam_s, 1e-5, True, stat_in, orc.STAT_AMAX,
                              dx_dt, orc.F32)
    assert o["r"] == 0.25 and dX.scale_value() == o["dX_scale"]
    got = to_bits(dX.data, dx_dt)
    gv = orc.decode(Gb, x_dt) * orc.decode(gam, orc.BF16)[None, :]
    _, _, _, ro = orc.layernorm_fwd(Xb, x_dt, None, 0, 1.0, None, 0, 1.0, 1e-5, True, orc.F32)
    row_mag = np.abs(gv).max(axis=1) * ro / o["r"]
    exact = o["dx_f64"] / o["r"]
    ok = within(got, o["dX"], dx_dt, exact, row_mag[:, None], 2.0 ** -18)
    assert ok.all(), int((~ok).sum())
    assert abs(float(ws.statistic().item()) - o["stat"]) <= 2.0 ** -18 * (row_mag.max() * o["r"])


ONE_PASS_SHAPES = [(37, 768), (300, 1024), (5, 4096), (1000, 768), (64, 80), (9000, 2048)]


@pytest.mark.parametrize("R,d", ONE_PASS_SHAPES)
@pytest.mark.parametrize("stat", [sc.STAT_L2, sc.STAT_AMAX])
@pytest.mark.parametrize("x_dt,q_dt", [(orc.BF16, orc.E5M2), (orc.F16, orc.E4M3), (orc.F32, orc.E5M2)])
def test_one_pass_gradient_rescale_is_bit_identical_to_the_two_pass_call(R, d, stat, x_dt, q_dt):
    """dX = None: the rebalanced gradient is written in one pass with the power of two predicted from the
    statistic this workspace saw last, and written again only if the prediction failed.  Whatever the
    prediction word holds - nothing (first call), the right statistic, one with another power of two, infinity,
    NaN - the rebalanced data, its scale word, the statistic word, dgamma and dbeta are those of the two-pass
    call (which is compared with the oracle elsewhere in this file) bit for bit."""
    if x_dt == orc.F32 and d * 4 > 8192:
        pytest.skip("fp32 rows longer than 8 KiB are not supported by the LayerNorm kernels")
    c = si.layernorm_case(R, d, seed=47)
    spread = 6 if x_dt == orc.F16 else 10
    cast = lambda b: si.to_bits(orc.decode(b, orc.BF16).astype(np.float32), x_dt)
    x_s, gam_s = 2.0 ** 2, 2.0 ** -1
    X, gamma = st(cast(c["X"]), x_dt, x_s), st(c["gamma"], orc.BF16, gam_s)
    Y = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[x_dt])
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, st(c["beta"], orc.BF16, 1.0), Y, mean=mean, rinv=rinv)
    ws1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    ws2 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    g_bits = cast(c["G"])
    g_val = orc.decode(g_bits, x_dt).astype(np.float32)
    steps = [(1.0, None), (1.0, None), (2.0 ** spread, None), (2.0 ** -spread, None), (1.0, float("inf")),
             (1.0, float("nan")), (1.3, None), (1.0, 0.0)]
    for mult, hint in steps:
        G = st(si.to_bits(g_val * np.float32(mult), x_dt), x_dt, 2.0 ** -10)
        dX = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[x_dt])
        q2 = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[q_dt])
        dg2, db2 = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
        sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws2, stat_dx=stat, dXq=q2, dgamma=dg2, dbeta=db2)
        q1 = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[q_dt])
        q1.data.view(torch.uint8).fill_(0x55)
        dg1, db1 = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
        if hint is not None:
            ws1.prediction().fill_(hint)
        sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, None, ws1, stat_dx=stat, dXq=q1, dgamma=dg1, dbeta=db1)
        assert ws1.check_status() == 0 and ws2.check_status() == 0
        tag = (mult, hint)
        assert torch.equal(ws1.statistic().view(torch.int32), ws2.statistic().view(torch.int32)), tag
        assert q1.scale_value() == q2.scale_value(), tag
        assert torch.equal(q1.data.view(torch.uint8), q2.data.view(torch.uint8)), tag
        assert dg1.scale_value() == dg2.scale_value() and db1.scale_value() == db2.scale_value()
        assert torch.equal(dg1.data.view(torch.int32), dg2.data.view(torch.int32)), tag
        assert torch.equal(db1.data.view(torch.int32), db2.data.view(torch.int32)), tag
        # the call leaves its own statistic as the next prediction
        assert torch.equal(ws1.prediction().view(torch.int32), ws1.statistic().view(torch.int32)), tag


@pytest.mark.parametrize("with_gamma,with_dgamma", [(False, False), (True, False), (False, True)])
def test_one_pass_gradient_rescale_without_gamma_or_column_sums(with_gamma, with_dgamma):
    R, d = 77, 512
    c = si.layernorm_case(R, d, seed=49)
    X, G = st(c["X"], orc.BF16, 2.0), st(c["G"], orc.BF16, 2.0 ** -7)
    gamma = st(c["gamma"], orc.BF16, 0.5) if with_gamma else None
    Y = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, st(c["beta"], orc.BF16, 1.0) if with_gamma else None, Y, mean=mean, rinv=rinv)
    outs = []
    for one_pass in (False, True):
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
        dX = None if one_pass else sc.ScaledTensor.empty((R, d), torch.bfloat16)
        q = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
        dg = sc.ScaledTensor.empty((d,), torch.float32) if with_dgamma else None
        db = sc.ScaledTensor.empty((d,), torch.float32) if with_dgamma else None
        for _ in range(2):   # without and with a prediction
            sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws, stat_dx=sc.STAT_AMAX, dXq=q, dgamma=dg, dbeta=db)
        assert ws.check_status() == 0
        outs.append((q.data.view(torch.uint8).clone(), q.scale_value(), float(ws.statistic().item()),
                     None if dg is None else dg.data.clone(), None if db is None else db.data.clone()))
    a, b = outs
    assert torch.equal(a[0], b[0]) and a[1] == b[1] and a[2] == b[2]
    if with_dgamma:
        assert torch.equal(a[3], b[3]) and torch.equal(a[4], b[4])


def test_one_pass_gradient_rescale_argument_checks():
    R, d = 16, 256
    z = lambda dt: sc.ScaledTensor.make(torch.zeros((R, d), device="cuda").to(dt), 1.0)
    G, X = z(torch.bfloat16), z(torch.bfloat16)
    mean, rinv = torch.zeros(R, device="cuda"), torch.ones(R, device="cuda")
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    with pytest.raises(sc.ScalifyError):   # nothing to write
        sc.scalify_scaled_layernorm_bwd(G, X, None, mean, rinv, None, ws, stat_dx=sc.STAT_AMAX)
    with pytest.raises(sc.ScalifyError):   # the one-pass form writes FP8
        sc.scalify_scaled_layernorm_bwd(G, X, None, mean, rinv, None, ws, stat_dx=sc.STAT_AMAX, dXq=z(torch.bfloat16))
    with pytest.raises(sc.ScalifyError):   # a dynamic rescale needs a statistic
        sc.scalify_scaled_layernorm_bwd(G, X, None, mean, rinv, None, ws, stat_dx=sc.STAT_NONE,
                                        dXq=z(torch.float8_e5m2))
