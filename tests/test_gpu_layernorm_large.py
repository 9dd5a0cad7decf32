"""LayerNorm parity on the launch shapes that the benchmark and the GPT-shaped step use.

The small shapes of test_gpu_layernorm.py run one row per team of warps; the shapes here make every
team walk several rows (forward: its block's run of consecutive rows, with the shared-memory row
ring refilled and wrapping; backward: the persistent grid's stride loop over hundreds of rows, with
the register prefetch or, for long rows, the staged ring wrapping).  Each test first asserts, from
the library's own launch plan, that the shape reaches that path.

Everything is compared in full, in chunks of rows: Y / dX element by element under the bars of the
small cases, mean and 1/sigma, dgamma and dbeta against fp64 column sums, the statistic word, every
scale word, and the rescaled gradient bit for bit against the oracle's rescale of the library's own
dX (stage isolation).
"""
import math

import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, ulp_of, within

pytestmark = pytest.mark.gpu

BF = orc.BF16
CHUNK = 8192
EPS = 1e-5


def st(bits, dt, scale=None):
    t = to_dev(bits, dt)
    return sc.ScaledTensor.make(t, scale) if scale is not None else sc.ScaledTensor(t, None)


def chunks(R):
    for r0 in range(0, R, CHUNK):
        yield r0, min(R, r0 + CHUNK)


# (R, d, y dtype, least number of rows a team must walk)
FWD_CASES = [
    (131072, 1024, BF, 5),          # the benchmark's shape: 6 rows per team, the 4-slot ring wraps
    (131072, 1024, orc.E4M3, 5),    # the FP8-output form (operand of the next matmul)
    (8192, 768, BF, 1),             # configs 3 and 5
    (8192, 768, orc.E4M3, 1),
    (16384, 256, BF, 2),            # one warp per row, eight teams per block
    (65536, 768, BF, 5),
    (16384, 4096, BF, 5),           # four vectors per thread, four warps per row
    (20000, 1000, BF, 2),           # ragged: rows that end inside a block's run, a row that is not a whole number of warps
]


@pytest.mark.parametrize("R,d,y_dt,min_rows", FWD_CASES)
def test_layernorm_forward_on_benchmarked_launch_shapes(R, d, y_dt, min_rows):
    plan = sc.scalify_debug_layernorm_plan(R, d, BF, False)
    assert plan["rows_per_team"] >= min_rows, plan
    if min_rows >= 5:
        assert plan["rows_per_team"] > plan["stages"], plan      # a ring slot is refilled and read again
    c = si.layernorm_case(R, d, seed=51)
    gs, bs = 2.0 ** -1, 2.0 ** 1
    Y = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[y_dt])
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(st(c["X"], BF, 2.0 ** 4), st(c["gamma"], BF, gs), st(c["beta"], BF, bs), Y, eps=EPS,
                                mean=mean, rinv=rinv)
    got = to_bits(Y.data, y_dt)
    gm, gr = mean.cpu().numpy(), rinv.cpu().numpy()
    assert Y.scale_value() == 2.0
    gv = orc.decode(c["gamma"], BF) * (gs / 2.0)
    bv = orc.decode(c["beta"], BF) * (bs / 2.0)
    for r0, r1 in chunks(R):
        Xc = c["X"][r0:r1]
        yo, ys, mo, ro = orc.layernorm_fwd(Xc, BF, c["gamma"], BF, gs, c["beta"], BF, bs, EPS, False, y_dt)
        assert ys == 2.0
        n32, _, _, _ = orc.layernorm_fwd(Xc, BF, None, 0, 1.0, None, 0, 1.0, EPS, False, orc.F32)
        nv = orc.decode(n32, orc.F32)
        exact = nv * gv + bv
        ok = within(got[r0:r1], yo, y_dt, exact, np.abs(nv * gv) + np.abs(bv) + 1e-3, 2e-6)
        assert ok.all(), (r0, int((~ok).sum()))
        assert np.allclose(gm[r0:r1], mo, rtol=0, atol=2e-6)
        assert np.allclose(gr[r0:r1], ro, rtol=2e-6)


def _forward_stats(X, x_scale, gamma, gam_s, beta):
    """mean and 1/sigma from the library's own forward call (the backward's inputs)."""
    R, d = X.data.shape
    Y = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(X, gamma, beta, Y, eps=EPS, mean=mean, rinv=rinv)
    return mean, rinv


def _column_sums_check(c, R, d, dg, db, g_s):
    """dgamma / dbeta against fp64 column sums taken chunk by chunk (error relative to the summed magnitudes)."""
    f = orc.kf(R)
    sg, sb, mg, mb = (np.zeros(d) for _ in range(4))
    for r0, r1 in chunks(R):
        n32, _, _, _ = orc.layernorm_fwd(c["X"][r0:r1], BF, None, 0, 1.0, None, 0, 1.0, EPS, False, orc.F32)
        nv = orc.decode(n32, orc.F32)
        Gd = orc.decode(c["G"][r0:r1], BF)
        p = Gd * nv
        sg += p.sum(axis=0)
        sb += Gd.sum(axis=0)
        mg += np.abs(p).sum(axis=0)
        mb += np.abs(Gd).sum(axis=0)
    got_dg = orc.decode(to_bits(dg.data, orc.F32), orc.F32)
    got_db = orc.decode(to_bits(db.data, orc.F32), orc.F32)
    assert dg.scale_value() == g_s * f and db.scale_value() == g_s * f
    assert np.all(np.abs(got_dg - sg / f) <= 2e-5 * mg / f + 1e-30)
    assert np.all(np.abs(got_db - sb / f) <= 2e-5 * mb / f + 1e-30)


# (R, d, least number of rows per team)
BWD_CASES = [
    (131072, 1024, 100),     # the benchmark's shape: every team of the 296 blocks walks 111 rows
    (8192, 768, 7),          # configs 3 and 5
    (65536, 768, 50),
    (4096, 4096, 10),        # long rows, one team per block
    (3001, 4096, 10),        # ... with a ragged last stride
    (9000, 2048, 7),         # four warps per row, two teams per block
]


@pytest.mark.parametrize("R,d,min_rows", BWD_CASES)
@pytest.mark.parametrize("stat", [sc.STAT_L2, sc.STAT_AMAX])
def test_layernorm_backward_with_gradient_rescale_on_benchmarked_launch_shapes(R, d, min_rows, stat):
    plan = sc.scalify_debug_layernorm_plan(R, d, BF, True)
    assert plan["rows_per_team"] >= min_rows, plan
    assert plan["rows_per_team"] > 2 * plan["stages"] > 0, plan      # every slot of the row ring is reused
    c = si.layernorm_case(R, d, seed=53)
    x_s, g_s, gam_s = 2.0 ** 2, 2.0 ** -10, 2.0 ** -1
    X, G, gamma = st(c["X"], BF, x_s), st(c["G"], BF, g_s), st(c["gamma"], BF, gam_s)
    mean, rinv = _forward_stats(X, x_s, gamma, gam_s, st(c["beta"], BF, 1.0))
    dX = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    dXq = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
    dg, db = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws, eps=EPS, stat_dx=stat, dXq=dXq, dgamma=dg,
                                    dbeta=db)
    assert ws.check_status() == 0
    got = to_bits(dX.data, BF)
    gamv = orc.decode(c["gamma"], BF)
    dx_scale = None
    for r0, r1 in chunks(R):
        o = orc.layernorm_bwd(c["G"][r0:r1], BF, g_s, c["X"][r0:r1], BF, x_s, c["gamma"], BF, gam_s, EPS, False, BF,
                              orc.F32, want_f64=True)
        dx_scale = o["dX_scale"]
        _, _, _, ro = orc.layernorm_fwd(c["X"][r0:r1], BF, None, 0, 1.0, None, 0, 1.0, EPS, False, BF)
        row_mag = np.abs(orc.decode(c["G"][r0:r1], BF) * gamv[None, :]).max(axis=1) * ro
        ok = within(got[r0:r1], o["dX"], BF, o["dx_f64"], row_mag[:, None], 2.0 ** -18)
        assert ok.all(), (r0, int((~ok).sum()))
    assert dX.scale_value() == dx_scale == g_s * gam_s / x_s
    _column_sums_check(c, R, d, dg, db, g_s)
    # statistic and rescaled gradient, stage-isolated on the library's own dX, in full
    so = orc.statistic(got, BF, stat)
    gstat = float(ws.statistic().item())
    if stat == sc.STAT_AMAX:
        assert gstat == so
    else:
        assert abs(gstat - so) <= 2e-6 * so
        assert abs(math.log2(so) - round(math.log2(so))) > 1e-5, "seed lands on a binade edge: pick another"
    qo, qs, _ = orc.rescale(got, BF, dx_scale, stat, orc.E5M2)
    assert dXq.scale_value() == qs
    assert np.array_equal(to_bits(dXq.data, orc.E5M2), qo)
    # the one-pass form (dX = None) on the same launch shape: first with nothing to predict from (its second
    # launch writes the gradient again), then with the right prediction; the same bits as above both times
    ws1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    for _ in range(2):
        q1 = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
        dg1, db1 = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
        sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, None, ws1, eps=EPS, stat_dx=stat, dXq=q1, dgamma=dg1,
                                        dbeta=db1)
        assert ws1.check_status() == 0
        assert torch.equal(ws1.statistic().view(torch.int32), ws.statistic().view(torch.int32))
        assert q1.scale_value() == qs
        assert torch.equal(q1.data.view(torch.uint8), dXq.data.view(torch.uint8))
        assert torch.equal(dg1.data.view(torch.int32), dg.data.view(torch.int32))
        assert torch.equal(db1.data.view(torch.int32), db.data.view(torch.int32))


DELAYED_CASES = [
    (131072, 1024, orc.E5M2, sc.STAT_L2, 2.0 ** -7 * 1.3),
    (131072, 1024, BF, sc.STAT_AMAX, 0.011),
    (8192, 768, orc.E5M2, sc.STAT_L2, 2.0 ** -7 * 1.3),
    (4096, 4096, orc.E5M2, sc.STAT_AMAX, 0.011),
    (4096, 4096, orc.E4M3, sc.STAT_L2, 0.0),
    (9000, 2048, orc.E5M2, sc.STAT_L2, 0.37),
]


@pytest.mark.parametrize("R,d,dx_dt,stat,stat_in", DELAYED_CASES)
def test_layernorm_backward_with_delayed_rescale_on_benchmarked_launch_shapes(R, d, dx_dt, stat, stat_in):
    """The one-pass form: the gradient leaves already divided by the power of two of an earlier statistic,
    rounded once; this step's statistic is that of the un-rebalanced, unrounded derivative (fp64 here)."""
    plan = sc.scalify_debug_layernorm_plan(R, d, BF, True)
    assert plan["rows_per_team"] >= 3, plan
    c = si.layernorm_case(R, d, seed=57)
    x_s, g_s, gam_s = 2.0 ** 2, 2.0 ** -10, 2.0 ** -1
    X, G, gamma = st(c["X"], BF, x_s), st(c["G"], BF, g_s), st(c["gamma"], BF, gam_s)
    mean, rinv = _forward_stats(X, x_s, gamma, gam_s, st(c["beta"], BF, 1.0))
    dX = sc.ScaledTensor.empty((R, d), sc.TORCH_DTYPE[dx_dt])
    dg, db = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    ws.statistic().fill_(stat_in)
    sc.scalify_scaled_layernorm_bwd_delayed(G, X, gamma, mean, rinv, ws.statistic(), dX, ws, eps=EPS, stat_dx=stat,
                                            dgamma=dg, dbeta=db)
    assert ws.check_status() == 0
    usable = np.isfinite(stat_in) and stat_in >= 2.0 ** -126
    r = orc.p2f(float(np.float32(stat_in))) if usable else 1.0
    got = to_bits(dX.data, dx_dt)
    gamv = orc.decode(c["gamma"], BF)
    amax, ssq, mag_max = 0.0, 0.0, 0.0
    for r0, r1 in chunks(R):
        o = orc.layernorm_bwd(c["G"][r0:r1], BF, g_s, c["X"][r0:r1], BF, x_s, c["gamma"], BF, gam_s, EPS, False,
                              orc.F32, orc.F32, want_f64=True)
        dx = o["dx_f64"]
        _, _, _, ro = orc.layernorm_fwd(c["X"][r0:r1], BF, None, 0, 1.0, None, 0, 1.0, EPS, False, BF)
        row_mag = np.abs(orc.decode(c["G"][r0:r1], BF) * gamv[None, :]).max(axis=1) * ro
        exact = dx / r
        ok = within(got[r0:r1], orc.encode(exact, dx_dt), dx_dt, exact, row_mag[:, None] / r, 2.0 ** -18)
        assert ok.all(), (r0, int((~ok).sum()))
        amax = max(amax, float(np.abs(dx).max()))
        ssq += float((dx * dx).sum())
        mag_max = max(mag_max, float(row_mag.max()))
        assert dX.scale_value() == o["dX_scale"] * r
    gstat = float(ws.statistic().item())
    if stat == sc.STAT_AMAX:
        assert abs(gstat - amax) <= 2.0 ** -18 * mag_max
    else:
        want = math.sqrt(ssq / (R * d))
        assert abs(gstat - want) <= 2e-6 * want
    _column_sums_check(c, R, d, dg, db, g_s)
