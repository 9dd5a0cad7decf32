"""Config 3: a GPT-style MLP block, forward and backward, composed from the C-ABI calls.

    fwd:  h0 = LN(x) -> E4M3 -> a1 = h0 W1 (+ b1) -> h1 = GELU(a1) -> E4M3 -> a2 = h1 W2 (+ b2) -> out = x + a2
    bwd:  dOut -> E5M2 -> dH1 = dY W2^T, dW2 = h1^T dY, db2 = 1^T dY -> GELU' -> E5M2
          -> dH0 = dA1 W1^T, dW1 = h0^T dA1, db1 = 1^T dA1 -> LN backward with L2 rescale -> dx = dOut + dLN

Shapes d = 768, ffn = 3072, GELU tanh, LayerNorm in BF16, matmuls FP8 (E4M3 forward operands, E5M2
gradients), weights N(0, 0.02) as E4M3 data at scale 2^-6, upstream gradient N(0,1)*2^-10.  Rows
R = 8192 (batch 8 x seq 1024), the stated size: the oracle's six matmuls are 1.2e11 multiply-adds,
some tens of seconds on the host cores.

Parity is stage-isolated: every library call is compared with the oracle applied to the SAME
inputs (the library's own previous outputs), so each stage is held to its own tolerance and no
binade-edge decision propagates.  At the end the value of the block output and of dx is compared
with an unscaled fp64 evaluation of the same network (model invariance, Section 1): they agree
to FP8 quantisation noise.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu

R, D, F = 8192, 768, 3072
BF, E4, E5 = orc.BF16, orc.E4M3, orc.E5M2


def ST(bits, dt, scale):
    return sc.ScaledTensor.make(to_dev(bits, dt), scale)


def bits(t, dt):
    return to_bits(t.data, dt)


class Lib:
    """Thin helpers around the binding that return (bits, scale) and check the status word."""

    def __init__(self):
        self.ws = sc.Workspace(max(sc.scalify_workspace_bytes(sc.OP_MATMUL, F, F),
                                   sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, D)))

    def cast(self, X, dt):
        Y = sc.ScaledTensor.empty(tuple(X.data.shape), sc.TORCH_DTYPE[dt])
        sc.scalify_rescale(X, Y)
        return Y

    def matmul(self, A, B, shape, transA=False, transB=False):
        Y = sc.ScaledTensor.empty(shape, torch.bfloat16)
        sc.scalify_scaled_matmul(A, B, Y, self.ws, transA=transA, transB=transB)
        assert self.ws.check_status() == 0
        return Y

    def add(self, A, B, subtract=False):
        Y = sc.ScaledTensor.empty(tuple(A.data.shape), torch.bfloat16)
        sc.scalify_scaled_add(A, B, Y, subtract=subtract)
        return Y


def check_cast(X, Y, x_dt, y_dt):
    assert Y.scale_value() == X.scale_value()
    assert np.array_equal(bits(Y, y_dt), orc.encode(orc.decode(bits(X, x_dt), x_dt), y_dt))


def check_matmul(A, a_dt, B, b_dt, Y, transA=False, transB=False):
    Yo, ys, acc, sab = orc.scaled_matmul(bits(A, a_dt), a_dt, A.scale_value(), bits(B, b_dt), b_dt, B.scale_value(),
                                         BF, transA=transA, transB=transB, want_acc=True)
    assert Y.scale_value() == ys
    ok = within(bits(Y, BF), Yo, BF, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())


def check_add(A, B, Y, subtract=False):
    a, b = bits(A, BF), bits(B, BF)
    yo, ys = orc.scaled_add(a, BF, A.scale_value(), b, BF, B.scale_value(), BF, subtract=subtract)
    assert Y.scale_value() == ys
    fa, fb = A.scale_value() / ys, B.scale_value() / ys
    av, bv = orc.decode(a, BF) * fa, orc.decode(b, BF) * fb
    exact = av - bv if subtract else av + bv
    ok = within(bits(Y, BF), yo, BF, exact, np.abs(av) + np.abs(bv), 2.0 ** -23)
    assert ok.all(), int((~ok).sum())


def test_mlp_block_forward_and_backward():
    L = Lib()
    # ------------------------------------------------------------------ inputs
    x = ST(si.scaled_normal(3, 1, (R, D), BF), BF, 1.0)
    gamma = ST(si.to_bits(1.0 + 0.1 * si.normal(3, 2, (D,)), BF), BF, 1.0)
    beta = ST(si.to_bits(0.1 * si.normal(3, 3, (D,)), BF), BF, 1.0)
    W1 = ST(si.scaled_normal(3, 4, (D, F), E4, 0.02 * 64), E4, 2.0 ** -6)   # [K, N]
    W2 = ST(si.scaled_normal(3, 5, (F, D), E4, 0.02 * 64), E4, 2.0 ** -6)
    b1 = ST(si.to_bits(0.02 * 64 * si.normal(3, 6, (F,)), BF), BF, 2.0 ** -6)
    b2 = ST(si.to_bits(0.02 * 64 * si.normal(3, 7, (D,)), BF), BF, 2.0 ** -6)
    dOut = ST(si.scaled_normal(3, 8, (R, D), BF), BF, 2.0 ** -10)
    ones = ST(si.to_bits(np.ones((1, R), dtype=np.float32), E4), E4, 1.0)

    # ------------------------------------------------------------------ forward
    h0 = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    mean = torch.empty(R, dtype=torch.float32, device="cuda")
    rinv = torch.empty(R, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_layernorm(x, gamma, beta, h0, eps=1e-5, mean=mean, rinv=rinv)
    yo, ys, _, _ = orc.layernorm_fwd(bits(x, BF), BF, bits(gamma, BF), BF, 1.0, bits(beta, BF), BF, 1.0, 1e-5, False, BF)
    n32, _, _, _ = orc.layernorm_fwd(bits(x, BF), BF, None, 0, 1.0, None, 0, 1.0, 1e-5, False, orc.F32)
    nv = orc.decode(n32, orc.F32)
    gv, bv = orc.decode(bits(gamma, BF), BF), orc.decode(bits(beta, BF), BF)
    assert h0.scale_value() == ys == 1.0
    ok = within(bits(h0, BF), yo, BF, nv * gv + bv, np.abs(nv * gv) + np.abs(bv) + 1e-3, 2e-6)
    assert ok.all()

    h0q = L.cast(h0, E4)
    check_cast(h0, h0q, BF, E4)
    a1 = L.matmul(h0q, W1, (R, F))                                  # NN: B is [K, N]
    check_matmul(h0q, E4, W1, E4, a1)
    assert a1.scale_value() == 1.0 * 2.0 ** -6 * 16
    a1b = L.add(a1, b1)
    check_add(a1, sc.ScaledTensor(b1.data.expand(R, F).contiguous(), b1.scale), a1b)
    h1 = sc.ScaledTensor.empty((R, F), torch.bfloat16)
    sc.scalify_scaled_gelu(a1b, h1)
    go, gs = orc.gelu_fwd(bits(a1b, BF), BF, a1b.scale_value(), BF)
    assert h1.scale_value() == gs and ulp_diff(bits(h1, BF), go, BF).max() <= 1
    h1q = L.cast(h1, E4)
    check_cast(h1, h1q, BF, E4)
    a2 = L.matmul(h1q, W2, (R, D))
    check_matmul(h1q, E4, W2, E4, a2)
    a2b = L.add(a2, b2)
    out = L.add(x, a2b)
    check_add(x, a2b, out)

    # ------------------------------------------------------------------ backward
    dyq = L.cast(dOut, E5)
    check_cast(dOut, dyq, BF, E5)
    dH1 = L.matmul(dyq, W2, (R, F), transB=True)                    # dY W2^T: W2 stored [F, D] = [N, K]
    check_matmul(dyq, E5, W2, E4, dH1, transB=True)
    dW2 = L.matmul(h1q, dyq, (F, D), transA=True)                   # h1^T dY: h1q stored [R, F] = [K, M]
    check_matmul(h1q, E4, dyq, E5, dW2, transA=True)
    db2 = L.matmul(ones, dyq, (1, D))                               # column sum as a contraction over R
    check_matmul(ones, E4, dyq, E5, db2)
    assert db2.scale_value() == dOut.scale_value() * orc.kf(R)
    dA1 = sc.ScaledTensor.empty((R, F), torch.bfloat16)
    sc.scalify_scaled_gelu_bwd(dH1, a1b, dA1)
    do, ds = orc.gelu_bwd(bits(dH1, BF), BF, dH1.scale_value(), bits(a1b, BF), BF, a1b.scale_value(), BF)
    assert dA1.scale_value() == ds == dH1.scale_value()
    dd = ulp_diff(bits(dA1, BF), do, BF)
    bad = dd > 1  # f' crosses zero near x = -0.75: absolute bound there
    if bad.any():
        err = np.abs(orc.decode(bits(dA1, BF), BF) - orc.decode(do, BF))
        assert np.all(err[bad] <= 2.0 ** -9 * 2e-2 * np.abs(orc.decode(bits(dH1, BF), BF))[bad] + 2.0 ** -16)
    dA1q = L.cast(dA1, E5)
    check_cast(dA1, dA1q, BF, E5)
    dH0 = L.matmul(dA1q, W1, (R, D), transB=True)                   # dA1 W1^T: W1 stored [D, F] = [N, K]
    check_matmul(dA1q, E5, W1, E4, dH0, transB=True)
    dW1 = L.matmul(h0q, dA1q, (D, F), transA=True)
    check_matmul(h0q, E4, dA1q, E5, dW1, transA=True)
    db1 = L.matmul(ones, dA1q, (1, F))
    check_matmul(ones, E4, dA1q, E5, db1)

    dX = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    dXq = sc.ScaledTensor.empty((R, D), torch.bfloat16)
    dg = sc.ScaledTensor.empty((D,), torch.float32)
    db = sc.ScaledTensor.empty((D,), torch.float32)
    sc.scalify_scaled_layernorm_bwd(dH0, x, gamma, mean, rinv, dX, L.ws, eps=1e-5, stat_dx=sc.STAT_L2, dXq=dXq,
                                    dgamma=dg, dbeta=db)
    assert L.ws.check_status() == 0
    o = orc.layernorm_bwd(bits(dH0, BF), BF, dH0.scale_value(), bits(x, BF), BF, 1.0, bits(gamma, BF), BF, 1.0, 1e-5,
                          False, BF, orc.F32, want_f64=True)
    assert dX.scale_value() == o["dX_scale"]
    _, _, _, ro = orc.layernorm_fwd(bits(x, BF), BF, None, 0, 1.0, None, 0, 1.0, 1e-5, False, BF)
    ghat = orc.decode(bits(dH0, BF), BF) * gv[None, :]
    row_mag = np.abs(ghat).max(axis=1) * ro
    got = bits(dX, BF)
    ok = within(got, o["dX"], BF, o["dx_f64"], row_mag[:, None], 2.0 ** -18)
    assert ok.all(), int((~ok).sum())
    so = orc.statistic(got, BF, orc.STAT_L2)
    assert abs(float(L.ws.statistic().item()) - so) <= 2e-6 * so
    assert abs(so / orc.p2f(so) - 1.5) < 0.499
    qo, qs, _ = orc.rescale(got, BF, o["dX_scale"], orc.STAT_L2, BF)
    assert dXq.scale_value() == qs and np.array_equal(bits(dXq, BF), qo)
    dx = L.add(dOut, dXq)
    check_add(dOut, dXq, dx)

    # ------------------------------------------------------------------ model invariance (fp64, unscaled)
    def val(T, dt):
        return orc.decode(bits(T, dt), dt) * T.scale_value()
    xv, W1v, W2v = val(x, BF), val(W1, E4), val(W2, E4)
    b1v, b2v = val(b1, BF), val(b2, BF)
    xt = torch.from_numpy(xv).requires_grad_(True)
    mu = xt.mean(1, keepdim=True)
    sig = ((xt - mu) ** 2).mean(1, keepdim=True).sqrt()
    h0t = (xt - mu) / (sig + 1e-5) * torch.from_numpy(gv) + torch.from_numpy(bv)
    a1t = h0t @ torch.from_numpy(W1v) + torch.from_numpy(b1v)
    h1t = torch.nn.functional.gelu(a1t, approximate="tanh")
    outt = xt + h1t @ torch.from_numpy(W2v) + torch.from_numpy(b2v)
    outt.backward(torch.from_numpy(val(dOut, BF)))

    def rel_rms(a, b):
        return float(np.sqrt(np.mean((a - b) ** 2)) / np.sqrt(np.mean(b ** 2)))
    assert rel_rms(val(out, BF), outt.detach().numpy()) < 0.02
    assert rel_rms(val(dx, BF), xt.grad.numpy()) < 0.08
    # every propagated scale is a power of two and the data components stay near unit scale
    for T, dt in [(a1, BF), (h1, BF), (a2, BF), (out, BF), (dH1, BF), (dA1, BF), (dH0, BF), (dXq, BF), (dW1, BF),
                  (dW2, BF)]:
        s = T.scale_value()
        assert s > 0 and np.log2(s) == round(np.log2(s))
        rms = float(np.sqrt(np.mean(orc.decode(bits(T, dt), dt) ** 2)))
        assert 2.0 ** -6 < rms < 2.0 ** 4, (rms, s)
