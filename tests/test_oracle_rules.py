"""Pins of the oracle's scaled operations against what the paper and the
mathematics fix: exact rational brute force, library routines (numpy matmul,
torch LayerNorm / GELU / Adam and autograd), closed forms, and the invariants
of scale propagation (value = data * scale; model invariance; power-of-two
scales rounded down)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle as orc
import scalify_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ULP_HALF = {orc.BF16: 2.0 ** -9, orc.F16: 2.0 ** -12, orc.E4M3: 2.0 ** -5, orc.E5M2: 2.0 ** -4}


def is_pow2(x):
    m, _ = math.frexp(x)
    return m == 0.5


def vals(bits, dtype):
    """Independent (library) decode."""
    return si.from_bits(bits, dtype)


# ---------------------------------------------------------------- matmul

@pytest.mark.parametrize("a_dtype,b_dtype", [(orc.E4M3, orc.E4M3), (orc.E5M2, orc.E4M3)])
def test_matmul_tiny_exact_rational(a_dtype, b_dtype):
    M, N, K = 5, 7, 6
    A = si.scaled_normal(1, 1, (M, K), a_dtype, 4.0)
    B = si.scaled_normal(1, 2, (K, N), b_dtype, 0.3)
    Y, ys, acc, sab = orc.scaled_matmul(A, a_dtype, 0.5, B, b_dtype, 4.0, orc.F32, want_acc=True)
    Av, Bv = vals(A, a_dtype), vals(B, b_dtype)
    assert orc.kf(K) == 2.0
    assert ys == 0.5 * 4.0 * 2.0
    for i in range(M):
        for j in range(N):
            s = sum(Fraction(float(Av[i, k])) * Fraction(float(Bv[k, j])) for k in range(K))
            sa = sum(abs(Fraction(float(Av[i, k])) * Fraction(float(Bv[k, j]))) for k in range(K))
            assert Fraction(float(acc[i, j])) == s / 2  # fp64 accumulation of FP8 products is exact here
            assert Fraction(float(sab[i, j])) == sa / 2
    assert np.array_equal(Y.view(np.float32).astype(np.float64), acc.astype(np.float32).astype(np.float64))


def test_matmul_identity_and_one_hot_copy_rows():
    K = 16  # kf = 4
    A = si.scaled_normal(2, 1, (8, K), orc.E4M3)
    eye = si.to_bits(np.eye(K, dtype=np.float32) * 4.0, orc.E4M3)
    Y, ys, _, _ = orc.scaled_matmul(A, orc.E4M3, 1.0, eye, orc.E4M3, 1.0, orc.BF16)
    assert ys == 4.0
    # (A . 4I)/kf(16) = A exactly, and every E4M3 value is a BF16 value
    assert np.array_equal(vals(Y, orc.BF16), vals(A, orc.E4M3))
    perm = np.random.default_rng(0).permutation(K)
    P = np.zeros((K, K), dtype=np.float32)
    P[perm, np.arange(K)] = 4.0
    Y, _, _, _ = orc.scaled_matmul(A, orc.E4M3, 1.0, si.to_bits(P, orc.E4M3), orc.E4M3, 1.0, orc.BF16)
    assert np.array_equal(vals(Y, orc.BF16), vals(A, orc.E4M3)[:, perm])


def test_matmul_matches_numpy_and_transpose_flags():
    M, N, K = 33, 20, 48
    A = si.scaled_normal(3, 1, (M, K), orc.E5M2)
    B = si.scaled_normal(3, 2, (K, N), orc.E4M3)
    Y, ys, acc, sab = orc.scaled_matmul(A, orc.E5M2, 2.0 ** -10, B, orc.E4M3, 2.0 ** -6, orc.BF16, want_acc=True)
    ref = vals(A, orc.E5M2) @ vals(B, orc.E4M3) / orc.kf(K)
    assert np.allclose(acc, ref, rtol=0, atol=1e-12 * np.abs(ref).max())
    assert np.array_equal(sab, np.abs(vals(A, orc.E5M2)) @ np.abs(vals(B, orc.E4M3)) / orc.kf(K))
    assert ys == 2.0 ** -10 * 2.0 ** -6 * 4.0
    At = np.ascontiguousarray(A.T)
    Bt = np.ascontiguousarray(B.T)
    for ta, tb, a, b in [(True, False, At, B), (False, True, A, Bt), (True, True, At, Bt)]:
        Y2, ys2, acc2, _ = orc.scaled_matmul(a, orc.E5M2, 2.0 ** -10, b, orc.E4M3, 2.0 ** -6, orc.BF16,
                                             transA=ta, transB=tb, want_acc=True)
        assert np.array_equal(Y2, Y) and ys2 == ys and np.array_equal(acc2, acc)
    rows = np.array([0, 5, 32, 17])
    cols = np.array([19, 0, 7, 7])
    s_acc, s_sab = orc.scaled_matmul_samples(A, orc.E5M2, Bt, orc.E4M3, rows, cols, transB=True)
    assert np.array_equal(s_acc, acc[rows, cols]) and np.array_equal(s_sab, sab[rows, cols])


def test_matmul_scale_is_static_and_data_is_scale_invariant():
    c = si.config1()
    Y, ys, _, _ = orc.scaled_matmul(c["A"], c["a_dtype"], c["a_scale"], c["B"], c["b_dtype"], c["b_scale"], orc.BF16)
    assert ys == 8.0  # 2^-3 * 2^2 * kf(256)=16
    Y2, ys2, _, _ = orc.scaled_matmul(c["A"], c["a_dtype"], c["a_scale"] * 32, c["B"], c["b_dtype"], c["b_scale"] / 4,
                                      orc.BF16)
    assert np.array_equal(Y, Y2) and ys2 == ys * 8
    # the rule does not look at the data: zeros give the same scale
    Z = np.zeros_like(c["A"])
    _, ys3, _, _ = orc.scaled_matmul(Z, c["a_dtype"], c["a_scale"], c["B"], c["b_dtype"], c["b_scale"], orc.BF16)
    assert ys3 == ys


@pytest.mark.parametrize("K,lo,hi", [(256, 0.93, 1.07), (512, 1.32, 1.50), (1024, 0.93, 1.07)])
def test_matmul_rule_keeps_unit_scale_for_unit_gaussian_operands(K, lo, hi):
    A = si.scaled_normal(5, 1, (96, K), orc.E4M3)
    B = si.scaled_normal(5, 2, (K, 96), orc.E4M3)
    _, _, acc, _ = orc.scaled_matmul(A, orc.E4M3, 1.0, B, orc.E4M3, 1.0, orc.BF16, want_acc=True)
    rms = math.sqrt(np.mean(acc ** 2))
    assert lo < rms < hi, rms  # sqrt(K)/kf(K) is 1 for even powers of two, sqrt(2) for odd ones


# ---------------------------------------------------------------- rescale / set_scaling

def test_rescale_worked_example_golden():
    g = {}
    for line in open(os.path.join(GOLDEN, "rescale_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        g[k] = [float(t) for t in v]
    x = si.to_bits(np.array(g["in"], dtype=np.float32), orc.BF16)
    y, ys, s = orc.rescale(x, orc.BF16, g["in_scale"][0], orc.STAT_AMAX, orc.BF16)
    assert s == 3.0 and ys == g["amax_scale"][0]
    assert np.array_equal(vals(y, orc.BF16), np.array(g["amax_out"]))
    y, ys, s = orc.rescale(x, orc.BF16, g["in_scale"][0], orc.STAT_L2, orc.BF16)
    assert abs(s - math.sqrt((9 + 0.25 + 0.5625) / 3)) < 1e-15 and ys == g["l2_scale"][0]
    assert np.array_equal(vals(y, orc.BF16), np.array(g["l2_out"]))


@pytest.mark.parametrize("stat", [orc.STAT_AMAX, orc.STAT_L2])
@pytest.mark.parametrize("mag", [2.0 ** -9, 1.0, 300.0])
def test_rescale_postconditions_value_invariance_idempotence(stat, mag):
    x = si.to_bits(si.normal(6, 1, (4096,), mag), orc.BF16)
    xs = 2.0 ** -5
    y, ys, s = orc.rescale(x, orc.BF16, xs, stat, orc.BF16)
    assert is_pow2(ys)
    # BF16 -> BF16 by a power of two is exact: value unchanged
    assert np.array_equal(vals(y, orc.BF16) * ys, vals(x, orc.BF16) * xs)
    new_stat = orc.statistic(y, orc.BF16, stat)
    assert 1.0 <= new_stat < 2.0
    assert s == orc.statistic(x, orc.BF16, stat)
    y2, ys2, _ = orc.rescale(y, orc.BF16, ys, stat, orc.BF16)
    assert np.array_equal(y2, y) and ys2 == ys


def test_statistic_definitions_against_numpy():
    x = si.scaled_normal(7, 1, (1000,), orc.F16, 3.0)
    v = vals(x, orc.F16)
    assert orc.statistic(x, orc.F16, orc.STAT_AMAX) == np.abs(v).max()
    assert abs(orc.statistic(x, orc.F16, orc.STAT_L2) - np.sqrt(np.mean(v * v))) < 1e-12


def test_rescale_to_fp8_rounds_once_from_the_exact_quotient():
    x = si.to_bits(si.normal(8, 1, (2048,), 37.0), orc.BF16)
    y, ys, s = orc.rescale(x, orc.BF16, 1.0, orc.STAT_AMAX, orc.E4M3)
    r = ys
    q = vals(x, orc.BF16) / r
    assert np.array_equal(y, si.to_bits(q, orc.E4M3))  # q is exact in fp32, library cast rounds once
    assert 1.0 <= np.abs(vals(y, orc.E4M3)).max() <= 2.0  # [1,2) before rounding; rounding may reach 2


def test_rescale_degenerate_statistics_leave_array_unchanged():
    z = np.zeros(16, dtype=np.uint16)
    y, ys, s = orc.rescale(z, orc.BF16, 0.25, orc.STAT_AMAX, orc.BF16)
    assert s == 0.0 and ys == 0.25 and np.array_equal(y, z)
    x = si.to_bits(np.array([1.0, float("inf"), -2.0], dtype=np.float32), orc.BF16)
    y, ys, s = orc.rescale(x, orc.BF16, 0.25, orc.STAT_AMAX, orc.BF16)
    assert math.isinf(s) and ys == 0.25 and np.array_equal(y, x)
    x = si.to_bits(np.array([1.0, float("nan"), -2.0], dtype=np.float32), orc.BF16)
    y, ys, s = orc.rescale(x, orc.BF16, 0.25, orc.STAT_L2, orc.BF16)
    assert math.isnan(s) and ys == 0.25


def test_delayed_rescale_uses_supplied_statistic():
    x = si.to_bits(np.array([3.0, -0.5], dtype=np.float32), orc.BF16)
    y, ys, s = orc.rescale(x, orc.BF16, 1.0, orc.STAT_AMAX, orc.BF16, stat_override=9.0)
    assert s == 9.0 and ys == 8.0
    assert np.array_equal(vals(y, orc.BF16), np.array([0.375, -0.0625]))


def test_set_scaling_rescales_by_ratio_and_floors_requested_scale():
    x = si.scaled_normal(9, 1, (512,), orc.BF16)
    y, ys = orc.set_scaling(x, orc.BF16, 2.0 ** -3, 2.0 ** 2, orc.BF16)
    assert ys == 4.0
    assert np.array_equal(vals(y, orc.BF16) * 4.0, vals(x, orc.BF16) * 2.0 ** -3)
    y2, ys2 = orc.set_scaling(x, orc.BF16, 2.0 ** -3, 0.02, orc.BF16)
    assert ys2 == 2.0 ** -6
    assert np.array_equal(vals(y2, orc.BF16) * ys2, vals(x, orc.BF16) * 2.0 ** -3)
    # as_scaled_array of an unscaled input: old scale 1
    y3, ys3 = orc.set_scaling(x, orc.BF16, 1.0, 0.5, orc.E4M3)
    assert np.array_equal(y3, si.to_bits(vals(x, orc.BF16) * 2.0, orc.E4M3))


# ---------------------------------------------------------------- add

@pytest.mark.parametrize("sa,sb", [(1.0, 1.0), (2.0 ** -6, 2.0 ** 3), (8.0, 2.0 ** -10)])
def test_add_rule_closed_form_commutes_and_is_correctly_rounded(sa, sb):
    A = si.scaled_normal(10, 1, (17, 40), orc.BF16)
    B = si.scaled_normal(10, 2, (17, 40), orc.BF16)
    Y, ys = orc.scaled_add(A, orc.BF16, sa, B, orc.BF16, sb, orc.BF16)
    assert ys == max(sa, sb)  # p2f(sqrt(a^2+b^2)) = max for power-of-two scales
    Y2, ys2 = orc.scaled_add(B, orc.BF16, sb, A, orc.BF16, sa, orc.BF16)
    assert np.array_equal(Y, Y2) and ys == ys2
    exact = (vals(A, orc.BF16) * sa + vals(B, orc.BF16) * sb) / ys  # exact in fp64 for these magnitudes
    got = vals(Y, orc.BF16)
    assert np.all(np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-300)
    assert np.array_equal(Y, orc.encode(exact, orc.BF16))
    D, ds = orc.scaled_add(A, orc.BF16, sa, B, orc.BF16, sb, orc.BF16, subtract=True)
    exact = (vals(A, orc.BF16) * sa - vals(B, orc.BF16) * sb) / ds
    assert np.array_equal(D, orc.encode(exact, orc.BF16))


def test_add_zero_returns_operand_at_larger_scale_and_bias_broadcasts():
    A = si.scaled_normal(11, 1, (8, 24), orc.BF16)
    Z = np.zeros_like(A)
    Y, ys = orc.scaled_add(A, orc.BF16, 0.5, Z, orc.BF16, 4.0, orc.BF16)
    assert ys == 4.0
    assert np.array_equal(vals(Y, orc.BF16) * 4.0, vals(A, orc.BF16) * 0.5)
    b = si.scaled_normal(11, 2, (24,), orc.BF16)
    Y, ys = orc.scaled_add(A, orc.BF16, 1.0, b, orc.BF16, 1.0, orc.F32)
    exact = vals(A, orc.BF16) + vals(b, orc.BF16)[None, :]
    assert np.array_equal(Y.view(np.float32).astype(np.float64), exact)


def test_add_rule_keeps_unit_scale_within_a_binade():
    A = si.scaled_normal(12, 1, (1 << 16,), orc.BF16).reshape(1, -1)
    B = si.scaled_normal(12, 2, (1 << 16,), orc.BF16).reshape(1, -1)
    Y, ys = orc.scaled_add(A, orc.BF16, 1.0, B, orc.BF16, 1.0, orc.BF16)
    rms = math.sqrt(np.mean(vals(Y, orc.BF16) ** 2))
    assert 1.0 <= rms < 2.0  # sqrt(2) expected


# ---------------------------------------------------------------- LayerNorm

def test_layernorm_fwd_reduces_to_textbook_when_eps_inside():
    c = si.layernorm_case(12, 96)
    Y, ys, mean, rinv = orc.layernorm_fwd(c["X"], c["x_dtype"], c["gamma"], orc.BF16, 1.0, c["beta"], orc.BF16, 1.0,
                                          1e-5, True, orc.F32)
    x = torch.from_numpy(vals(c["X"], orc.BF16))
    ref = torch.nn.functional.layer_norm(x, (96,), torch.from_numpy(vals(c["gamma"], orc.BF16)),
                                         torch.from_numpy(vals(c["beta"], orc.BF16)), 1e-5)
    assert ys == 1.0
    assert np.allclose(Y.view(np.float32), ref.numpy(), rtol=0, atol=2e-7 * 8)
    assert np.array_equal(Y, orc.encode(ref.numpy(), orc.F32)) or \
        np.max(np.abs(Y.view(np.float32).astype(np.float64) - ref.numpy())) < 1e-6
    assert np.allclose(mean, x.mean(1).numpy(), atol=1e-15)
    assert np.allclose(rinv, 1.0 / np.sqrt(x.var(1, unbiased=False).numpy() + 1e-5), rtol=1e-14)


def test_layernorm_fwd_eps_outside_closed_forms():
    X = si.scaled_normal(13, 1, (10, 64), orc.BF16, 3.0)
    eps = 0.25  # large, so that the placement of eps matters
    Y, ys, mean, rinv = orc.layernorm_fwd(X, orc.BF16, None, 0, 1.0, None, 0, 1.0, eps, False, orc.F32)
    n = Y.view(np.float32).astype(np.float64)
    sig = vals(X, orc.BF16).std(axis=1)  # biased
    assert ys == 1.0
    assert np.allclose(n.mean(axis=1), 0.0, atol=1e-7)
    assert np.allclose(np.sqrt((n ** 2).mean(axis=1)), sig / (sig + eps), rtol=1e-6)
    assert np.allclose(rinv, 1.0 / (sig + eps), rtol=1e-14)
    # differs from the textbook placement
    Y2, _, _, _ = orc.layernorm_fwd(X, orc.BF16, None, 0, 1.0, None, 0, 1.0, eps, True, orc.F32)
    n2 = Y2.view(np.float32).astype(np.float64)
    assert np.allclose(np.sqrt((n2 ** 2).mean(axis=1)), sig / np.sqrt(sig ** 2 + eps), rtol=1e-6)


def test_layernorm_constant_rows_and_affine_scale_rule():
    X = si.to_bits(np.full((3, 32), 5.0, dtype=np.float32), orc.BF16)
    g = si.to_bits(np.full(32, 1.5, dtype=np.float32), orc.BF16)
    b = si.to_bits(np.full(32, 0.75, dtype=np.float32), orc.BF16)
    Y, ys, _, rinv = orc.layernorm_fwd(X, orc.BF16, g, orc.BF16, 2.0 ** -2, b, orc.BF16, 2.0 ** 3, 1e-5, False, orc.BF16)
    assert ys == 8.0  # max(gamma_s, beta_s)
    assert np.array_equal(vals(Y, orc.BF16), np.full((3, 32), 0.75))  # n = 0/(0+eps) = 0 -> beta_d*(b_s/Y_s)
    assert np.allclose(rinv, 1e5)
    # value-space check of the affine part: Y_d*Y_s = n*gamma + beta
    c = si.layernorm_case(6, 48)
    Y, ys, _, _ = orc.layernorm_fwd(c["X"], orc.BF16, c["gamma"], orc.BF16, 2.0 ** -2, c["beta"], orc.BF16, 2.0, 1e-5,
                                    False, orc.F32)
    N, _, _, _ = orc.layernorm_fwd(c["X"], orc.BF16, None, 0, 1.0, None, 0, 1.0, 1e-5, False, orc.F32)
    n = N.view(np.float32).astype(np.float64)
    want = n * vals(c["gamma"], orc.BF16) * 0.25 + vals(c["beta"], orc.BF16) * 2.0
    assert ys == 2.0
    assert np.allclose(Y.view(np.float32).astype(np.float64) * ys, want, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("eps_inside", [False, True])
def test_layernorm_bwd_matches_autograd_of_the_printed_forward(eps_inside):
    R, d, eps = 16, 40, 0.05
    c = si.layernorm_case(R, d, seed=14)
    gs, xs, gam_s = 2.0 ** -10, 2.0 ** 2, 2.0 ** -1
    out = orc.layernorm_bwd(c["G"], orc.BF16, gs, c["X"], orc.BF16, xs, c["gamma"], orc.BF16, gam_s, eps, eps_inside,
                            orc.F32, orc.F32, want_f64=True)
    x = torch.from_numpy(vals(c["X"], orc.BF16)).requires_grad_(True)
    gamma = torch.from_numpy(vals(c["gamma"], orc.BF16)).requires_grad_(True)
    beta = torch.zeros(d, dtype=torch.float64, requires_grad=True)
    mu = x.mean(1, keepdim=True)
    var = ((x - mu) ** 2).mean(1, keepdim=True)
    n = (x - mu) / (torch.sqrt(var + eps) if eps_inside else torch.sqrt(var) + eps)
    y = n * gamma + beta
    G = torch.from_numpy(vals(c["G"], orc.BF16))
    y.backward(G)
    assert np.allclose(out["dx_f64"], x.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(out["dx_f64"].sum(axis=1), 0.0, atol=1e-12)
    f = orc.kf(R)
    assert f == 4.0
    assert np.allclose(out["dgamma"].view(np.float32) * f, gamma.grad.numpy(), rtol=1e-6, atol=1e-6)
    assert np.allclose(out["dbeta"].view(np.float32) * f, beta.grad.numpy(), rtol=1e-6, atol=1e-6)
    assert out["dX_scale"] == gs * gam_s / xs
    assert out["dgamma_scale"] == gs * f and out["dbeta_scale"] == gs * f


def test_layernorm_bwd_zero_variance_row_has_no_second_term():
    X = si.to_bits(np.full((1, 16), 2.0, dtype=np.float32), orc.BF16)
    G = si.scaled_normal(15, 1, (1, 16), orc.BF16)
    out = orc.layernorm_bwd(G, orc.BF16, 1.0, X, orc.BF16, 1.0, None, 0, 1.0, 1e-3, False, orc.F32, orc.F32,
                            want_f64=True)
    g = vals(G, orc.BF16)
    assert np.allclose(out["dx_f64"], (g - g.mean()) / 1e-3, rtol=1e-12)


# ---------------------------------------------------------------- GELU

@pytest.mark.parametrize("exact", [False, True])
def test_gelu_scaled_form_matches_library_and_autograd(exact):
    X = si.scaled_normal(16, 1, (4000,), orc.BF16)
    xs = 2.0 ** 1
    Y, ys = orc.gelu_fwd(X, orc.BF16, xs, orc.F32, exact_erf=exact)
    xv = torch.from_numpy(vals(X, orc.BF16) * xs).requires_grad_(True)
    ref = torch.nn.functional.gelu(xv, approximate="none" if exact else "tanh")
    # value = Y_d * Y_s = x_d * g(x) * x_s = gelu(x)
    assert ys == xs
    assert np.allclose(Y.view(np.float32).astype(np.float64) * ys, ref.detach().numpy(), rtol=1e-6, atol=1e-7)
    G = si.scaled_normal(16, 2, (4000,), orc.BF16)
    ref.backward(torch.from_numpy(vals(G, orc.BF16)))
    dX, dxs = orc.gelu_bwd(G, orc.BF16, 2.0 ** -10, X, orc.BF16, xs, orc.F32, exact_erf=exact)
    assert dxs == 2.0 ** -10  # the gradient scale passes through unchanged
    assert np.allclose(dX.view(np.float32), xv.grad.numpy(), rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------- Adam

def test_adam_value_space_equals_library_adam_over_several_steps():
    n = 257
    w0 = si.normal(17, 1, (n,), 0.02)
    p = torch.nn.Parameter(torch.from_numpy(w0.astype(np.float64)))
    f32 = lambda c: float(np.float32(c))  # the C interface carries fp32 hyper-parameters
    opt = torch.optim.Adam([p], lr=f32(3e-4), betas=(f32(0.9), f32(0.999)), eps=f32(1e-8))
    # fp32 everything with arbitrary power-of-two scales: model invariance says values follow textbook Adam
    ws, ms, vs, gs = 2.0 ** -6, 2.0 ** -3, 2.0 ** -20, 2.0 ** -12
    w = orc.encode(w0 / ws, orc.F32)
    m = np.zeros(n, dtype=np.uint32)
    v = np.zeros(n, dtype=np.uint32)
    for t in range(1, 6):
        gv = si.normal(17, 10 + t, (n,))
        g = si.to_bits(gv, orc.E5M2)
        p.grad = torch.from_numpy(vals(g, orc.E5M2) * gs)
        opt.step()
        m, v, w, ms, vs, ws = orc.adam_step(g, orc.E5M2, gs, m, v, orc.F32, ms, vs, w, orc.F32, ws,
                                            3e-4, 0.9, 0.999, 1e-8, t)
        for s in (ms, vs, ws):
            assert is_pow2(s)
        st = opt.state[p]
        b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))  # the oracle sees fp32 hyper-parameters
        assert np.allclose(w.view(np.float32) * ws, p.detach().numpy(), rtol=2e-6, atol=1e-9)
        assert np.allclose(m.view(np.float32) * ms, st["exp_avg"].numpy(), rtol=2e-6, atol=1e-12)
        assert np.allclose(v.view(np.float32) * vs, st["exp_avg_sq"].numpy(), rtol=2e-6, atol=1e-15)


def test_adam_first_step_is_sign_update():
    n = 64
    g = si.scaled_normal(18, 1, (n,), orc.E5M2)
    w = np.zeros(n, dtype=np.uint32)
    z = np.zeros(n, dtype=np.uint32)
    m, v, w2, ms, vs, ws = orc.adam_step(g, orc.E5M2, 1.0, z, z, orc.F32, 1.0, 1.0, w, orc.F32, 1.0,
                                         1e-3, 0.9, 0.999, 1e-8, 1)
    gv = vals(g, orc.E5M2)
    want = -1e-3 * gv / (np.abs(gv) + 1e-8)
    assert np.allclose(w2.view(np.float32) * ws, want, rtol=1e-5, atol=1e-12)


def test_adam_scale_words_golden_cfg4():
    want = {}
    for line in open(os.path.join(GOLDEN, "adam_scales_cfg4.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        want[k] = int(v)
    c = si.adam_case(1024)
    m, v, w, ms, vs, ws = orc.adam_step(c["g"], c["g_dtype"], c["g_scale"], c["m"], c["v"], c["mv_dtype"],
                                        c["m_scale"], c["v_scale"], c["w"], c["w_dtype"], c["w_scale"],
                                        c["lr"], c["beta1"], c["beta2"], c["eps"], c["step"])
    assert ms == 2.0 ** want["m_scale_log2"]
    assert vs == 2.0 ** want["v_scale_log2"]
    assert ws == 2.0 ** want["w_scale_log2"]
    # FP16 outputs are the correctly rounded value/scale: compare with an independent fp64 evaluation
    gv = vals(c["g"], orc.E5M2) * c["g_scale"]
    mv = vals(c["m"], orc.F16) * c["m_scale"]
    vv = vals(c["v"], orc.F16) * c["v_scale"]
    wv = vals(c["w"], orc.F16) * c["w_scale"]
    b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))
    lr, eps = float(np.float32(3e-4)), float(np.float32(1e-8))
    m2 = b1 * mv + (1 - b1) * gv
    v2 = b2 * vv + (1 - b2) * gv * gv
    w2 = wv - lr * (m2 / (1 - b1 ** 1000)) / (np.sqrt(v2 / (1 - b2 ** 1000)) + eps)
    for got, exact, s in [(m, m2, ms), (v, v2, vs), (w, w2, ws)]:
        d = vals(got, orc.F16)
        q = exact / s
        assert np.all(np.abs(d - q) <= np.maximum(np.abs(q) * 2.0 ** -11, 2.0 ** -25) * 1.0000001)


# ---------------------------------------------------------------- delayed rescaling (Section 3.3)

def test_delayed_matmul_equals_matmul_followed_by_rescale_with_the_old_statistic():
    M, N, K = 24, 40, 64
    A = si.scaled_normal(19, 1, (M, K), orc.E4M3)
    B = si.scaled_normal(19, 2, (K, N), orc.E4M3)
    # E4M3 products summed over K=64 are exact in fp32, so the fp32 intermediate loses nothing
    Y32, ys, acc, _ = orc.scaled_matmul(A, orc.E4M3, 0.5, B, orc.E4M3, 2.0, orc.F32, want_acc=True)
    assert np.array_equal(orc.decode(Y32, orc.F32), acc)
    for stat_in in (9.0, 0.3, 0.0, float("inf")):
        Yd, yds, s_now = orc.scaled_matmul_delayed(A, orc.E4M3, 0.5, B, orc.E4M3, 2.0, stat_in, orc.STAT_AMAX, orc.E4M3)
        want, ws, _ = orc.rescale(Y32, orc.F32, ys, orc.STAT_AMAX, orc.E4M3,
                                  stat_override=stat_in if np.isfinite(stat_in) and stat_in > 0 else 1.0)
        assert np.array_equal(Yd, want) and yds == ws
        assert s_now == np.abs(acc).max()
    _, _, s_l2 = orc.scaled_matmul_delayed(A, orc.E4M3, 0.5, B, orc.E4M3, 2.0, 1.0, orc.STAT_L2, orc.BF16)
    assert abs(s_l2 - np.sqrt(np.mean(acc ** 2))) < 1e-12


def test_delayed_layernorm_bwd_composition_reduces_to_the_plain_call_and_keeps_values():
    """The composition the GPU tests use for the delayed LayerNorm gradient (tests/helpers.py): with a
    statistic that cannot define a scale it IS the plain oracle call; with any other the represented
    values are unchanged up to one rounding of the output format, the scale moves by exactly p2f(stat_in),
    and the statistic handed on is that of the un-rebalanced derivative."""
    from helpers import layernorm_bwd_delayed, ulp_of
    R, d = 12, 48
    G = si.scaled_normal(33, 1, (R, d), orc.BF16)
    X = si.scaled_normal(33, 2, (R, d), orc.BF16)
    gam = si.to_bits(1.0 + 0.1 * si.normal(33, 3, (d,), 1.0), orc.BF16)
    args = (G, orc.BF16, 2.0 ** -10, X, orc.BF16, 0.5, gam, orc.BF16, 1.0, 1e-5, False)
    plain = orc.layernorm_bwd(*args, orc.E5M2, orc.F32, want_f64=True)
    for bad in (0.0, float("inf"), float("nan"), 2.0 ** -130):
        o = layernorm_bwd_delayed(*args, bad, orc.STAT_AMAX, orc.E5M2, orc.F32)
        assert o["r"] == 1.0 and o["dX_scale"] == plain["dX_scale"] and np.array_equal(o["dX"], plain["dX"])
    dx = plain["dx_f64"]
    for stat_in in (9.0, 0.3, 2.0 ** -7, 1.0):
        o = layernorm_bwd_delayed(*args, stat_in, orc.STAT_L2, orc.E5M2, orc.F32)
        m, e = math.frexp(o["r"])
        assert m == 0.5 and o["r"] <= stat_in < 2 * o["r"]                 # the power of two below the statistic
        assert o["dX_scale"] == plain["dX_scale"] * o["r"]
        vals_q = orc.decode(o["dX"], orc.E5M2) * o["r"]                        # back at the static scale
        assert np.all(np.abs(vals_q - dx) <= 0.5 * ulp_of(dx / o["r"], orc.E5M2) * o["r"])
        assert abs(o["stat"] - np.sqrt(np.mean(dx * dx))) < 1e-15
        assert np.array_equal(o["dgamma"], plain["dgamma"]) and o["dgamma_scale"] == plain["dgamma_scale"]
    o = layernorm_bwd_delayed(*args, 1.0, orc.STAT_AMAX, orc.E5M2, orc.F32)
    assert o["stat"] == np.abs(dx).max()
