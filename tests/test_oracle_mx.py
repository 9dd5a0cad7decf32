"""Pins of the oracle's block-scale functions (Section 2: block scales in E8M0, the OCP MX formats).

None of these re-types the oracle's formulas: they use the OCP definitions of E8M0 and MXFP8
(exponent-only byte with bias 127; shared exponent = floor(log2(amax)) - emax of the element format),
hand-computed bit patterns, an independent library decode (torch's float8 dtypes), brute force in
Python floats, and special cases that reduce to the per-tensor matmul pinned elsewhere."""
import math

import numpy as np
import pytest
import torch

import oracle as orc
import scalify_inputs as si


def torch_decode_fp8(bits: np.ndarray, dt: int) -> np.ndarray:
    tdt = torch.float8_e4m3fn if dt == orc.E4M3 else torch.float8_e5m2
    return torch.from_numpy(bits.copy()).view(tdt).to(torch.float64).numpy()


def torch_decode_e8m0(codes: np.ndarray) -> np.ndarray:
    return torch.from_numpy(codes.copy()).view(torch.float8_e8m0fnu).to(torch.float64).numpy()


def test_e8m0_is_an_exponent_only_byte_with_bias_127():
    # OCP MX: E8M0 value = 2^(code-127) for code 0..254, code 255 = NaN
    assert orc.e8m0_decode(127) == 1.0
    assert orc.e8m0_decode(0) == 2.0 ** -127
    assert orc.e8m0_decode(254) == 2.0 ** 127
    assert math.isnan(orc.e8m0_decode(255))
    codes = np.arange(255, dtype=np.uint8)
    mine = np.array([orc.e8m0_decode(int(c)) for c in codes])
    assert np.array_equal(mine, torch_decode_e8m0(codes))
    assert np.all(mine[1:] == 2.0 * mine[:-1])


def test_quantize_hand_computed_block():
    # block maximum 3.0: floor(log2 3) = 1, E4M3 emax = 8  =>  e = -7, code 120;
    # 3.0 * 2^7 = 384 = 1.5 * 2^8 -> sign 0, exponent field 8+7 = 15, mantissa .100 -> 0x7C
    # 1.0 * 2^7 = 128 = 1.0 * 2^7 -> exponent field 14, mantissa 0 -> 0x70
    # -0.75 * 2^7 = -96 = -1.5 * 2^6 -> 0x80 | (13 << 3) | 4 = 0xEC
    x = np.zeros((1, 32), dtype=np.float32)
    x[0, 0], x[0, 1], x[0, 2] = 3.0, 1.0, -0.75
    data, codes = orc.mx_quantize(x.view(np.uint32), orc.F32, orc.E4M3)
    assert codes[0, 0] == 120
    assert data[0, 0] == 0x7C and data[0, 1] == 0x70 and data[0, 2] == 0xEC
    assert np.all(data[0, 3:] == 0)
    # the same block with E5M2 elements: emax = 15  =>  e = 1 - 15 = -14, code 113;
    # 3.0 * 2^14 = 1.5 * 2^15 -> exponent field 15+15 = 30, mantissa .10 -> (30 << 2) | 2 = 0x7A
    data, codes = orc.mx_quantize(x.view(np.uint32), orc.F32, orc.E5M2)
    assert codes[0, 0] == 113 and data[0, 0] == 0x7A


def test_quantize_degenerate_and_saturating_blocks():
    x = np.zeros((1, 96), dtype=np.float32)
    x[0, 32] = np.inf          # a block that cannot define a scale: exponent 0, element saturates
    x[0, 64] = 500.0           # 500 = 1.95 * 2^8: e = 0, 500 > 448 saturates to the largest E4M3
    x[0, 65] = 1.0
    data, codes = orc.mx_quantize(x.view(np.uint32), orc.F32, orc.E4M3)
    assert list(codes[0]) == [127, 127, 127]
    assert np.all(data[0, :32] == 0)
    assert data[0, 32] == 0x7E
    assert data[0, 64] == 0x7E and data[0, 65] == 0x38  # 1.0 in E4M3: exponent field 7, mantissa 0


@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_quantize_properties_against_the_mx_definition(elem):
    R, K = 64, 256
    x = si.normal(7, 1, (R, K), 1.0).astype(np.float64)
    x *= np.exp2(np.random.default_rng(3).integers(-20, 20, size=(R, K // 32))).repeat(32, axis=1)  # wide range
    xb = si.to_bits(x.astype(np.float32), orc.BF16)
    xv = orc.decode(xb, orc.BF16).reshape(R, K)
    data, codes = orc.mx_quantize(xb, orc.BF16, elem)
    emax = 8 if elem == orc.E4M3 else 15
    amax = np.abs(xv).reshape(R, K // 32, 32).max(axis=2)
    # shared exponent per the OCP rule, computed here with numpy's exact frexp
    want = np.frexp(amax)[1] - 1 - emax + 127
    assert np.array_equal(codes.astype(np.int64), want)
    # element values through an independent decode; dequantised block maxima land in [2^emax, 2^(emax+1))
    dq = torch_decode_fp8(data, elem).reshape(R, K // 32, 32)
    top = np.abs(dq).max(axis=2)
    assert np.all(top >= 2.0 ** emax) and np.all(top <= (448.0 if elem == orc.E4M3 else 57344.0))
    # relative error of every element that is not tiny against its block maximum: half an ulp of the format
    mant = 3 if elem == orc.E4M3 else 2
    back = dq * torch_decode_e8m0(codes)[:, :, None]
    ref = xv.reshape(R, K // 32, 32)
    sat_limit = (448.0 if elem == orc.E4M3 else 57344.0) * torch_decode_e8m0(codes)[:, :, None]
    big = (np.abs(ref) >= amax[:, :, None] * 2.0 ** -6) & (np.abs(ref) <= sat_limit)
    rel = np.abs(back - ref)[big] / np.abs(ref)[big]
    assert rel.max() <= 2.0 ** -(mant + 1) * (1 + 1e-12)
    # shifting a block by a power of two moves its code and nothing else
    xs = xv.copy()
    xs[:, :32] *= 8.0
    d2, c2 = orc.mx_quantize(si.to_bits(xs.astype(np.float32), orc.BF16), orc.BF16, elem)
    assert np.array_equal(c2[:, 0], codes[:, 0] + 3) and np.array_equal(d2, data)


def test_mx_matmul_brute_force_tiny():
    M, N, K = 5, 4, 64
    a = si.to_bits(si.normal(11, 1, (M, K), 1.0), orc.E4M3)
    b = si.to_bits(si.normal(11, 2, (N, K), 1.0), orc.E5M2)
    rng = np.random.default_rng(5)
    ea = rng.integers(120, 135, size=(M, K // 32)).astype(np.uint8)
    eb = rng.integers(120, 135, size=(N, K // 32)).astype(np.uint8)
    Y, ys, acc, sab = orc.mx_matmul(a, orc.E4M3, ea, 0.5, b, orc.E5M2, eb, 4.0, orc.F32, want_acc=True)
    av, bv = torch_decode_fp8(a, orc.E4M3), torch_decode_fp8(b, orc.E5M2)
    sa, sb = torch_decode_e8m0(ea), torch_decode_e8m0(eb)
    kf = 8.0  # K = 64: floor(log2 64) = 6, half of it 3
    assert ys == 0.5 * 4.0 * kf
    for i in range(M):
        for j in range(N):
            tot = 0.0
            for k in range(K):
                tot += (av[i, k] * sa[i, k // 32]) * (bv[j, k] * sb[j, k // 32])
            assert abs(acc[i, j] - tot / kf) <= 1e-12 * sab[i, j]
            assert np.float32(acc[i, j]).view(np.uint32) == Y[i, j]  # the stored fp32 is the rounded fp64 result


def test_mx_matmul_reduces_to_the_per_tensor_matmul_when_block_exponents_are_uniform():
    M, N, K = 33, 17, 160
    a = si.to_bits(si.normal(12, 1, (M, K), 1.0), orc.E4M3)
    b = si.to_bits(si.normal(12, 2, (N, K), 1.0), orc.E4M3)
    ea = np.full((M, K // 32), 124, dtype=np.uint8)   # 2^-3
    eb = np.full((N, K // 32), 130, dtype=np.uint8)   # 2^+3
    Y, ys, acc, _ = orc.mx_matmul(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.BF16, want_acc=True)
    Y0, ys0, acc0, _ = orc.scaled_matmul(a, orc.E4M3, 1.0, b, orc.E4M3, 1.0, orc.BF16, transB=True, want_acc=True)
    assert ys == ys0 and np.array_equal(acc, acc0) and np.array_equal(Y, Y0)
    # and with 2^-3 * 2^+1 the data component is exactly a quarter of it
    eb[:] = 128
    _, _, acc2, _ = orc.mx_matmul(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.BF16, want_acc=True)
    assert np.array_equal(acc2, acc0 * 0.25)


def test_block_scales_keep_more_signal_than_one_tensor_scale_on_rows_of_mixed_magnitude():
    # the point of the finer scale (Section 2): quantisation noise stays relative to each block's own size,
    # while under one tensor-wide scale the small blocks fall below E4M3's 17 binades and are lost
    R, K = 128, 512
    x = si.normal(13, 1, (R, K), 1.0).astype(np.float64)
    x *= np.exp2(np.random.default_rng(9).integers(-24, 1, size=(R, K // 32))).repeat(32, axis=1)
    xb = si.to_bits(x.astype(np.float32), orc.BF16)
    xv = orc.decode(xb, orc.BF16).reshape(R, K)
    data, codes = orc.mx_quantize(xb, orc.BF16, orc.E4M3)
    back = torch_decode_fp8(data, orc.E4M3) * np.repeat(torch_decode_e8m0(codes), 32, axis=1)
    top = 2.0 ** math.floor(math.log2(np.abs(xv).max()))
    one_scale = torch_decode_fp8(orc.encode(xv.reshape(-1) / top * 256.0, orc.E4M3), orc.E4M3).reshape(R, K) \
        / 256.0 * top

    def block_error(q):
        err = np.sum(((q - xv) ** 2).reshape(R, K // 32, 32), axis=2)
        return err / np.sum((xv ** 2).reshape(R, K // 32, 32), axis=2)

    assert block_error(back).max() < 0.01
    assert np.percentile(block_error(one_scale), 75) > 0.5
