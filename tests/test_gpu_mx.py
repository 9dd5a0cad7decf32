"""GPU parity of the block-scaled path (E8M0 exponent per 32 elements of K) against the fp64 oracle.

Bars: quantised FP8 bytes, exponent bytes and scale words bit-exact; the matmul's fp32 output within
1e-5 * sum|a*b| per element; BF16 / F16 outputs within 1 ulp (or half an ulp plus the accumulation bar
where the dot product cancels); the fused AMAX equal to the maximum of the stored output."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, within

pytestmark = pytest.mark.gpu


def wide_range_input(seed, rows, K, dt, spread=20):
    x = si.normal(seed, 1, (rows, K), 1.0).astype(np.float64)
    x *= np.exp2(np.random.default_rng(seed).integers(-spread, spread, size=(rows, K // 32))).repeat(32, axis=1)
    return si.to_bits(x.astype(np.float32), dt)


@pytest.mark.parametrize("rows,K", [(1, 128), (300, 256), (513, 1024), (128, 4096)])
@pytest.mark.parametrize("x_dt", [orc.BF16, orc.F16, orc.F32])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_mx_quantize_bit_exact(rows, K, x_dt, elem):
    xb = wide_range_input(100 + rows, rows, K, x_dt, spread=6 if x_dt == orc.F16 else 20)
    X = sc.ScaledTensor.make(to_dev(xb, x_dt), 2.0 ** -4)
    Y = sc.MxTensor(rows, K, sc.TORCH_DTYPE[elem])
    Y.sf.fill_(0xFF)  # whatever was there, padding rows included, must be overwritten
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_mx_quantize(X, Y, status=status)
    assert int(status.item()) == 0
    data, codes = orc.mx_quantize(xb, x_dt, elem)
    assert np.array_equal(Y.exponents().cpu().numpy(), codes)
    assert np.array_equal(to_bits(Y.data, elem), data)
    assert Y.scale_value() == 2.0 ** -4
    # every exponent byte of the padding rows is the neutral code
    pr = (rows + 255) // 256 * 256
    full = Y.sf.view(pr // 128, K // 128, 32, 4, 4).permute(0, 3, 2, 1, 4).reshape(pr, K // 32)
    assert bool((full[rows:] == 127).all())


def test_mx_quantize_degenerate_blocks_and_strided_input():
    rows, K = 5, 256
    x = np.zeros((rows, K + 64), dtype=np.float32)
    x[:, :K] = si.normal(3, 1, (rows, K), 1.0)
    x[0, :32] = 0.0                      # all-zero block
    x[1, 40] = np.inf                    # a block that cannot define a scale
    x[2, 70] = np.nan
    x[3, 96:128] = 2.0 ** -140           # fp32 subnormals: exponent clamps at the bottom of E8M0
    x[4, 128] = 500.0                    # saturates E4M3 after scaling
    buf = torch.from_numpy(x).cuda()
    X = sc.ScaledTensor.make(buf[:, :K], 1.0)
    Y = sc.MxTensor(rows, K)
    sc.scalify_mx_quantize(X, Y)
    xb = np.ascontiguousarray(x[:, :K]).view(np.uint32)
    data, codes = orc.mx_quantize(xb, orc.F32, orc.E4M3)
    assert np.array_equal(Y.exponents().cpu().numpy(), codes)
    got = to_bits(Y.data, orc.E4M3)
    nan = (data & 0x7F) == 0x7F
    assert np.array_equal(got[~nan], data[~nan]) and np.all((got[nan] & 0x7F) == 0x7F)
    assert codes[0, 0] == 127 and codes[1, 1] == 127 and codes[2, 2] == 127 and codes[3, 3] == 0


@pytest.mark.parametrize("x_dt,lead,skip", [(orc.BF16, 16, 8), (orc.BF16, 8, 0), (orc.F32, 4, 4)])
def test_mx_quantize_rows_aligned_to_16_bytes_only(x_dt, lead, skip):
    # a window of a wider buffer whose first element, or whose row stride, is a multiple of 16 bytes
    # but not of 32: the kernel's 32-byte loads must fall back to 16-byte ones
    rows, K = 70, 256
    xb = np.ascontiguousarray(wide_range_input(9, rows, K + 32, x_dt, spread=10)[:, :K + lead])
    buf = to_dev(xb, x_dt)
    X = sc.ScaledTensor.make(buf[:, skip:skip + K], 1.0)
    Y = sc.MxTensor(rows, K)
    sc.scalify_mx_quantize(X, Y)
    data, codes = orc.mx_quantize(np.ascontiguousarray(xb[:, skip:skip + K]), x_dt, orc.E4M3)
    assert np.array_equal(Y.exponents().cpu().numpy(), codes)
    assert np.array_equal(to_bits(Y.data, orc.E4M3), data)


def run_mx_matmul(a, a_dt, ea, a_s, b, b_dt, eb, b_s, y_dt, stat=sc.STAT_NONE):
    M, K = a.shape
    N = b.shape[0]
    A = sc.MxTensor(M, K, sc.TORCH_DTYPE[a_dt])
    B = sc.MxTensor(N, K, sc.TORCH_DTYPE[b_dt])
    A.data.copy_(to_dev(a, a_dt)); B.data.copy_(to_dev(b, b_dt))
    A.set_exponents(torch.from_numpy(ea)); B.set_exponents(torch.from_numpy(eb))
    A.scale.fill_(a_s); B.scale.fill_(b_s)
    Y = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[y_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    sc.scalify_mx_matmul(A, B, Y, ws, stat=stat)
    assert ws.check_status() == 0
    return to_bits(Y.data, y_dt), Y.scale_value(), float(ws.statistic().item())


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (64, 40, 256), (200, 304, 384), (257, 520, 1024)])
@pytest.mark.parametrize("a_dt,b_dt", [(orc.E4M3, orc.E4M3), (orc.E5M2, orc.E4M3)])
def test_mx_matmul_against_oracle(M, N, K, a_dt, b_dt):
    a = si.to_bits(si.normal(21, M + K, (M, K), 1.0), a_dt)
    b = si.to_bits(si.normal(22, N + K, (N, K), 1.0), b_dt)
    rng = np.random.default_rng(M * 7 + N)
    ea = rng.integers(117, 138, size=(M, K // 32)).astype(np.uint8)   # a different exponent for every block
    eb = rng.integers(117, 138, size=(N, K // 32)).astype(np.uint8)
    Yo, ys, acc, sab = orc.mx_matmul(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.BF16, want_acc=True)
    g32, s32, _ = run_mx_matmul(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.F32)
    assert s32 == ys
    err = np.abs(orc.decode(g32, orc.F32).reshape(M, N) - acc)
    assert np.all(err <= 1e-5 * sab + 1e-30), float((err / (sab + 1e-30)).max())
    gb, sb, stat = run_mx_matmul(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.BF16, stat=sc.STAT_AMAX)
    assert sb == ys
    ok = within(gb, Yo, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    assert stat == float(np.abs(orc.decode(gb, orc.BF16)).max())


@pytest.mark.parametrize("M,N,K", [(2304, 2560, 640), (1280, 4864, 128)])
def test_mx_matmul_more_tiles_than_ctas(M, N, K):
    """90 and 95 output tiles of 256 x 256 on 74 CTA pairs: some pairs compute two tiles, so the ring of
    operand slots and exponent buffers runs on across a tile boundary at a K-block count (5, 1) that is neither
    a multiple of the ring depth nor of the exponent warps' load group.  Every element against the oracle."""
    a_dt = b_dt = orc.E4M3
    a = si.to_bits(si.normal(31, M + K, (M, K), 1.0), a_dt)
    b = si.to_bits(si.normal(32, N + K, (N, K), 1.0), b_dt)
    rng = np.random.default_rng(M + 3 * N + K)
    ea = rng.integers(117, 138, size=(M, K // 32)).astype(np.uint8)
    eb = rng.integers(117, 138, size=(N, K // 32)).astype(np.uint8)
    Yo, ys, acc, sab = orc.mx_matmul(a, a_dt, ea, 0.5, b, b_dt, eb, 2.0, orc.BF16, want_acc=True)
    gb, sb, stat = run_mx_matmul(a, a_dt, ea, 0.5, b, b_dt, eb, 2.0, orc.BF16, stat=sc.STAT_AMAX)
    assert sb == ys
    ok = within(gb, Yo, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    assert stat == float(np.abs(orc.decode(gb, orc.BF16)).max())


@pytest.mark.parametrize("M", [128, 256])
def test_mx_matmul_distinguishes_every_exponent_byte(M):
    """One block of A and one block of B get a large exponent each, at every position in turn: a kernel
    that picked the wrong exponent byte (wrong row group, wrong K block, wrong half of a 256-column tile,
    wrong CTA of a pair: M = 256 runs the two-CTA form) would miss the product."""
    N, K = 256, 256
    a = si.to_bits(np.ones((M, K), dtype=np.float32), orc.E4M3)
    b = si.to_bits(np.ones((N, K), dtype=np.float32), orc.E4M3)
    for (i, kb, j) in [(0, 0, 0), (31, 1, 33), (32, 2, 127), (64, 3, 128), (97, 4, 200), (127, 7, 255),
                       (M - 128, 5, 129), (M - 1, 6, 64), (M - 60, 0, 250)]:
        ea = np.full((M, K // 32), 127, dtype=np.uint8)
        eb = np.full((N, K // 32), 127, dtype=np.uint8)
        ea[i, kb] = 130
        eb[j, kb] = 125
        Yo, _, acc, _ = orc.mx_matmul(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.F32, want_acc=True)
        g, _, _ = run_mx_matmul(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.F32)
        assert np.array_equal(orc.decode(g, orc.F32).reshape(M, N), acc), (i, kb, j)


def test_mx_matmul_f16_output_and_l2_statistic():
    M, N, K = 320, 272, 256
    a = si.to_bits(si.normal(41, 1, (M, K), 1.0), orc.E5M2)
    b = si.to_bits(si.normal(41, 2, (N, K), 1.0), orc.E5M2)
    rng = np.random.default_rng(11)
    ea = rng.integers(122, 130, size=(M, K // 32)).astype(np.uint8)
    eb = rng.integers(122, 130, size=(N, K // 32)).astype(np.uint8)
    Yo, ys, acc, sab = orc.mx_matmul(a, orc.E5M2, ea, 1.0, b, orc.E5M2, eb, 2.0 ** -5, orc.F16, want_acc=True)
    g, s, stat = run_mx_matmul(a, orc.E5M2, ea, 1.0, b, orc.E5M2, eb, 2.0 ** -5, orc.F16, stat=sc.STAT_L2)
    assert s == ys
    ok = within(g, Yo, orc.F16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    want = float(np.sqrt(np.mean(orc.decode(g, orc.F16).astype(np.float64) ** 2)))
    assert abs(stat - want) <= 2e-6 * want


def test_quantize_then_matmul_matches_the_oracle_pipeline():
    M, N, K = 384, 512, 512
    xa = wide_range_input(31, M, K, orc.BF16, spread=8)
    xb = wide_range_input(32, N, K, orc.BF16, spread=8)
    A, B = sc.MxTensor(M, K), sc.MxTensor(N, K)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(xa, orc.BF16), 0.5), A)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(xb, orc.BF16), 2.0), B)
    Y = sc.ScaledTensor.empty((M, N), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    sc.scalify_mx_matmul(A, B, Y, ws)
    da, ea = orc.mx_quantize(xa, orc.BF16, orc.E4M3)
    db, eb = orc.mx_quantize(xb, orc.BF16, orc.E4M3)
    _, ys, acc, sab = orc.mx_matmul(da, orc.E4M3, ea, 0.5, db, orc.E4M3, eb, 2.0, orc.F32, want_acc=True)
    assert Y.scale_value() == ys
    err = np.abs(orc.decode(to_bits(Y.data, orc.F32), orc.F32).reshape(M, N) - acc)
    assert np.all(err <= 1e-5 * sab)
    # and the block-scaled product is close to the product of the un-quantised operands
    va, vb = orc.decode(xa, orc.BF16).reshape(M, K), orc.decode(xb, orc.BF16).reshape(N, K)
    exact = va @ vb.T / orc.kf(K)
    rel = np.linalg.norm(acc - exact) / np.linalg.norm(exact)
    assert rel < 0.05


def test_quantize_and_matmul_full_size_8192_sampled():
    """The benchmark's block-scaled row at its full size: sampled rows of both quantised operands are
    bit-exact, sampled outputs agree with the oracle, and the statistic word is the AMAX of what was stored."""
    n = 8192
    xa = wide_range_input(41, n, n, orc.BF16, spread=8)
    xb = wide_range_input(42, n, n, orc.BF16, spread=8)
    A, B = sc.MxTensor(n, n), sc.MxTensor(n, n)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(xa, orc.BF16), 0.5), A)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(xb, orc.BF16), 2.0), B)
    Y = sc.ScaledTensor.empty((n, n), torch.bfloat16)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n))
    sc.scalify_mx_matmul(A, B, Y, ws, stat=sc.STAT_AMAX)
    assert ws.check_status() == 0
    rng = np.random.default_rng(9)
    rows = np.unique(np.concatenate([rng.integers(0, n, 40), [0, 127, 128, 255, 256, n - 129, n - 1]]))
    cols = np.unique(np.concatenate([rng.integers(0, n, 40), [0, 255, 256, 511, 512, n - 257, n - 1]]))
    da, ea = orc.mx_quantize(xa[rows], orc.BF16, orc.E4M3)
    db, eb = orc.mx_quantize(xb[cols], orc.BF16, orc.E4M3)
    tr, tc = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    assert np.array_equal(to_bits(A.data[tr], orc.E4M3), da) and np.array_equal(to_bits(B.data[tc], orc.E4M3), db)
    assert np.array_equal(A.exponents()[tr].cpu().numpy(), ea) and np.array_equal(B.exponents()[tc].cpu().numpy(), eb)
    Yo, ys, acc, sab = orc.mx_matmul(da, orc.E4M3, ea, 0.5, db, orc.E4M3, eb, 2.0, orc.BF16, want_acc=True)
    assert Y.scale_value() == ys
    got = to_bits(Y.data[tr][:, tc], orc.BF16)
    ok = within(got, Yo, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    assert float(ws.statistic().item()) == float(Y.data.float().abs().max())


@pytest.mark.parametrize("rows,K", [(16, 128), (304, 256), (528, 1024), (128, 4096)])
@pytest.mark.parametrize("x_dt", [orc.BF16, orc.F16, orc.F32])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_mx_quantize_transposed_bit_exact(rows, K, x_dt, elem):
    """The transposed form reads X stored [K, rows] and writes the FP8 data in the same orientation; the
    blocks still run along K (down the columns), so codes and exponents equal those of the oracle applied
    to the operand written out [rows, K]."""
    xb = wide_range_input(200 + rows, rows, K, x_dt, spread=6 if x_dt == orc.F16 else 20)
    X = sc.ScaledTensor.make(to_dev(np.ascontiguousarray(xb.T), x_dt), 2.0 ** 3)
    Y = sc.MxTensor(rows, K, sc.TORCH_DTYPE[elem], transposed=True)
    Y.sf.fill_(0xFF)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_mx_quantize(X, Y, status=status)
    assert int(status.item()) == 0
    data, codes = orc.mx_quantize(xb, x_dt, elem)
    assert np.array_equal(Y.exponents().cpu().numpy(), codes)
    assert np.array_equal(to_bits(Y.data, elem), np.ascontiguousarray(data.T))
    assert Y.scale_value() == 2.0 ** 3
    pr = (rows + 255) // 256 * 256
    full = Y.sf.view(pr // 128, K // 128, 32, 4, 4).permute(0, 3, 2, 1, 4).reshape(pr, K // 32)
    assert bool((full[rows:] == 127).all())


def test_mx_quantize_transposed_degenerate_blocks_and_strided_input():
    rows, K = 48, 256
    x = np.zeros((rows, K), dtype=np.float32)
    x[:] = si.normal(5, 1, (rows, K), 1.0)
    x[0, :32] = 0.0
    x[1, 40] = np.inf
    x[2, 70] = np.nan
    x[3, 96:128] = 2.0 ** -140
    x[4, 128] = 500.0
    wide = np.zeros((K, rows + 16), dtype=np.float32)      # a window of a wider buffer: ldx != rows
    wide[:, 4:4 + rows] = x.T
    buf = torch.from_numpy(wide).cuda()
    X = sc.ScaledTensor.make(buf[:, 4:4 + rows], 1.0)
    Y = sc.MxTensor(rows, K, transposed=True)
    sc.scalify_mx_quantize(X, Y)
    data, codes = orc.mx_quantize(np.ascontiguousarray(x).view(np.uint32), orc.F32, orc.E4M3)
    assert np.array_equal(Y.exponents().cpu().numpy(), codes)
    got = to_bits(Y.data, orc.E4M3).T
    nan = (data & 0x7F) == 0x7F
    assert np.array_equal(got[~nan], data[~nan]) and np.all((got[nan] & 0x7F) == 0x7F)
    assert codes[0, 0] == 127 and codes[1, 1] == 127 and codes[2, 2] == 127 and codes[3, 3] == 0


def run_mx_matmul_t(a, a_dt, ea, a_s, b, b_dt, eb, b_s, y_dt, ta, tb, stat=sc.STAT_NONE):
    """As run_mx_matmul, with operand A and / or B handed over in the transposed ([K, rows]) storage."""
    M, K = a.shape
    N = b.shape[0]
    A = sc.MxTensor(M, K, sc.TORCH_DTYPE[a_dt], transposed=ta)
    B = sc.MxTensor(N, K, sc.TORCH_DTYPE[b_dt], transposed=tb)
    A.data.copy_(to_dev(np.ascontiguousarray(a.T) if ta else a, a_dt))
    B.data.copy_(to_dev(np.ascontiguousarray(b.T) if tb else b, b_dt))
    A.set_exponents(torch.from_numpy(ea)); B.set_exponents(torch.from_numpy(eb))
    A.scale.fill_(a_s); B.scale.fill_(b_s)
    Y = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[y_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    sc.scalify_mx_matmul(A, B, Y, ws, stat=stat)
    assert ws.check_status() == 0
    return to_bits(Y.data, y_dt), Y.scale_value(), float(ws.statistic().item())


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (64, 48, 256), (208, 304, 384), (272, 528, 1024)])
@pytest.mark.parametrize("ta,tb", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("a_dt,b_dt", [(orc.E4M3, orc.E4M3), (orc.E5M2, orc.E4M3)])
def test_mx_matmul_transposed_operands_against_oracle(M, N, K, ta, tb, a_dt, b_dt):
    """The gradient products hand an operand over with K as the slow axis; the product is the same."""
    a = si.to_bits(si.normal(23, M + K, (M, K), 1.0), a_dt)
    b = si.to_bits(si.normal(24, N + K, (N, K), 1.0), b_dt)
    rng = np.random.default_rng(M * 5 + N)
    ea = rng.integers(117, 138, size=(M, K // 32)).astype(np.uint8)
    eb = rng.integers(117, 138, size=(N, K // 32)).astype(np.uint8)
    Yo, ys, acc, sab = orc.mx_matmul(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.BF16, want_acc=True)
    g32, s32, _ = run_mx_matmul_t(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.F32, ta, tb)
    assert s32 == ys
    err = np.abs(orc.decode(g32, orc.F32).reshape(M, N) - acc)
    assert np.all(err <= 1e-5 * sab + 1e-30), float((err / (sab + 1e-30)).max())
    gb, sb, stat = run_mx_matmul_t(a, a_dt, ea, 0.25, b, b_dt, eb, 8.0, orc.BF16, ta, tb, stat=sc.STAT_AMAX)
    assert sb == ys
    ok = within(gb, Yo, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    assert stat == float(np.abs(orc.decode(gb, orc.BF16)).max())


@pytest.mark.parametrize("M", [128, 256])
@pytest.mark.parametrize("ta,tb", [(True, False), (False, True), (True, True)])
def test_mx_matmul_transposed_distinguishes_every_element_and_exponent(M, ta, tb):
    """A single non-zero element in each operand, at awkward positions in turn: the product has exactly one
    non-zero entry, at (i, j), only if the transposed tiles are read with rows and K the right way round."""
    N, K = 256, 256
    for (i, k, j) in [(0, 0, 0), (31, 33, 33), (32, 70, 127), (64, 101, 128), (97, 130, 200), (127, 255, 255),
                      (M - 128, 160, 129), (M - 1, 200, 64), (M - 60, 31, 250)]:
        av = np.zeros((M, K), dtype=np.float32); av[i, k] = 1.5
        bv = np.zeros((N, K), dtype=np.float32); bv[j, k] = -2.0
        a, b = si.to_bits(av, orc.E4M3), si.to_bits(bv, orc.E4M3)
        ea = np.full((M, K // 32), 127, dtype=np.uint8); ea[i, k // 32] = 131
        eb = np.full((N, K // 32), 127, dtype=np.uint8); eb[j, k // 32] = 124
        _, _, acc, _ = orc.mx_matmul(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.F32, want_acc=True)
        g, _, _ = run_mx_matmul_t(a, orc.E4M3, ea, 1.0, b, orc.E4M3, eb, 1.0, orc.F32, ta, tb)
        got = orc.decode(g, orc.F32).reshape(M, N)
        assert np.array_equal(got, acc), (i, k, j)
        assert np.count_nonzero(got) == 1 and got[i, j] != 0


def test_quantize_transposed_then_matmul_is_the_weight_gradient_product():
    """dW[out, in] = sum over tokens of dY[token, out] * X[token, in]: both operands are stored with the
    contraction axis (tokens) slow, which is what the transposed quantiser and operand form are for."""
    T, O, I = 512, 384, 272
    dy = wide_range_input(51, O, T, orc.BF16, spread=8)      # operand view [O, T]; stored [T, O]
    xx = wide_range_input(52, I, T, orc.BF16, spread=8)      # operand view [I, T]; stored [T, I]
    A, B = sc.MxTensor(O, T, transposed=True), sc.MxTensor(I, T, transposed=True)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(np.ascontiguousarray(dy.T), orc.BF16), 0.5), A)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(np.ascontiguousarray(xx.T), orc.BF16), 2.0), B)
    Y = sc.ScaledTensor.empty((O, I), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, O, I))
    sc.scalify_mx_matmul(A, B, Y, ws)
    assert ws.check_status() == 0
    da, ea = orc.mx_quantize(dy, orc.BF16, orc.E4M3)
    db, eb = orc.mx_quantize(xx, orc.BF16, orc.E4M3)
    _, ys, acc, sab = orc.mx_matmul(da, orc.E4M3, ea, 0.5, db, orc.E4M3, eb, 2.0, orc.F32, want_acc=True)
    assert Y.scale_value() == ys
    err = np.abs(orc.decode(to_bits(Y.data, orc.F32), orc.F32).reshape(O, I) - acc)
    assert np.all(err <= 1e-5 * sab)


def test_quantize_and_matmul_transposed_full_size_8192_sampled():
    """The benchmark's transposed block-scaled rows at their full size (two-CTA tiles, every operand MN-major)."""
    n = 8192
    xa = wide_range_input(43, n, n, orc.BF16, spread=8)      # operand views [rows, K]
    xb = wide_range_input(44, n, n, orc.BF16, spread=8)
    A, B = sc.MxTensor(n, n, transposed=True), sc.MxTensor(n, n, transposed=True)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(np.ascontiguousarray(xa.T), orc.BF16), 0.5), A)
    sc.scalify_mx_quantize(sc.ScaledTensor.make(to_dev(np.ascontiguousarray(xb.T), orc.BF16), 2.0), B)
    Y = sc.ScaledTensor.empty((n, n), torch.bfloat16)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n))
    sc.scalify_mx_matmul(A, B, Y, ws, stat=sc.STAT_AMAX)
    assert ws.check_status() == 0
    rng = np.random.default_rng(10)
    rows = np.unique(np.concatenate([rng.integers(0, n, 40), [0, 127, 128, 255, 256, n - 129, n - 1]]))
    cols = np.unique(np.concatenate([rng.integers(0, n, 40), [0, 255, 256, 511, 512, n - 257, n - 1]]))
    da, ea = orc.mx_quantize(xa[rows], orc.BF16, orc.E4M3)
    db, eb = orc.mx_quantize(xb[cols], orc.BF16, orc.E4M3)
    tr, tc = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    assert np.array_equal(to_bits(A.data[:, tr].t().contiguous(), orc.E4M3), da)
    assert np.array_equal(to_bits(B.data[:, tc].t().contiguous(), orc.E4M3), db)
    assert np.array_equal(A.exponents()[tr].cpu().numpy(), ea) and np.array_equal(B.exponents()[tc].cpu().numpy(), eb)
    Yo, ys, acc, sab = orc.mx_matmul(da, orc.E4M3, ea, 0.5, db, orc.E4M3, eb, 2.0, orc.BF16, want_acc=True)
    assert Y.scale_value() == ys
    got = to_bits(Y.data[tr][:, tc], orc.BF16)
    ok = within(got, Yo, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    assert float(ws.statistic().item()) == float(Y.data.float().abs().max())


def test_mx_argument_checks():
    A = sc.MxTensor(64, 128)
    B = sc.MxTensor(32, 256)
    Y = sc.ScaledTensor.empty((64, 32), torch.bfloat16)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, 64, 32))
    with pytest.raises(sc.ScalifyError):
        sc.scalify_mx_matmul(A, B, Y, ws)      # K differs
    assert sc.scalify_mx_sf_bytes(64, 100) == 0  # K must be a multiple of 128
    X = sc.ScaledTensor.make(torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda"), 1.0)
    with pytest.raises(sc.ScalifyError):
        sc.scalify_mx_quantize(X, A)           # shape differs
    At = sc.MxTensor(64, 128, transposed=True)
    with pytest.raises(sc.ScalifyError):
        sc.scalify_mx_quantize(sc.ScaledTensor.make(torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda"), 1.0), At)  # X must be [K, rows]
    At._d.rows = 72                            # a transposed operand needs rows % 16 == 0
    with pytest.raises(sc.ScalifyError):
        sc.scalify_mx_matmul(At, sc.MxTensor(32, 128), Y, ws)
    At._d.rows, At._d.transposed = 64, 2       # the flag is 0 or 1
    with pytest.raises(sc.ScalifyError):
        sc.scalify_mx_matmul(At, sc.MxTensor(32, 128), Y, ws)
