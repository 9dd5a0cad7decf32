"""Arrays beyond 2^31 elements or bytes: the kernels index with 64-bit offsets.  The oracle checks
windows of the result (the start, the region around the 2^31 boundary, the ragged end) element by
element, and the statistic must see an extreme value placed in the last few elements."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_bits, within

pytestmark = pytest.mark.gpu


def windows(n, width=4096):
    edge = 1 << 31
    w = [(0, width), (n - width - 3, n)]
    if n > edge + width:
        w.append((edge - width // 2, edge + width // 2))
    return w


def fill_bytes(t: torch.Tensor, hi: int, seed: int):
    g = torch.Generator(device=t.device).manual_seed(seed)
    step = 1 << 28
    for s in range(0, t.numel(), step):
        e = min(t.numel(), s + step)
        t[s:e] = torch.randint(0, hi, (e - s,), dtype=torch.uint8, device=t.device, generator=g)


def test_dynamic_rescale_of_more_than_2_31_elements():
    n = (1 << 31) + 4099
    raw = torch.empty(n, dtype=torch.uint8, device="cuda")
    fill_bytes(raw, 0x60, 1)            # E4M3 codes below 0x60: |x| <= 30
    raw[n - 3] = 0x7E                   # 448, the largest E4M3, three elements before the end
    X = sc.ScaledTensor.make(raw.view(torch.float8_e4m3fn), 2.0 ** -2)
    Y = sc.ScaledTensor.empty((n,), torch.float8_e5m2)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, n))
    sc.scalify_rescale(X, Y, stat=sc.STAT_AMAX, ws=ws)
    assert ws.check_status() == 0
    assert float(ws.statistic().item()) == 448.0
    assert Y.scale_value() == 2.0 ** -2 * 256.0
    for a, b in windows(n):
        xin = raw[a:b].cpu().numpy()
        want, ys, _ = orc.rescale(xin, orc.E4M3, 2.0 ** -2, orc.STAT_AMAX, orc.E5M2, stat_override=448.0)
        assert np.array_equal(to_bits(Y.data[a:b], orc.E5M2), want), (a, b)
    # the statistic-only entry point over the same array
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    sc.scalify_statistic(X, sc.STAT_AMAX, ws, out=out)
    assert float(out.item()) == 448.0


def test_scaled_add_of_more_than_2_31_bytes():
    n = (1 << 30) + 520                 # BF16: 2 GiB + 1040 bytes per operand
    a = torch.empty(n, dtype=torch.int16, device="cuda")
    b = torch.empty(n, dtype=torch.int16, device="cuda")
    # bit patterns of moderate BF16 values: exponent field 120..130, any mantissa, either sign
    g = torch.Generator(device="cuda").manual_seed(2)
    step = 1 << 27
    for t in (a, b):
        for s in range(0, n, step):
            e = min(n, s + step)
            expo = torch.randint(120, 131, (e - s,), device="cuda", generator=g, dtype=torch.int32)
            mant = torch.randint(0, 128, (e - s,), device="cuda", generator=g, dtype=torch.int32)
            sign = torch.randint(0, 2, (e - s,), device="cuda", generator=g, dtype=torch.int32)
            v = (sign << 15) | (expo << 7) | mant
            t[s:e] = torch.where(v >= 32768, v - 65536, v).to(torch.int16)
    A = sc.ScaledTensor.make(a.view(torch.bfloat16), 2.0 ** -3)
    B = sc.ScaledTensor.make(b.view(torch.bfloat16), 2.0 ** 1)
    Y = sc.ScaledTensor.empty((n,), torch.bfloat16)
    sc.scalify_scaled_add(A, B, Y)
    assert Y.scale_value() == 2.0
    for lo, hi in windows(n, 2048) + [((1 << 30) - 1024, (1 << 30) + 520)]:
        ab = to_bits(A.data[lo:hi], orc.BF16)
        bb = to_bits(B.data[lo:hi], orc.BF16)
        want, ys = orc.scaled_add(ab, orc.BF16, 2.0 ** -3, bb, orc.BF16, 2.0, orc.BF16)
        got = to_bits(Y.data[lo:hi], orc.BF16)
        assert np.array_equal(got, want), (lo, hi)


def test_matmul_output_of_more_than_2_31_elements():
    M, N, K = 49152, 45056, 128         # 2.2e9 outputs, 4.4 GB of BF16
    a = si.to_bits(si.normal(71, 1, (M, K), 1.0), orc.E4M3)
    b = si.to_bits(si.normal(71, 2, (N, K), 1.0), orc.E4M3)
    a[M - 1, :] = 0x70                  # 128.0 in every element of the last row of A ...
    b[N - 2, :] = 0x70                  # ... and of the last-but-one row of B: the largest output by far
    from helpers import to_dev
    A = sc.ScaledTensor.make(to_dev(a, orc.E4M3), 1.0)
    B = sc.ScaledTensor.make(to_dev(b, orc.E4M3), 1.0)
    Y = sc.ScaledTensor.empty((M, N), torch.bfloat16)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    sc.scalify_scaled_matmul(A, B, Y, ws, transB=True, stat=sc.STAT_AMAX)
    assert ws.check_status() == 0
    rng = np.random.default_rng(3)
    rows = np.concatenate([rng.integers(0, M, 4000), np.full(64, M - 1), rng.integers(M - 300, M, 500),
                           np.array([0, M - 1, 47662])])
    cols = np.concatenate([rng.integers(0, N, 4000), rng.integers(N - 64, N, 64), rng.integers(0, N, 500),
                           np.array([0, N - 2, 45055])])
    acc, sab = orc.scaled_matmul_samples(a, orc.E4M3, b, orc.E4M3, rows, cols, transB=True)
    got = Y.data[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()]
    gb = to_bits(got, orc.BF16)
    want = orc.encode(acc, orc.BF16)
    ok = within(gb, want, orc.BF16, acc, sab, 1e-5)
    assert ok.all(), int((~ok).sum())
    # the largest element: 128 * 128 * 128 / kf(128) = 2^21 / 8
    assert float(ws.statistic().item()) == 2.0 ** 18
    assert float(Y.data[M - 1, N - 2].float().item()) == 2.0 ** 18
