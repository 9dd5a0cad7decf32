"""GPU parity of the scaled FP8 matmul (tcgen05 kernel) against the fp64 oracle.

Bars (stated by the benchmark contract): the propagated scale and every FP8 /
scale word bit-exact; the fp32 pre-cast values within 1e-5 * sum|a*b| per
element; BF16/F16 outputs within 1 ulp; the fused statistic equal to the
statistic of the stored output; the rescaled output bit-exact against the
oracle's rescale of the library's own intermediate (stage-isolated), because a
power-of-two rescale of identical BF16 input has exactly one correct answer.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu


def run_matmul(A, a_dt, a_s, B, b_dt, b_s, y_dt, transA=False, transB=False, stat=sc.STAT_NONE, q_dt=None,
               lda_pad=0, ldb_pad=0, splitk=False):
    """A, B: numpy bit arrays as stored (2-D or 3-D). Returns dict of numpy results."""
    def dev(x, dt, pad):
        if pad == 0:
            return to_dev(x, dt)
        shp = list(x.shape)
        shp[-1] += pad
        buf = torch.zeros(shp, dtype=torch.uint8, device="cuda").view(sc.TORCH_DTYPE[dt])
        view = buf[..., : x.shape[-1]]
        view.copy_(to_dev(x, dt))
        return view
    Ad, Bd = dev(A, a_dt, lda_pad), dev(B, b_dt, ldb_pad)
    M = A.shape[-1] if transA else A.shape[-2]
    N = B.shape[-2] if transB else B.shape[-1]
    shape = (M, N) if A.ndim == 2 else (A.shape[0], M, N)
    Y = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[y_dt])
    Yq = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[q_dt]) if q_dt is not None else None
    rows = M * (A.shape[0] if A.ndim == 3 else 1)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL_SPLITK if splitk else sc.OP_MATMUL, rows, N))
    sc.scalify_scaled_matmul(sc.ScaledTensor.make(Ad, a_s), sc.ScaledTensor.make(Bd, b_s), Y, ws, transA=transA,
                             transB=transB, stat=stat, Yq=Yq)
    status = ws.check_status()
    out = dict(Y=to_bits(Y.data, y_dt), y_scale=Y.scale_value(), status=status,
               stat=float(ws.statistic().item()))
    if Yq is not None:
        out["Yq"] = to_bits(Yq.data, q_dt)
        out["yq_scale"] = Yq.scale_value()
    return out


def check_against_oracle(A, a_dt, a_s, B, b_dt, b_s, transA, transB, **kw):
    # fp32 dump: accumulator error bar
    g32 = run_matmul(A, a_dt, a_s, B, b_dt, b_s, orc.F32, transA, transB, **kw)
    assert g32["status"] == 0
    gb = run_matmul(A, a_dt, a_s, B, b_dt, b_s, orc.BF16, transA, transB, **kw)
    assert gb["status"] == 0
    if A.ndim == 2:
        A3, B3 = A[None], B[None]
    else:
        A3, B3 = A, (B if B.ndim == 3 else np.broadcast_to(B, (A.shape[0],) + B.shape))
    for b in range(A3.shape[0]):
        Yo, ys, acc, sab = orc.scaled_matmul(A3[b], a_dt, a_s, B3[b], b_dt, b_s, orc.BF16, transA=transA,
                                             transB=transB, want_acc=True)
        g = g32["Y"].reshape((-1,) + Yo.shape)[b].view(np.float32).astype(np.float64)
        assert g32["y_scale"] == ys and gb["y_scale"] == ys
        err = np.abs(g - acc)
        bound = 1e-5 * sab + 1e-30
        assert np.all(err <= bound), (float((err / bound).max()), np.unravel_index(np.argmax(err / bound), err.shape))
        # BF16: one rounding of an fp32 value that is within 1e-5*sum|a*b| of the exact one
        ok = within(gb["Y"].reshape((-1,) + Yo.shape)[b], Yo, orc.BF16, acc, sab, 1e-5)
        assert ok.all(), int((~ok).sum())
        # bit-exact whenever the pre-cast fp32 value is identical: encode the library's own fp32 dump
        assert np.array_equal(gb["Y"].reshape((-1,) + Yo.shape)[b], orc.encode(g, orc.BF16))


def test_config1_256_cubed_with_dynamic_rescale():
    c = si.config1()
    Bt = np.ascontiguousarray(c["B"].T)
    for transB, Bmat in [(True, Bt), (False, c["B"])]:
        check_against_oracle(c["A"], orc.E4M3, c["a_scale"], Bmat, orc.E4M3, c["b_scale"], False, transB)
        g = run_matmul(c["A"], orc.E4M3, c["a_scale"], Bmat, orc.E4M3, c["b_scale"], orc.BF16, False, transB,
                       stat=sc.STAT_AMAX, q_dt=orc.BF16)
        assert g["status"] == 0 and g["y_scale"] == 8.0
        # the fused statistic is the AMAX of the stored intermediate
        assert g["stat"] == orc.statistic(g["Y"], orc.BF16, orc.STAT_AMAX)
        yq, yqs, _ = orc.rescale(g["Y"], orc.BF16, g["y_scale"], orc.STAT_AMAX, orc.BF16)
        assert np.array_equal(g["Yq"], yq) and g["yq_scale"] == yqs
        # end to end against the oracle chain
        Yo, ys, _, _ = orc.scaled_matmul(c["A"], orc.E4M3, c["a_scale"], c["B"], orc.E4M3, c["b_scale"], orc.BF16)
        yo, yos, so = orc.rescale(Yo, orc.BF16, ys, orc.STAT_AMAX, orc.BF16)
        assert abs(so / orc.p2f(so) - 1.5) < 0.49  # this seed is not a binade-edge case
        assert g["yq_scale"] == yos
        assert ulp_diff(g["Yq"], yo, orc.BF16).max() <= 1


@pytest.mark.parametrize("transA,transB", [(False, True), (False, False), (True, True), (True, False)])
@pytest.mark.parametrize("a_dt,b_dt", [(orc.E4M3, orc.E4M3), (orc.E5M2, orc.E4M3), (orc.E4M3, orc.E5M2)])
def test_ragged_shapes_all_layouts_and_formats(transA, transB, a_dt, b_dt):
    M, N, K = 208, 304, 176  # ragged in every tile dimension; strides stay multiples of 16 bytes
    A = si.scaled_normal(21, 1, (K, M) if transA else (M, K), a_dt)
    B = si.scaled_normal(21, 2, (N, K) if transB else (K, N), b_dt)
    check_against_oracle(A, a_dt, 2.0 ** -10, B, b_dt, 2.0 ** -6, transA, transB)


def test_several_tiles_long_k_and_padded_leading_dimensions():
    M, N, K = 384, 528, 1040
    A = si.scaled_normal(22, 1, (M, K), orc.E5M2)
    Bt = si.scaled_normal(22, 2, (N, K), orc.E4M3)
    check_against_oracle(A, orc.E5M2, 1.0, Bt, orc.E4M3, 2.0 ** -6, False, True, lda_pad=48, ldb_pad=16)
    B = np.ascontiguousarray(Bt.T)
    check_against_oracle(A, orc.E5M2, 1.0, B, orc.E4M3, 2.0 ** -6, False, False, lda_pad=16, ldb_pad=32)


def test_tiny_and_degenerate_shapes():
    for (M, N, K) in [(1, 16, 16), (16, 16, 16), (129, 264, 144), (128, 256, 128)]:
        A = si.scaled_normal(23, M, (M, K), orc.E4M3)
        Bt = si.scaled_normal(23, 1000 + N, (N, K), orc.E4M3)
        check_against_oracle(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, False, True)
    # identity operand: exact copy of A (power-of-two rescale only)
    K = 256
    A = si.scaled_normal(23, 7, (128, K), orc.E4M3)
    eye = si.to_bits(np.eye(K, dtype=np.float32) * 16.0, orc.E4M3)
    g = run_matmul(A, orc.E4M3, 1.0, eye, orc.E4M3, 1.0, orc.BF16, False, False)
    assert np.array_equal(orc.decode(g["Y"], orc.BF16), orc.decode(A, orc.E4M3))
    assert g["y_scale"] == 16.0


def test_batched_attention_like_shapes():
    # QK^T-like: [b, T, 64] x [b, T, 64]^T ; PV-like: [b, T, T] x [b, T, 64]
    b, T, hd = 3, 160, 64
    Q = si.scaled_normal(24, 1, (b, T, hd), orc.E4M3)
    Kt = si.scaled_normal(24, 2, (b, T, hd), orc.E4M3)
    check_against_oracle(Q, orc.E4M3, 1.0, Kt, orc.E4M3, 1.0, False, True)
    P = si.scaled_normal(24, 3, (b, T, T), orc.E4M3, 0.25)
    V = si.scaled_normal(24, 4, (b, T, hd), orc.E4M3)
    check_against_oracle(P, orc.E4M3, 1.0, V, orc.E4M3, 1.0, False, False)
    # shared 2-D weight for every batch
    W = si.scaled_normal(24, 5, (hd, 96), orc.E4M3)
    check_against_oracle(Q, orc.E4M3, 1.0, W, orc.E4M3, 2.0 ** -6, False, False)


@pytest.mark.parametrize("kind", ["fwd", "grad"])
def test_config2_1024_full_compare_with_fused_amax_rescale_to_e4m3(kind):
    c = si.gemm_case(1024, kind, seed=1)
    check_against_oracle(c["A"], c["a_dtype"], c["a_scale"], c["Bt"], c["b_dtype"], c["b_scale"], False, True)
    for stat in (sc.STAT_AMAX, sc.STAT_L2):
        g = run_matmul(c["A"], c["a_dtype"], c["a_scale"], c["Bt"], c["b_dtype"], c["b_scale"], orc.BF16, False, True,
                       stat=stat, q_dt=orc.E4M3)
        assert g["status"] == 0
        so = orc.statistic(g["Y"], orc.BF16, stat)
        if stat == sc.STAT_AMAX:
            assert g["stat"] == so
        else:
            assert abs(g["stat"] - so) <= 2e-6 * so
            assert abs(so / orc.p2f(so) - 1.5) < 0.499  # not at a binade edge
        yq, yqs, _ = orc.rescale(g["Y"], orc.BF16, g["y_scale"], stat, orc.E4M3)
        assert g["yq_scale"] == yqs
        assert np.array_equal(g["Yq"], yq)


@pytest.mark.parametrize("n,kind", [(4096, "fwd"), (8192, "fwd"), (8192, "grad")])
def test_config2_full_size_sampled_outputs_and_properties(n, kind):
    c = si.gemm_case(n, kind, seed=2)
    g = run_matmul(c["A"], c["a_dtype"], c["a_scale"], c["Bt"], c["b_dtype"], c["b_scale"], orc.BF16, False, True,
                   stat=sc.STAT_AMAX, q_dt=orc.E4M3)
    assert g["status"] == 0
    assert g["y_scale"] == c["a_scale"] * c["b_scale"] * orc.kf(n)
    rng = np.random.default_rng(5)
    rows = np.concatenate([rng.integers(0, n, 2000), [0, n - 1, 127, 128, n - 129]])
    cols = np.concatenate([rng.integers(0, n, 2000), [0, n - 1, 255, 256, n - 257]])
    acc, sab = orc.scaled_matmul_samples(c["A"], c["a_dtype"], c["Bt"], c["b_dtype"], rows, cols, transB=True)
    want = orc.encode(acc, orc.BF16)
    got = g["Y"][rows, cols]
    assert within(got, want, orc.BF16, acc, sab, 1e-5).all()
    # properties that hold at any size: statistic word = AMAX of the stored output; the rescaled
    # output is the exact power-of-two rebalance of the stored intermediate
    yv = torch.from_numpy(g["Y"].view(np.int16)).view(torch.bfloat16).float()
    amax = float(yv.abs().max())
    assert g["stat"] == amax
    r = orc.p2f(amax)
    assert g["yq_scale"] == g["y_scale"] * r
    want_q = (yv / r).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(g["Yq"], want_q)
    assert 1.0 <= float(torch.from_numpy(g["Yq"]).view(torch.float8_e4m3fn).float().abs().max()) <= 2.0


def test_accumulator_precision_with_adversarial_magnitudes():
    # one large product followed by many small ones of the same sign: a narrow accumulator would
    # lose the small terms.  Bound: 1e-5 * sum|a*b|.
    M, N, K = 128, 256, 8192
    a = np.full((M, K), 2.0 ** -3, dtype=np.float32)
    a[:, 0] = 256.0
    b = np.full((N, K), 2.0 ** -3, dtype=np.float32)
    b[:, 0] = 256.0
    A, Bt = si.to_bits(a, orc.E4M3), si.to_bits(b, orc.E4M3)
    g = run_matmul(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, orc.F32, False, True)
    exact = (65536.0 + (K - 1) * 2.0 ** -6) / orc.kf(K)
    got = g["Y"].view(np.float32).astype(np.float64)
    assert np.all(np.abs(got - exact) <= 1e-5 * exact), float(np.abs(got - exact).max() / exact)


def test_bad_scale_is_reported_in_status_word():
    A = si.scaled_normal(25, 1, (128, 128), orc.E4M3)
    Bt = si.scaled_normal(25, 2, (256, 128), orc.E4M3)
    g = run_matmul(A, orc.E4M3, 3.0, Bt, orc.E4M3, 1.0, orc.BF16, False, True)
    assert g["status"] & sc.DEV_BAD_SCALE


# ---------------------------------------------------------------- delayed rescaling: one kernel, FP8 out

def run_delayed(A, a_dt, a_s, B, b_dt, b_s, stat_in, y_dt, transB=True, stat=sc.STAT_AMAX, state=None):
    M = A.shape[0]
    N = B.shape[0] if transB else B.shape[1]
    Y = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[y_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    st_in = state if state is not None else torch.tensor([stat_in], dtype=torch.float32, device="cuda")
    st_out = state if state is not None else torch.zeros(1, dtype=torch.float32, device="cuda")
    sc.scalify_scaled_matmul_delayed(sc.ScaledTensor.make(to_dev(A, a_dt), a_s), sc.ScaledTensor.make(to_dev(B, b_dt), b_s),
                                     st_in, Y, ws, transB=transB, stat=stat, stat_out=st_out)
    status = ws.check_status()
    return to_bits(Y.data, y_dt), Y.scale_value(), float(st_out.item()), status


@pytest.mark.parametrize("a_dt,y_dt", [(orc.E4M3, orc.E4M3), (orc.E5M2, orc.E5M2), (orc.E4M3, orc.BF16)])
@pytest.mark.parametrize("stat", [sc.STAT_AMAX, sc.STAT_L2])
def test_delayed_rescale_matmul_single_pass_fp8_output(a_dt, y_dt, stat):
    M, N, K = 384, 528, 1040
    A = si.scaled_normal(26, 1, (M, K), a_dt)
    Bt = si.scaled_normal(26, 2, (N, K), orc.E4M3)
    for stat_in in (5.3, 0.07, 0.0):
        got, gs, gstat, status = run_delayed(A, a_dt, 2.0 ** -10, Bt, orc.E4M3, 2.0 ** -6, stat_in, y_dt, stat=stat)
        assert status == 0
        Yo, ys, so = orc.scaled_matmul_delayed(A, a_dt, 2.0 ** -10, Bt, orc.E4M3, 2.0 ** -6, stat_in, stat, y_dt,
                                               transB=True)
        assert gs == ys
        assert abs(gstat - so) <= 2e-5 * so
        _, _, acc, sab = orc.scaled_matmul(A, a_dt, 2.0 ** -10, Bt, orc.E4M3, 2.0 ** -6, orc.F32, transB=True,
                                           want_acc=True)
        r = orc.p2f(stat_in) if stat_in >= 2.0 ** -126 else 1.0
        assert within(got, Yo, y_dt, acc / r, sab / r, 1e-5).all()
        # bit-exact against the encoding of the library's own fp32 values
        g32, _, _, _ = run_delayed(A, a_dt, 2.0 ** -10, Bt, orc.E4M3, 2.0 ** -6, stat_in, orc.F32, stat=stat)
        assert np.array_equal(got, orc.encode(orc.decode(g32, orc.F32), y_dt))


def test_delayed_rescale_state_word_updated_in_place_over_steps():
    M, N, K = 256, 256, 512
    state = torch.tensor([1.0], dtype=torch.float32, device="cuda")  # initial guess of the statistic
    prev = 1.0
    for step in range(3):
        A = si.scaled_normal(27, 10 + step, (M, K), orc.E4M3, 1.0 + step)  # the data grow from step to step
        Bt = si.scaled_normal(27, 20 + step, (N, K), orc.E4M3)
        got, gs, gstat, status = run_delayed(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, None, orc.E4M3, state=state)
        Yo, ys, so = orc.scaled_matmul_delayed(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, prev, orc.STAT_AMAX, orc.E4M3,
                                               transB=True)
        assert status == 0 and gs == ys and abs(gstat - so) <= 2e-5 * so
        assert ulp_diff(got, Yo, orc.E4M3).max() <= 1
        prev = gstat  # the library's own statistic drives the next step on both sides


def test_delayed_rescale_nonfinite_statistic_is_flagged_and_ignored():
    A = si.scaled_normal(28, 1, (128, 128), orc.E4M3)
    Bt = si.scaled_normal(28, 2, (256, 128), orc.E4M3)
    got, gs, gstat, status = run_delayed(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, float("inf"), orc.BF16)
    assert status == sc.DEV_NONFINITE_STAT
    Yo, ys, _ = orc.scaled_matmul_delayed(A, orc.E4M3, 1.0, Bt, orc.E4M3, 1.0, float("inf"), orc.STAT_AMAX, orc.BF16,
                                          transB=True)
    assert gs == ys and ulp_diff(got, Yo, orc.BF16).max() <= 1


def test_delayed_rescale_full_size_8192_sampled():
    n = 8192
    c = si.gemm_case(n, "fwd", seed=2)
    stat_in = 6.0
    got, gs, gstat, status = run_delayed(c["A"], orc.E4M3, c["a_scale"], c["Bt"], orc.E4M3, c["b_scale"], stat_in, orc.E4M3)
    assert status == 0 and gs == c["a_scale"] * c["b_scale"] * orc.kf(n) * 4.0
    rng = np.random.default_rng(6)
    rows = np.concatenate([rng.integers(0, n, 2000), [0, n - 1, 255, 256]])
    cols = np.concatenate([rng.integers(0, n, 2000), [0, n - 1, 255, 256]])
    acc, sab = orc.scaled_matmul_samples(c["A"], orc.E4M3, c["Bt"], orc.E4M3, rows, cols, transB=True)
    want = orc.encode(acc / 4.0, orc.E4M3)
    assert within(got[rows, cols], want, orc.E4M3, acc / 4.0, sab / 4.0, 1e-5).all()
    # the statistic is the AMAX of the un-rebalanced values: at least the max over the sample, and
    # consistent with the stored FP8 data (|data| * r <= stat rounded up by one FP8 ulp)
    assert gstat >= np.abs(acc).max() * (1 - 1e-5)
    stored_max = float(torch.from_numpy(got).view(torch.float8_e4m3fn).float().abs().max()) * 4.0
    assert stored_max * (1 - 2.0 ** -4) <= gstat <= stored_max * (1 + 2.0 ** -4)


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (520, 304, 384), (100, 48, 128)])
@pytest.mark.parametrize("y_dt,q_dt", [(orc.BF16, orc.E4M3), (orc.F16, orc.E5M2)])
def test_speculative_rescale_is_the_exact_dynamic_rescale(M, N, K, y_dt, q_dt):
    """Whatever the predicted statistic is (right binade, wrong binade either way, zero, NaN), the intermediate,
    the FP8 output, both scale words and the statistic equal those of the plain call bit for bit, and the hint
    leaves as this call's statistic."""
    A = si.to_bits(si.normal(81, M + K, (M, K), 1.0), orc.E4M3)
    B = si.to_bits(si.normal(82, N + K, (N, K), 1.0), orc.E5M2)
    plain = run_matmul(A, orc.E4M3, 2.0 ** -2, B, orc.E5M2, 2.0 ** 3, y_dt, transB=True, stat=sc.STAT_AMAX, q_dt=q_dt)
    assert plain["status"] == 0
    stat = plain["stat"]
    # the plain path itself against the oracle's rescale of its own intermediate
    qo, qs, _ = orc.rescale(plain["Y"].reshape(-1), y_dt, plain["y_scale"], orc.STAT_AMAX, q_dt)
    assert plain["yq_scale"] == qs and np.array_equal(plain["Yq"].reshape(-1), qo)
    Ad = sc.ScaledTensor.make(to_dev(A, orc.E4M3), 2.0 ** -2)
    Bd = sc.ScaledTensor.make(to_dev(B, orc.E5M2), 2.0 ** 3)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    for hint in (stat, stat * 1.3, stat / 1.3, stat * 64.0, stat / 1000.0, 0.0, float("nan"), float("inf")):
        Y = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[y_dt])
        Yq = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[q_dt])
        Yq.data.view(torch.uint8).fill_(0x55)
        h = torch.tensor([hint], dtype=torch.float32, device="cuda")
        sc.scalify_scaled_matmul_speculative(Ad, Bd, Y, Yq, h, ws, transB=True)
        assert ws.check_status() == 0
        assert float(h.item()) == stat and float(ws.statistic().item()) == stat
        assert Y.scale_value() == plain["y_scale"] and Yq.scale_value() == plain["yq_scale"]
        assert np.array_equal(to_bits(Y.data, y_dt), plain["Y"])
        assert np.array_equal(to_bits(Yq.data, q_dt), plain["Yq"]), hint


@pytest.mark.parametrize("M,N,K,transA,transB", [(768, 768, 8192, True, False), (300, 528, 4096, False, True),
                                                  (144, 272, 2048, True, True), (64, 1040, 6144, False, False)])
def test_split_contraction_with_a_large_workspace(M, N, K, transA, transB):
    """Few output tiles and a long K (weight gradients): with the larger workspace the K range is split, the
    partial products are added in a fixed order by a second launch.  Same bars as the single launch; the fused
    statistic and the rescaled output are those of the stored result."""
    a = si.to_bits(si.normal(31, M, (K, M) if transA else (M, K), 1.0), orc.E4M3)
    b = si.to_bits(si.normal(32, N, (N, K) if transB else (K, N), 1.0), orc.E5M2)
    check_against_oracle(a, orc.E4M3, 2.0 ** -2, b, orc.E5M2, 2.0 ** -9, transA, transB, splitk=True)
    for stat in (sc.STAT_AMAX, sc.STAT_L2):
        g = run_matmul(a, orc.E4M3, 2.0 ** -2, b, orc.E5M2, 2.0 ** -9, orc.BF16, transA, transB, stat=stat, q_dt=orc.E5M2,
                       splitk=True)
        assert g["status"] == 0
        want_stat = orc.statistic(g["Y"], orc.BF16, stat)
        assert g["stat"] == want_stat if stat == sc.STAT_AMAX else abs(g["stat"] - want_stat) <= 2e-6 * want_stat
        yq, ys, _ = orc.rescale(g["Y"], orc.BF16, g["y_scale"], stat, orc.E5M2, stat_override=g["stat"])
        assert g["yq_scale"] == ys and np.array_equal(g["Yq"], yq)
        # replays give the same bits (fixed summation order)
        g2 = run_matmul(a, orc.E4M3, 2.0 ** -2, b, orc.E5M2, 2.0 ** -9, orc.BF16, transA, transB, stat=stat, q_dt=orc.E5M2,
                        splitk=True)
        assert np.array_equal(g["Y"], g2["Y"]) and g["stat"] == g2["stat"]
    if K == 8192:
        # the split did happen: fp32 sums in another order differ somewhere from the single launch's
        one = run_matmul(a, orc.E4M3, 2.0 ** -2, b, orc.E5M2, 2.0 ** -9, orc.F32, transA, transB)
        many = run_matmul(a, orc.E4M3, 2.0 ** -2, b, orc.E5M2, 2.0 ** -9, orc.F32, transA, transB, splitk=True)
        assert not np.array_equal(one["Y"], many["Y"])


@pytest.mark.parametrize("M,N,K,transB", [(256, 256, 256, True), (520, 304, 384, False), (100, 48, 128, True),
                                          (8192, 768, 768, False)])
@pytest.mark.parametrize("y_dt,bias_dt", [(orc.BF16, orc.BF16), (orc.F32, orc.F32), (orc.E4M3, orc.F16)])
def test_matmul_with_bias_in_the_epilogue(M, N, K, transB, y_dt, bias_dt):
    """Y = A B + bias by the add rule with ONE rounding: Y_s = max(A_s B_s kf(K), bias_s), both terms brought to
    it by exact powers of two.  The exact value comes from the oracle's exact accumulation; bars as for the
    plain matmul (1 ulp of the output format, or half an ulp plus 1e-5 of the summed magnitudes)."""
    a = si.to_bits(si.normal(51, M, (M, K), 1.0), orc.E4M3)
    b = si.to_bits(si.normal(52, N, (N, K) if transB else (K, N), 1.0), orc.E4M3)
    for a_s, b_s, bias_s in ((2.0 ** -3, 2.0 ** -6, 2.0 ** -6), (1.0, 2.0 ** -6, 2.0 ** 2)):
        bias = si.to_bits(si.normal(53, N, (N,), 1.0), bias_dt)
        A = sc.ScaledTensor.make(to_dev(a, orc.E4M3), a_s)
        B = sc.ScaledTensor.make(to_dev(b, orc.E4M3), b_s)
        Bi = sc.ScaledTensor.make(to_dev(bias, bias_dt), bias_s)
        Y = sc.ScaledTensor.empty((M, N), sc.TORCH_DTYPE[y_dt])
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
        sc.scalify_scaled_matmul_bias(A, B, Bi, Y, ws, transB=transB, stat=sc.STAT_AMAX)
        assert ws.check_status() == 0
        rows = np.arange(M) if M <= 520 else np.random.default_rng(1).integers(0, M, 300)
        _, ab_s, acc, sab = orc.scaled_matmul(a[rows], orc.E4M3, a_s, b, orc.E4M3, b_s, orc.F32, transB=transB,
                                              want_acc=True)
        kf = orc.kf(K)
        assert ab_s == a_s * b_s * kf
        ys = max(ab_s, bias_s)
        assert Y.scale_value() == ys
        fa, fb = ab_s / ys, bias_s / ys
        bv = orc.decode(bias, bias_dt)
        exact = acc * fa + bv[None, :] * fb          # acc: the exact data component of the product, (A_d B_d) / kf(K)
        mag = sab * fa + np.abs(bv)[None, :] * fb
        got = to_bits(Y.data, y_dt)[rows]
        ok = within(got, orc.encode(exact, y_dt), y_dt, exact, mag, 1e-5)
        assert ok.all(), int((~ok).sum())
        if M <= 520:
            assert float(ws.statistic().item()) == float(np.abs(orc.decode(got, y_dt)).max())


def _two_pass_reference(Ad, Bd, shape, y_dt, q_dt, **kw):
    """The unpredicted path: GEMM with fused AMAX into the 16-bit intermediate, then the rebalance pass."""
    Y = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[y_dt])
    Yq = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[q_dt])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, shape[-2] * (shape[0] if len(shape) == 3 else 1), shape[-1]))
    sc.scalify_scaled_matmul(Ad, Bd, Y, ws, stat=sc.STAT_AMAX, **kw)
    sc.scalify_rescale(Y, Yq, stat=sc.STAT_AMAX, stat_in=ws.statistic())
    assert ws.check_status() == 0
    return dict(Y=to_bits(Y.data, y_dt), Yq=to_bits(Yq.data, q_dt), y_scale=Y.scale_value(), yq_scale=Yq.scale_value(),
                stat=float(ws.statistic().item()))


@pytest.mark.parametrize("shape_a,shape_b,transB", [((256, 256), (256, 256), True), ((520, 384), (384, 304), False),
                                                     ((100, 128), (48, 128), True), ((3, 300, 192), (3, 272, 192), True),
                                                     ((1024, 512), (768, 512), True)])
@pytest.mark.parametrize("q_dt", [orc.E4M3, orc.E5M2])
def test_main_call_predicts_the_rescale_and_the_fp8_only_form_is_bit_identical(shape_a, shape_b, transB, q_dt):
    """scalify_scaled_matmul(..., AMAX, Yq) lets the GEMM write the FP8 output with the power of two of the
    statistic its workspace saw last, and with Y = None stores nothing else.  For a fresh workspace, a right, a
    wrong and a degenerate prediction alike: Y, Yq, both scale words and the statistic word are those of the
    two-pass path (GEMM + AMAX, then the rebalance pass) bit for bit, and the prediction word leaves as this
    call's statistic."""
    A = si.to_bits(si.normal(91, 1, shape_a, 1.0), orc.E4M3)
    B = si.to_bits(si.normal(92, 2, shape_b, 1.0), orc.E5M2)
    Ad = sc.ScaledTensor.make(to_dev(A, orc.E4M3), 2.0 ** -2)
    Bd = sc.ScaledTensor.make(to_dev(B, orc.E5M2), 2.0 ** 3)
    M, N = shape_a[-2], (shape_b[-2] if transB else shape_b[-1])
    shape = (M, N) if len(shape_a) == 2 else (shape_a[0], M, N)
    ref = _two_pass_reference(Ad, Bd, shape, orc.BF16, q_dt, transB=transB)
    qo, qs, _ = orc.rescale(ref["Y"].reshape(-1), orc.BF16, ref["y_scale"], orc.STAT_AMAX, q_dt)
    assert ref["yq_scale"] == qs and np.array_equal(ref["Yq"].reshape(-1), qo)
    stat = ref["stat"]
    rows = M * (shape[0] if len(shape) == 3 else 1)
    for fp8_only in (False, True):
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, rows, N))
        for k, hint in enumerate((None, None, stat * 1.3, stat * 64.0, stat / 1000.0, float("nan"), float("inf"), stat)):
            if hint is not None:
                ws.prediction().fill_(hint)      # (None: what the workspace holds: zero at first, then the statistic)
            Y = None if fp8_only else sc.ScaledTensor.empty(shape, torch.bfloat16)
            Yq = sc.ScaledTensor.empty(shape, sc.TORCH_DTYPE[q_dt])
            Yq.data.view(torch.uint8).fill_(0x55)
            sc.scalify_scaled_matmul(Ad, Bd, Y, ws, transB=transB, stat=sc.STAT_AMAX, Yq=Yq)
            assert ws.check_status() == 0
            assert float(ws.statistic().item()) == stat and float(ws.prediction().item()) == stat, (fp8_only, k)
            assert Yq.scale_value() == ref["yq_scale"]
            assert np.array_equal(to_bits(Yq.data, q_dt), ref["Yq"]), (fp8_only, k, hint)
            if Y is not None:
                assert Y.scale_value() == ref["y_scale"] and np.array_equal(to_bits(Y.data, orc.BF16), ref["Y"])


def test_fp8_only_form_argument_checks():
    A = sc.ScaledTensor.make(to_dev(si.to_bits(si.normal(93, 1, (64, 128), 1.0), orc.E4M3), orc.E4M3), 1.0)
    B = sc.ScaledTensor.make(to_dev(si.to_bits(si.normal(93, 2, (40, 128), 1.0), orc.E4M3), orc.E4M3), 1.0)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, 64, 40))
    Yq = sc.ScaledTensor.empty((64, 40), torch.float8_e4m3fn)
    with pytest.raises(sc.ScalifyError) as e:      # rows of 40 bytes: not a multiple of 16
        sc.scalify_scaled_matmul(A, B, None, ws, transB=True, stat=sc.STAT_AMAX, Yq=Yq)
    assert e.value.code == -4
    B16 = sc.ScaledTensor.make(to_dev(si.to_bits(si.normal(93, 3, (48, 128), 1.0), orc.E4M3), orc.E4M3), 1.0)
    Yq16 = sc.ScaledTensor.empty((64, 48), torch.float8_e4m3fn)
    for bad in (dict(stat=sc.STAT_L2, Yq=Yq16), dict(stat=sc.STAT_NONE, Yq=Yq16), dict(stat=sc.STAT_AMAX, Yq=None),
                dict(stat=sc.STAT_AMAX, Yq=sc.ScaledTensor.empty((64, 48), torch.bfloat16))):
        with pytest.raises(sc.ScalifyError):
            sc.scalify_scaled_matmul(A, B16, None, ws, transB=True, **bad)
