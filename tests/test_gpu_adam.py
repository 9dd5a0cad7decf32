"""GPU parity of the scaled Adam step against the oracle: scale words bit-exact
(closed form of the static rules), FP16 / FP32 / BF16 outputs within 1 ulp."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff, within

pytestmark = pytest.mark.gpu


def run_case(sizes, w_dt, mv_dt=orc.F16, g_dt=orc.E5M2, step=1000, seed=51, scales=None):
    cases = []
    G, M, V, W = [], [], [], []
    for i, n in enumerate(sizes):
        c = si.adam_case(n, seed=seed + i, w_dtype=w_dt if w_dt != orc.BF16 else orc.F16)
        if w_dt == orc.BF16:
            c["w"] = si.to_bits(si.normal(seed + i, 1, (n,), 0.02 * 64.0), orc.BF16)
            c["w_dtype"] = orc.BF16
        if mv_dt == orc.F32:
            c["m"] = orc.encode(orc.decode(c["m"], orc.F16), orc.F32)
            c["v"] = orc.encode(orc.decode(c["v"], orc.F16), orc.F32)
            c["mv_dtype"] = orc.F32
        if g_dt != orc.E5M2:
            c["g"] = orc.encode(orc.decode(c["g"], orc.E5M2), g_dt)
            c["g_dtype"] = g_dt
        if scales:
            c.update(scales)
        cases.append(c)
        G.append(sc.ScaledTensor.make(to_dev(c["g"], c["g_dtype"]), c["g_scale"]))
        M.append(sc.ScaledTensor.make(to_dev(c["m"], c["mv_dtype"]), c["m_scale"]))
        V.append(sc.ScaledTensor.make(to_dev(c["v"], c["mv_dtype"]), c["v_scale"]))
        W.append(sc.ScaledTensor.make(to_dev(c["w"], c["w_dtype"]), c["w_scale"]))
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(sizes)))
    tens = sc.AdamTensors(G, M, V, W)
    c0 = cases[0]
    sc.scalify_scaled_adam_step(tens, ws, lr=c0["lr"], beta1=c0["beta1"], beta2=c0["beta2"], eps=c0["eps"], step=step)
    assert ws.check_status() == 0
    for c, g, m, v, w in zip(cases, G, M, V, W):
        mo, vo, wo, ms, vs, wsc = orc.adam_step(c["g"], c["g_dtype"], c["g_scale"], c["m"], c["v"], c["mv_dtype"],
                                                c["m_scale"], c["v_scale"], c["w"], c["w_dtype"], c["w_scale"],
                                                c["lr"], c["beta1"], c["beta2"], c["eps"], step)
        assert (m.scale_value(), v.scale_value(), w.scale_value()) == (ms, vs, wsc)
        assert ulp_diff(to_bits(m.data, c["mv_dtype"]), mo, c["mv_dtype"]).max() <= (1 if mv_dt != orc.F32 else 4)
        assert ulp_diff(to_bits(v.data, c["mv_dtype"]), vo, c["mv_dtype"]).max() <= (1 if mv_dt != orc.F32 else 4)
        # w' = w - update in fp32: where the two cancel the error is relative to |w| + |update|
        wv = orc.decode(c["w"], c["w_dtype"]) * c["w_scale"]
        exact = orc.decode(wo, c["w_dtype"]) if c["w_dtype"] != orc.F32 else None
        w_new = orc.decode(orc.adam_step(c["g"], c["g_dtype"], c["g_scale"], c["m"], c["v"], c["mv_dtype"],
                                         c["m_scale"], c["v_scale"], orc.encode(orc.decode(c["w"], c["w_dtype"]),
                                                                                orc.F32), orc.F32, c["w_scale"],
                                         c["lr"], c["beta1"], c["beta2"], c["eps"], step)[2], orc.F32)
        mag = (np.abs(wv) + np.abs(w_new * wsc - wv)) / wsc
        ok = within(to_bits(w.data, c["w_dtype"]), wo, c["w_dtype"], w_new, mag, 8 * 2.0 ** -24)
        assert ok.all(), int((~ok).sum())
        # gradients are read-only
        assert np.array_equal(to_bits(g.data, c["g_dtype"]), c["g"])


@pytest.mark.parametrize("w_dt", [orc.F16, orc.F32, orc.BF16])
def test_single_tensor_ragged_sizes(w_dt):
    for n in (1, 7, 8, 1000, 8192 + 3, 256 * 8 * 4 * 3 + 9):
        run_case([n], w_dt)


@pytest.mark.parametrize("w_dt,mv_dt", [(orc.F16, orc.F16), (orc.F32, orc.F32)])
def test_multi_tensor_list(w_dt, mv_dt):
    sizes = [768, 2304, 768 * 64, 5, 8193, 3072, 1, 50257 * 8]
    run_case(sizes, w_dt, mv_dt=mv_dt)


def test_more_tensors_than_one_launch_holds():
    run_case([64 + (i % 7) for i in range(170)], orc.F16)


@pytest.mark.parametrize("step", [1, 2, 100000])
def test_bias_correction_steps(step):
    run_case([4096], orc.F16, step=step)


def test_bf16_gradients_and_other_scales():
    run_case([10000], orc.F32, g_dt=orc.BF16, scales=dict(g_scale=2.0 ** -3, m_scale=2.0 ** -2, v_scale=2.0 ** -9,
                                                           w_scale=2.0 ** 1))


def test_gpt2_small_parameter_list_shapes():
    # the 148 tensors of the GPT-2-small-shaped list, scaled down 16x in the large dimensions to stay quick
    shapes = si.gpt2_small_param_shapes()
    sizes = [max(1, int(np.prod(s)) // 16) for s in shapes]
    assert len(sizes) == 148
    run_case(sizes, orc.F16)


def _sampled_adam_parity(tensors_np, G, M, V, W, hyper, step, rng, n_samples):
    """Adam is elementwise: gather a sample of elements of each tensor, run the oracle on the sample with
    the tensor's scales and compare with the library's result at the same positions."""
    for c, g, m, v, w in zip(tensors_np, G, M, V, W):
        n = c["g"].size
        idx = np.unique(np.concatenate([rng.integers(0, n, min(n_samples, n)), [0, n - 1]]))
        mo, vo, wo, ms, vs, wsc = orc.adam_step(c["g"][idx], orc.E5M2, c["g_scale"], c["m"][idx], c["v"][idx], orc.F16,
                                                c["m_scale"], c["v_scale"], c["w"][idx], orc.F16, c["w_scale"],
                                                hyper["lr"], hyper["beta1"], hyper["beta2"], hyper["eps"], step)
        assert (m.scale_value(), v.scale_value(), w.scale_value()) == (ms, vs, wsc)
        tidx = torch.from_numpy(idx).cuda()
        assert ulp_diff(to_bits(m.data[tidx], orc.F16), mo, orc.F16).max() <= 1
        assert ulp_diff(to_bits(v.data[tidx], orc.F16), vo, orc.F16).max() <= 1
        assert ulp_diff(to_bits(w.data[tidx], orc.F16), wo, orc.F16).max() <= 1


def test_config4_flat_125m_parameters_sampled():
    """Full benchmark size, in the launch configuration the benchmark times: one flat tensor of 125M
    parameters; 200k sampled elements against the oracle."""
    n = 125_000_000
    c = si.adam_case(n, seed=4)
    G = [sc.ScaledTensor.make(to_dev(c["g"], orc.E5M2), c["g_scale"])]
    M = [sc.ScaledTensor.make(to_dev(c["m"], orc.F16), c["m_scale"])]
    V = [sc.ScaledTensor.make(to_dev(c["v"], orc.F16), c["v_scale"])]
    W = [sc.ScaledTensor.make(to_dev(c["w"], orc.F16), c["w_scale"])]
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1))
    hyper = dict(lr=c["lr"], beta1=c["beta1"], beta2=c["beta2"], eps=c["eps"])
    sc.scalify_scaled_adam_step(sc.AdamTensors(G, M, V, W), ws, step=c["step"], **hyper)
    assert ws.check_status() == 0
    _sampled_adam_parity([c], G, M, V, W, hyper, c["step"], np.random.default_rng(7), 200_000)


def test_config4_gpt2_small_parameter_list_full_size_sampled():
    """The 148 tensors (124,439,808 parameters) of the GPT-2-small-shaped list in one call."""
    shapes = si.gpt2_small_param_shapes()
    sizes = [int(np.prod(s)) for s in shapes]
    assert len(sizes) == 148 and sum(sizes) == 124_439_808
    cases, G, M, V, W = [], [], [], [], []
    for i, n in enumerate(sizes):
        c = si.adam_case(n, seed=400 + i)
        cases.append(c)
        G.append(sc.ScaledTensor.make(to_dev(c["g"], orc.E5M2), c["g_scale"]))
        M.append(sc.ScaledTensor.make(to_dev(c["m"], orc.F16), c["m_scale"]))
        V.append(sc.ScaledTensor.make(to_dev(c["v"], orc.F16), c["v_scale"]))
        W.append(sc.ScaledTensor.make(to_dev(c["w"], orc.F16), c["w_scale"]))
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(sizes)))
    hyper = dict(lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8)
    sc.scalify_scaled_adam_step(sc.AdamTensors(G, M, V, W), ws, step=1000, **hyper)
    assert ws.check_status() == 0
    _sampled_adam_parity(cases, G, M, V, W, hyper, 1000, np.random.default_rng(8), 2000)


@pytest.mark.parametrize("w_dt,c_dt", [(orc.F16, orc.E4M3), (orc.F32, orc.E4M3), (orc.F32, orc.BF16),
                                       (orc.BF16, orc.E5M2), (orc.F32, orc.F16)])
def test_adam_step_with_compute_copy(w_dt, c_dt):
    """The step that also emits the low-precision compute copy: m, v, w and their scales are bit-identical
    to the plain step, and the copy is the oracle's static cast of the weight as stored, with w's new scale."""
    sizes = [1, 13, 4096, 8192 * 3 + 5, 777]
    lists = []
    for variant in range(2):
        G, M, V, W, cases = [], [], [], [], []
        for i, n in enumerate(sizes):
            c = si.adam_case(n, seed=90 + i, w_dtype=w_dt if w_dt != orc.BF16 else orc.F16)
            if w_dt == orc.BF16:
                c["w"] = si.to_bits(si.normal(90 + i, 1, (n,), 0.02 * 64.0), orc.BF16)
                c["w_dtype"] = orc.BF16
            cases.append(c)
            G.append(sc.ScaledTensor.make(to_dev(c["g"], c["g_dtype"]), c["g_scale"]))
            M.append(sc.ScaledTensor.make(to_dev(c["m"], c["mv_dtype"]), c["m_scale"]))
            V.append(sc.ScaledTensor.make(to_dev(c["v"], c["mv_dtype"]), c["v_scale"]))
            W.append(sc.ScaledTensor.make(to_dev(c["w"], c["w_dtype"]), c["w_scale"]))
        lists.append((G, M, V, W, cases))
    c0 = lists[0][4][0]
    hyper = dict(lr=c0["lr"], beta1=c0["beta1"], beta2=c0["beta2"], eps=c0["eps"], step=7)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(sizes)))
    sc.scalify_scaled_adam_step(sc.AdamTensors(*lists[0][:4]), ws, **hyper)
    WC = [sc.ScaledTensor.make(torch.zeros(n, dtype=sc.TORCH_DTYPE[c_dt], device="cuda"), 123.0) for n in sizes]
    sc.scalify_scaled_adam_step_cast(sc.AdamTensors(*lists[1][:4]), WC, ws, **hyper)
    assert ws.check_status() == 0
    for k in range(len(sizes)):
        for a, b, dt in ((lists[0][1][k], lists[1][1][k], orc.F16), (lists[0][2][k], lists[1][2][k], orc.F16),
                         (lists[0][3][k], lists[1][3][k], w_dt)):
            assert a.scale_value() == b.scale_value()
            assert np.array_equal(to_bits(a.data, dt), to_bits(b.data, dt))
        w_bits = to_bits(lists[1][3][k].data, w_dt)
        want = orc.encode(orc.decode(w_bits, w_dt), c_dt)
        assert np.array_equal(to_bits(WC[k].data, c_dt), want)
        assert WC[k].scale_value() == lists[1][3][k].scale_value()


def test_adam_step_with_compute_copy_rejects_bad_arguments():
    n = 64
    c = si.adam_case(n, seed=5, w_dtype=orc.F16)
    G = [sc.ScaledTensor.make(to_dev(c["g"], c["g_dtype"]), c["g_scale"])]
    M = [sc.ScaledTensor.make(to_dev(c["m"], c["mv_dtype"]), c["m_scale"])]
    V = [sc.ScaledTensor.make(to_dev(c["v"], c["mv_dtype"]), c["v_scale"])]
    W = [sc.ScaledTensor.make(to_dev(c["w"], c["w_dtype"]), c["w_scale"])]
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1))
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    before = to_bits(W[0].data, orc.F16).copy()
    # a copy as wide as the weight is not a compute copy
    with pytest.raises(sc.ScalifyError):
        sc.scalify_scaled_adam_step_cast(sc.AdamTensors(G, M, V, W),
                                         [sc.ScaledTensor.make(torch.zeros(n, dtype=torch.float16, device="cuda"), 1.0)],
                                         ws, **hyper)
    # wrong element count
    with pytest.raises(sc.ScalifyError):
        sc.scalify_scaled_adam_step_cast(sc.AdamTensors(G, M, V, W),
                                         [sc.ScaledTensor.make(torch.zeros(n + 16, dtype=torch.float8_e4m3fn,
                                                                           device="cuda"), 1.0)], ws, **hyper)
    # a failed call launched nothing
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(W[0].data, orc.F16), before)
