"""The workspace-free Adam entry point against the ordinary one.

`scalify_scaled_adam_step_static` serves callers that cannot allocate a workspace (their own
memory pool already holds the whole device, or they must avoid cudaMalloc's synchronisation);
its scratch is a fixed array inside the library.  It runs the same kernels, so its results
must be identical, bit for bit, to those of `scalify_scaled_adam_step` - on a first call and on
a second call that finds the first call's leftovers in the shared array - and, like them, within
one FP16 ulp of the oracle's step with exactly the oracle's scale words.  This file is collected
last on purpose: a failure here stops a `-x` run only after every other test ran.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev, to_bits, ulp_diff

pytestmark = pytest.mark.gpu


def make_state(sizes, seed):
    out = []
    for i, n in enumerate(sizes):
        c = si.adam_case(n, seed=seed + i)
        out.append([sc.ScaledTensor.make(to_dev(c["g"], si.E5M2), c["g_scale"]),
                    sc.ScaledTensor.make(to_dev(c["m"], si.F16), c["m_scale"]),
                    sc.ScaledTensor.make(to_dev(c["v"], si.F16), c["v_scale"]),
                    sc.ScaledTensor.make(to_dev(c["w"], si.F16), c["w_scale"])])
    cols = list(zip(*out))
    return sc.AdamTensors(*cols)


def snapshot(t):
    return [(to_bits(x.data, dt), x.scale_value()) for lst, dt in ((t.keep[1], si.F16), (t.keep[2], si.F16),
                                                                   (t.keep[3], si.F16)) for x in lst]


def test_static_adam_matches_workspace_adam_on_two_calls_in_a_row():
    sizes = [4096, 1, 777, 50000, 8]
    hyper = dict(lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8)
    ref = make_state(sizes, 91)
    new = make_state(sizes, 91)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(sizes)))
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for step in (1000, 1001):  # the second call meets the scratch contents of the first
        before = [(to_bits(g.data, si.E5M2), g.scale_value(), to_bits(m.data, si.F16), m.scale_value(),
                   to_bits(v.data, si.F16), v.scale_value(), to_bits(w.data, si.F16), w.scale_value())
                  for g, m, v, w in zip(*new.keep)]
        sc.scalify_scaled_adam_step(ref, ws, step=step, **hyper)
        sc.scalify_scaled_adam_step_static(new, step=step, status_out=status, **hyper)
        torch.cuda.synchronize()
        assert ws.check_status() == 0 and int(status.item()) == 0
        for (a, sa), (b, sb) in zip(snapshot(ref), snapshot(new)):
            assert sa == sb
            assert np.array_equal(a, b)
        # ... and against the oracle's step on the same inputs
        for (g, gs, m0, ms0, v0, vs0, w0, ws0), m, v, w in zip(before, new.keep[1], new.keep[2], new.keep[3]):
            mo, vo, wo, ms, vs, wsn = orc.adam_step(g, orc.E5M2, gs, m0, v0, orc.F16, ms0, vs0, w0, orc.F16, ws0,
                                                    hyper["lr"], hyper["beta1"], hyper["beta2"], hyper["eps"], step)
            assert (m.scale_value(), v.scale_value(), w.scale_value()) == (ms, vs, wsn)
            assert ulp_diff(to_bits(m.data, si.F16), mo, orc.F16).max() <= 1
            assert ulp_diff(to_bits(v.data, si.F16), vo, orc.F16).max() <= 1
            assert ulp_diff(to_bits(w.data, si.F16), wo, orc.F16).max() <= 1


def test_static_adam_reports_bad_scale_and_then_starts_clean():
    bad = make_state([256], 92)
    bad.keep[1][0].scale.fill_(3.0)  # not a power of two
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_scaled_adam_step_static(bad, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1, status_out=status)
    assert int(status.item()) & sc.DEV_BAD_SCALE
    good = make_state([256], 93)
    sc.scalify_scaled_adam_step_static(good, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1, status_out=status)
    assert int(status.item()) == 0  # the status word of the previous call was cleared


def test_a_scale_word_shared_by_two_tensors_is_rejected_by_both_calls():
    two = make_state([64, 64], 95)
    two.keep[2][1].scale = two.keep[2][0].scale      # both v tensors point at one scale word
    shared = sc.AdamTensors(*two.keep)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 2))
    for call in (lambda: sc.scalify_scaled_adam_step(shared, ws, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1),
                 lambda: sc.scalify_scaled_adam_step_static(shared, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1)):
        with pytest.raises(sc.ScalifyError) as e:
            call()
        assert e.value.code == -8      # SCALIFY_ERR_ALIAS: nothing was enqueued


def test_static_adam_rejects_more_tensors_than_its_scratch_holds():
    one = make_state([16], 94)
    many = sc.AdamTensors(*[lst * 1025 for lst in one.keep])
    with pytest.raises(sc.ScalifyError) as e:
        sc.scalify_scaled_adam_step_static(many, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1)
    assert e.value.code == -5
