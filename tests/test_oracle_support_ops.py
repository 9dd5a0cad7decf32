"""Pins of the oracle's support operations (embedding, causal softmax, cross-entropy) against
library routines (torch index/scatter, softmax, cross_entropy and autograd) in fp64."""
import math

import numpy as np
import torch

import oracle as orc
import scalify_inputs as si


def vals(bits, dt):
    return si.from_bits(bits, dt)


def test_embedding_forward_and_backward_against_torch_indexing():
    V, T, d, B = 50, 8, 16, 3
    n = B * T
    ids = si.uniform_int(61, 1, (n,), V)
    wte = si.scaled_normal(61, 2, (V, d), orc.F16)
    wpe = si.scaled_normal(61, 3, (T, d), orc.F16)
    Y, ys = orc.embedding_fwd(ids, T, wte, orc.F16, 2.0 ** -6, wpe, orc.F16, 2.0 ** -8, orc.F32)
    assert ys == 2.0 ** -6
    want = vals(wte, orc.F16)[ids] * 2.0 ** -6 + np.tile(vals(wpe, orc.F16), (B, 1)) * 2.0 ** -8
    assert np.allclose(Y.view(np.float32) * ys, want, rtol=1e-7, atol=0)
    dY = si.scaled_normal(61, 4, (n, d), orc.BF16)
    dwte, s1, dwpe, s2 = orc.embedding_bwd(ids, T, V, dY, orc.BF16, 2.0 ** -10, orc.F32)
    g = torch.from_numpy(vals(dY, orc.BF16))
    ref_te = torch.zeros(V, d, dtype=torch.float64).index_add_(0, torch.from_numpy(ids), g)
    ref_pe = g.view(B, T, d).sum(0)
    assert s1 == 2.0 ** -10 and s2 == 2.0 ** -10 * orc.kf(B)
    assert np.allclose(dwte.view(np.float32), ref_te.numpy(), rtol=1e-6, atol=1e-6)
    assert np.allclose(dwpe.view(np.float32) * orc.kf(B), ref_pe.numpy(), rtol=1e-6, atol=1e-6)


def test_softmax_forward_and_backward_against_torch():
    b, Tq, Tk = 3, 12, 12
    S = si.scaled_normal(62, 1, (b, Tq, Tk), orc.BF16, 2.0)
    s_scale = 2.0 ** -1
    for causal in (False, True):
        P, ps = orc.softmax_fwd(S, orc.BF16, s_scale, causal, orc.F32)
        z = torch.from_numpy(vals(S, orc.BF16) * s_scale).requires_grad_(True)
        zz = z
        if causal:
            mask = torch.ones(Tq, Tk, dtype=torch.bool).tril()
            zz = z.masked_fill(~mask, float("-inf"))
        ref = torch.softmax(zz, dim=-1)
        assert ps == 1.0
        assert np.allclose(P.view(np.float32), ref.detach().numpy(), rtol=1e-6, atol=1e-9)
        if causal:
            assert np.all(P.view(np.float32)[:, np.triu_indices(Tq, 1)[0], np.triu_indices(Tq, 1)[1]] == 0.0)
        dP = si.scaled_normal(62, 2, (b, Tq, Tk), orc.BF16)
        ref.backward(torch.from_numpy(vals(dP, orc.BF16)))
        P64 = orc.encode(ref.detach().numpy(), orc.F32)
        dS, ss = orc.softmax_bwd(dP, orc.BF16, 2.0 ** -10, P64, orc.F32, 1.0, orc.F32)
        assert ss == 2.0 ** -10
        assert np.allclose(dS.view(np.float32), z.grad.numpy(), rtol=2e-5, atol=1e-7)
    # rectangular causal: a query block at the end of a longer key sequence
    S2 = si.scaled_normal(62, 3, (1, 4, 10), orc.BF16)
    P2, _ = orc.softmax_fwd(S2, orc.BF16, 1.0, True, orc.F32)
    p = P2.view(np.float32)[0]
    assert np.all(p[0, 7:] == 0) and p[0, 6] > 0 and np.all(p[3] > 0)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-6)


def test_cross_entropy_against_torch_with_padded_vocabulary():
    n, V, ld = 16, 37, 48
    logits = si.scaled_normal(63, 1, (n, ld), orc.BF16, 3.0)
    tgt = si.uniform_int(63, 2, (n,), V)
    l_scale = 2.0 ** -1
    loss, g, gs = orc.cross_entropy(logits, orc.BF16, l_scale, V, tgt, orc.F32)
    z = torch.from_numpy(vals(logits, orc.BF16)[:, :V] * l_scale).requires_grad_(True)
    ref = torch.nn.functional.cross_entropy(z, torch.from_numpy(tgt))
    ref.backward()
    assert abs(loss - float(ref.detach())) < 1e-12
    assert gs == 2.0 ** -4  # 1/16
    gv = g.view(np.float32).astype(np.float64) * gs
    assert np.allclose(gv[:, :V], z.grad.numpy(), rtol=1e-6, atol=1e-9)
    assert np.all(gv[:, V:] == 0.0)
    # n not a power of two: the remainder of 1/n stays in the data
    loss2, g2, gs2 = orc.cross_entropy(logits[:12], orc.BF16, l_scale, V, tgt[:12], orc.F32)
    assert gs2 == 2.0 ** -4 and math.isclose(gs2 * (16 / 12), 1 / 12)
    z2 = torch.from_numpy(vals(logits[:12], orc.BF16)[:, :V] * l_scale).requires_grad_(True)
    torch.nn.functional.cross_entropy(z2, torch.from_numpy(tgt[:12])).backward()
    assert np.allclose(g2.view(np.float32).astype(np.float64)[:, :V] * gs2, z2.grad.numpy(), rtol=1e-6, atol=1e-9)
