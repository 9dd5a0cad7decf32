"""Robustness on the GPU without faulting it: (1) a bounded device-side wait that runs out is
reported through the status word and leaves the context usable; (2) no kernel writes outside its
output: outputs are carved out of a larger buffer filled with a sentinel, ragged shapes are run,
and the guard regions before, after and between rows must be untouched."""
import numpy as np
import pytest
import torch

import paper_2407_17353_b200 as sc
import scalify_inputs as si
from helpers import to_dev

pytestmark = pytest.mark.gpu
SENT = 0x5A


def test_expired_wait_sets_timeout_status_and_context_survives():
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, 1024))
    waited = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_debug_expire_wait(ws, 1500, waited)
    assert ws.check_status() == sc.DEV_TIMEOUT
    assert 1500 <= int(waited.item()) < 200000
    assert ws.check_status() == 0  # cleared by the read
    # the context is alive: an ordinary call right after works
    x = sc.ScaledTensor.make(torch.ones(1024, dtype=torch.bfloat16, device="cuda"), 1.0)
    y = sc.ScaledTensor.empty((1024,), torch.float8_e4m3fn)
    sc.scalify_rescale(x, y, stat=sc.STAT_AMAX, ws=ws)
    assert ws.check_status() == 0 and float(y.data.float().abs().max()) == 1.0


def guarded(shape, dtype, row_pad=0, guard=4096):
    """A tensor view of `shape` inside a sentinel-filled byte buffer: guard bytes in front and behind,
    and (for 2-D) row_pad elements of padding after each row."""
    es = torch.empty(0, dtype=dtype).element_size()
    rows = int(np.prod(shape[:-1])) if len(shape) > 1 else 1
    cols = shape[-1]
    ld = cols + row_pad
    raw = torch.full((guard + rows * ld * es + guard,), SENT, dtype=torch.uint8, device="cuda")
    body = raw[guard:guard + rows * ld * es].view(dtype).view(rows, ld)
    view = body[:, :cols]
    if len(shape) == 1:
        view = view.reshape(cols) if row_pad == 0 else view[0]
    return raw, view, (guard, rows, ld, cols, es)


def assert_guards_intact(raw, meta):
    guard, rows, ld, cols, es = meta
    r = raw.cpu().numpy()
    assert np.all(r[:guard] == SENT) and np.all(r[-guard:] == SENT)
    if ld > cols:
        body = r[guard:-guard].reshape(rows, ld * es)
        assert np.all(body[:, cols * es:] == SENT)


@pytest.mark.parametrize("M,N,K", [(1, 16, 16), (130, 272, 144), (257, 528, 400)])
@pytest.mark.parametrize("y_dt", [torch.bfloat16, torch.float32, torch.float8_e4m3fn])
def test_matmul_writes_only_its_output(M, N, K, y_dt):
    A = sc.ScaledTensor.make(to_dev(si.scaled_normal(81, 1, (M, K), si.E4M3), si.E4M3), 1.0)
    Bt = sc.ScaledTensor.make(to_dev(si.scaled_normal(81, 2, (N, K), si.E4M3), si.E4M3), 1.0)
    pad = 16 // torch.empty(0, dtype=y_dt).element_size() * 3
    raw, view, meta = guarded((M, N), y_dt, row_pad=pad)
    Y = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, M, N))
    if y_dt == torch.float8_e4m3fn:
        sc.scalify_scaled_matmul_delayed(A, Bt, torch.ones(1, device="cuda"), Y, ws, transB=True)
    else:
        sc.scalify_scaled_matmul(A, Bt, Y, ws, transB=True, stat=sc.STAT_AMAX)
    assert ws.check_status() == 0
    assert_guards_intact(raw, meta)
    assert torch.isfinite(view.float()).all()


@pytest.mark.parametrize("n", [1, 17, 4099, 256 * 32 + 3])
def test_elementwise_kernels_write_only_their_output(n):
    x = sc.ScaledTensor.make(torch.randn(n, device="cuda").to(torch.bfloat16), 1.0)
    y = sc.ScaledTensor.make(torch.randn(n, device="cuda").to(torch.bfloat16), 0.5)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, n))
    for dt in (torch.float8_e4m3fn, torch.bfloat16, torch.float32):
        raw, view, meta = guarded((n,), dt)
        out = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
        sc.scalify_rescale(x, out, stat=sc.STAT_AMAX, ws=ws)
        assert_guards_intact(raw, meta)
        raw, view, meta = guarded((n,), dt)
        out = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
        sc.scalify_scaled_add(x, y, out)
        assert_guards_intact(raw, meta)
        raw, view, meta = guarded((n,), dt)
        out = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
        sc.scalify_scaled_gelu(x, out)
        assert_guards_intact(raw, meta)


@pytest.mark.parametrize("R,d", [(1, 8), (37, 776), (5, 4096)])
def test_layernorm_writes_only_its_outputs(R, d):
    x = sc.ScaledTensor.make(torch.randn(R, d, device="cuda").to(torch.bfloat16), 1.0)
    g = sc.ScaledTensor.make(torch.randn(R, d, device="cuda").to(torch.bfloat16), 2.0 ** -10)
    gamma = sc.ScaledTensor.make(torch.ones(d, device="cuda", dtype=torch.bfloat16), 1.0)
    beta = sc.ScaledTensor.make(torch.zeros(d, device="cuda", dtype=torch.bfloat16), 1.0)
    raw, view, meta = guarded((R, d), torch.bfloat16, row_pad=8)
    Y = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
    rawm, mean, mm = guarded((R,), torch.float32)
    rawr, rinv, mr = guarded((R,), torch.float32)
    sc.scalify_scaled_layernorm(x, gamma, beta, Y, mean=mean, rinv=rinv)
    for r_, m_ in ((raw, meta), (rawm, mm), (rawr, mr)):
        assert_guards_intact(r_, m_)
    rawd, dview, md = guarded((R, d), torch.bfloat16, row_pad=8)
    dX = sc.ScaledTensor(dview, torch.empty(1, dtype=torch.float32, device="cuda"))
    rawg, gview, mg = guarded((d,), torch.float32)
    rawb, bview, mb = guarded((d,), torch.float32)
    dg = sc.ScaledTensor(gview, torch.empty(1, dtype=torch.float32, device="cuda"))
    db = sc.ScaledTensor(bview, torch.empty(1, dtype=torch.float32, device="cuda"))
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    sc.scalify_scaled_layernorm_bwd(g, x, gamma, mean, rinv, dX, ws, stat_dx=sc.STAT_L2, dgamma=dg, dbeta=db)
    assert ws.check_status() == 0
    for r_, m_ in ((rawd, md), (rawg, mg), (rawb, mb)):
        assert_guards_intact(r_, m_)
    # delayed rescale: FP8 rows (8 bytes per vector of a BF16 input) in a padded buffer
    rawq, qview, mq = guarded((R, d), torch.float8_e5m2, row_pad=16 + (-d) % 16)
    dXq = sc.ScaledTensor(qview, torch.empty(1, dtype=torch.float32, device="cuda"))
    ws.statistic().fill_(2.0 ** -9)
    sc.scalify_scaled_layernorm_bwd_delayed(g, x, gamma, mean, rinv, ws.statistic(), dXq, ws, stat_dx=sc.STAT_AMAX,
                                            dgamma=dg, dbeta=db)
    assert ws.check_status() == 0
    for r_, m_ in ((rawq, mq), (rawg, mg), (rawb, mb)):
        assert_guards_intact(r_, m_)
    assert torch.isfinite(qview.float()).all()


@pytest.mark.parametrize("n", [1, 9, 8195])
def test_adam_writes_only_its_state(n):
    c = si.adam_case(n, seed=82)
    bufs = {}
    T = {}
    for name, dt, code in (("m", torch.float16, si.F16), ("v", torch.float16, si.F16), ("w", torch.float16, si.F16)):
        raw, view, meta = guarded((n,), dt)
        view.copy_(to_dev(c[name], code))
        bufs[name] = (raw, meta)
        T[name] = sc.ScaledTensor.make(view, c[name + "_scale"])
    G = sc.ScaledTensor.make(to_dev(c["g"], si.E5M2), c["g_scale"])
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1))
    sc.scalify_scaled_adam_step(sc.AdamTensors([G], [T["m"]], [T["v"]], [T["w"]]), ws, lr=3e-4, beta1=0.9, beta2=0.999,
                                eps=1e-8, step=10)
    assert ws.check_status() == 0
    for raw, meta in bufs.values():
        assert_guards_intact(raw, meta)


@pytest.mark.parametrize("H,Tq,Tk,causal", [(2, 200, 224, True), (1, 96, 32, False), (3, 129, 160, True)])
def test_attention_forward_and_backward_write_only_their_outputs(H, Tq, Tk, causal):
    """Ragged lengths: the last query / key blocks are partial; rows past the end, the padding after
    each 64-element row and the bytes around the buffers must stay untouched."""
    HD = 64

    def f8(tid, T, bits_dt, dt):
        return sc.ScaledTensor.make(to_dev(si.scaled_normal(83, tid, (H, T, HD), bits_dt), bits_dt).view(dt), 1.0)

    Q, K, V = (f8(1, Tq, si.E4M3, torch.float8_e4m3fn), f8(2, Tk, si.E4M3, torch.float8_e4m3fn),
               f8(3, Tk, si.E4M3, torch.float8_e4m3fn))
    dO = f8(4, Tq, si.E5M2, torch.float8_e5m2)
    outs = {}
    for name, T in (("O", Tq), ("dQ", Tq), ("dK", Tk), ("dV", Tk)):
        raw, view, meta = guarded((H * T, HD), torch.bfloat16, row_pad=8)
        ld = view.stride(0)
        heads = view.as_strided((H, T, HD), (T * ld, ld, 1), view.storage_offset())
        outs[name] = (raw, meta, sc.ScaledTensor(heads, torch.zeros(1, device="cuda")))
    rawp, pview, mp = guarded((H * Tq, Tk), torch.float8_e4m3fn)
    raws, sview, ms = guarded((H * Tq, Tk), torch.float8_e5m2)
    P = sc.ScaledTensor(pview.view(H, Tq, Tk), None)
    dS = sc.ScaledTensor(sview.view(H, Tq, Tk), torch.zeros(1, device="cuda"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.scalify_scaled_attention(Q, K, V, outs["O"][2], sm_scale=0.125, causal=causal, P_dump=P, status=status)
    sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, dS, outs["dQ"][2], outs["dK"][2], outs["dV"][2], sm_scale=0.125,
                                    causal=causal, status=status)
    assert int(status.item()) == 0
    for raw, meta, t in outs.values():
        assert_guards_intact(raw, meta)
        assert torch.isfinite(t.data.float()).all()
    assert_guards_intact(rawp, mp)
    assert_guards_intact(raws, ms)


@pytest.mark.parametrize("R,N", [(1, 16), (37, 1030), (300, 48)])
def test_column_sums_write_only_their_output(R, N):
    ld = (N // 16 + 2) * 16
    X = sc.ScaledTensor.make(to_dev(si.scaled_normal(84, 1, (R, ld), si.E5M2), si.E5M2)[:, :N], 1.0)
    raw, view, meta = guarded((N,), torch.bfloat16)
    Y = sc.ScaledTensor(view, torch.zeros(1, device="cuda"))
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N))
    sc.scalify_scaled_colsum(X, Y, ws)
    assert ws.check_status() == 0
    assert_guards_intact(raw, meta)
    assert torch.isfinite(view.float()).all()


@pytest.mark.parametrize("M,N,K", [(130, 272, 144), (257, 528, 2048), (64, 48, 4096)])
def test_bias_and_split_matmul_write_only_their_output(M, N, K):
    A = sc.ScaledTensor.make(to_dev(si.scaled_normal(85, 1, (M, K), si.E4M3), si.E4M3), 1.0)
    Bt = sc.ScaledTensor.make(to_dev(si.scaled_normal(85, 2, (N, K), si.E4M3), si.E4M3), 1.0)
    bias = sc.ScaledTensor.make(torch.ones(N, device="cuda").to(torch.bfloat16), 0.25)
    for kind in ("bias", "split"):
        raw, view, meta = guarded((M, N), torch.bfloat16, row_pad=24)
        Y = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL_SPLITK if kind == "split" else sc.OP_MATMUL, M, N))
        if kind == "bias":
            sc.scalify_scaled_matmul_bias(A, Bt, bias, Y, ws, transB=True, stat=sc.STAT_AMAX)
        else:
            sc.scalify_scaled_matmul(A, Bt, Y, ws, transB=True, stat=sc.STAT_L2)
        assert ws.check_status() == 0
        assert_guards_intact(raw, meta)
        assert torch.isfinite(view.float()).all()


@pytest.mark.parametrize("rows,K", [(1, 128), (300, 256)])
def test_block_quantiser_writes_only_its_data(rows, K):
    X = sc.ScaledTensor.make(to_dev(si.scaled_normal(86, 1, (rows, K), si.BF16), si.BF16), 1.0)
    Y = sc.MxTensor(rows, K)
    raw, view, meta = guarded((rows, K), torch.float8_e4m3fn)
    Y.data = view
    Y._d.data = view.data_ptr()
    sc.scalify_mx_quantize(X, Y)
    torch.cuda.synchronize()
    assert_guards_intact(raw, meta)
    assert torch.isfinite(view.float()).all()


@pytest.mark.parametrize("n,V,ld", [(700, 1000, 1008), (3, 37, 48)])
def test_cross_entropy_writes_only_its_gradient(n, V, ld):
    """Several rows per block: the kernel copies the next row in while it writes the current gradient row."""
    logits = sc.ScaledTensor.make(to_dev(si.scaled_normal(87, 1, (n, ld), si.BF16, 3.0), si.BF16), 0.5)
    tgt = torch.from_numpy(si.uniform_int(87, 2, (n,), V)).cuda()
    raw, view, meta = guarded((n, ld), torch.float8_e5m2)
    G = sc.ScaledTensor(view, torch.empty(1, dtype=torch.float32, device="cuda"))
    rawl, lview, ml = guarded((1,), torch.float32)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_CROSS_ENTROPY, n))
    sc.scalify_scaled_cross_entropy(logits, V, tgt, lview, G, ws)
    assert ws.check_status() == 0
    assert_guards_intact(raw, meta)
    assert_guards_intact(rawl, ml)
    assert torch.isfinite(view.float()).all() and bool(torch.isfinite(lview).all())
    assert bool((view.float()[:, V:] == 0).all())
