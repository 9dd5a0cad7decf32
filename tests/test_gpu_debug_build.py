"""The bounds-checking build (libscalify_debug.so, -DSCALIFY_DEBUG): the memory-bound kernels run on ragged
shapes with every checked access inside the arrays the entry points validated (no violation, same bits as
the ordinary build), and the checker itself is exercised by capping the registered spans, so that accesses
that are inside the caller's buffers but past the cap are refused, reported and skipped.  Nothing here reads
or writes outside an allocation.  Runs in a child process, because a process loads one of the two builds."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import json, sys, os
sys.path.insert(0, os.path.join(ROOT, "tests")); sys.path.insert(0, ROOT)
import numpy as np, torch
import paper_2407_17353_b200 as sc

torch.manual_seed(3)
debug = os.environ.get("SCALIFY_DEBUG_BUILD") == "1"
out = {}
def bits(t):
    return t.detach().contiguous().view(torch.uint8).cpu().numpy().tobytes().hex()

def run_all():
    res = {}
    def mark(name):   # debug build: the accesses refused while this operation ran
        if debug:
            res["violations_" + name] = sc.scalify_debug_bounds_report()["violations"]
    # ragged sizes: vector tails, rows that are not a multiple of the team width, several tensors
    n = 8 * 1024 * 5 + 13
    X = sc.ScaledTensor.make((torch.randn(n, device="cuda") * 7).bfloat16(), 0.25)
    ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, n, 0))
    for dt in (torch.float8_e4m3fn, torch.bfloat16):
        Y = sc.ScaledTensor.empty((n,), dt)
        sc.scalify_rescale(X, Y, stat=sc.STAT_AMAX, ws=ws)
        res["rescale_%s" % dt] = bits(Y.data) + "%r" % Y.scale_value()
    mark("rescale")
    A = sc.ScaledTensor.make(torch.randn(37, 784, device="cuda").bfloat16(), 2.0)
    B = sc.ScaledTensor.make(torch.randn(784, device="cuda").bfloat16(), 0.5)
    S = sc.ScaledTensor.empty((37, 784), torch.bfloat16)
    sc.scalify_scaled_add(A, B, S)
    res["add_bias"] = bits(S.data)
    mark("add")
    G = sc.ScaledTensor.empty((37, 784), torch.float8_e4m3fn)
    sc.scalify_scaled_gelu(A, G)
    res["gelu"] = bits(G.data)
    mark("gelu")
    R, d = 301, 1008
    Xl = sc.ScaledTensor.make(torch.randn(R, d, device="cuda").bfloat16(), 1.0)
    Gl = sc.ScaledTensor.make(torch.randn(R, d, device="cuda").bfloat16(), 2.0 ** -8)
    gam = sc.ScaledTensor.make(torch.randn(d, device="cuda").bfloat16(), 1.0)
    bet = sc.ScaledTensor.make(torch.randn(d, device="cuda").bfloat16(), 1.0)
    Yl = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    mean, rinv = torch.empty(R, device="cuda"), torch.empty(R, device="cuda")
    sc.scalify_scaled_layernorm(Xl, gam, bet, Yl, mean=mean, rinv=rinv)
    res["ln_fwd"] = bits(Yl.data)
    mark("ln_fwd")
    wsl = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d))
    dX = sc.ScaledTensor.empty((R, d), torch.bfloat16)
    dXq = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
    dg, db = sc.ScaledTensor.empty((d,), torch.float32), sc.ScaledTensor.empty((d,), torch.float32)
    sc.scalify_scaled_layernorm_bwd(Gl, Xl, gam, mean, rinv, dX, wsl, stat_dx=sc.STAT_L2, dXq=dXq, dgamma=dg, dbeta=db)
    res["ln_bwd"] = bits(dX.data) + bits(dXq.data) + bits(dg.data) + bits(db.data)
    mark("ln_bwd")
    q1 = sc.ScaledTensor.empty((R, d), torch.float8_e5m2)
    sc.scalify_scaled_layernorm_bwd(Gl, Xl, gam, mean, rinv, None, wsl, stat_dx=sc.STAT_L2, dXq=q1, dgamma=dg, dbeta=db)
    res["ln_bwd_one_pass"] = bits(q1.data)
    mark("ln_bwd_one_pass")
    sizes = [7, 1000, 8 * 1024 + 5]
    g = [sc.ScaledTensor.make(torch.randn(k, device="cuda").to(torch.float8_e5m2), 2.0 ** -12) for k in sizes]
    m = [sc.ScaledTensor.make(torch.randn(k, device="cuda").half(), 2.0 ** -16) for k in sizes]
    v = [sc.ScaledTensor.make((torch.randn(k, device="cuda") ** 2).half(), 2.0 ** -24) for k in sizes]
    w = [sc.ScaledTensor.make(torch.randn(k, device="cuda").half(), 2.0 ** -6) for k in sizes]
    adam = sc.AdamTensors(g, m, v, w)
    wsa = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(sizes)))
    sc.scalify_scaled_adam_step(adam, wsa, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=3)
    res["adam"] = "".join(bits(t.data) for t in m + v + w)
    mark("adam")
    rows, K = 304, 256
    Xm = sc.ScaledTensor.make(torch.randn(rows, K, device="cuda").bfloat16(), 1.0)
    Ym = sc.MxTensor(rows, K)
    sc.scalify_mx_quantize(Xm, Ym)
    Xt = sc.ScaledTensor.make(torch.randn(K, rows, device="cuda").bfloat16(), 1.0)
    Yt = sc.MxTensor(rows, K, transposed=True)
    sc.scalify_mx_quantize(Xt, Yt)
    res["mx"] = bits(Ym.data) + bits(Yt.data) + bits(Yt.sf)
    mark("mx")
    torch.cuda.synchronize()
    return res

out["results"] = run_all()
if debug:
    out["clean"] = sc.scalify_debug_bounds_report()
    # self-test of the checker: forget the spans, cap new ones at 4 KiB, run one op on a 64 KiB input
    sc.scalify_debug_bounds_report(reset_ranges=True, range_limit=4096)
    n = 32768
    X = sc.ScaledTensor.make(torch.ones(n, device="cuda").bfloat16(), 1.0)
    Y = sc.ScaledTensor.empty((n,), torch.bfloat16)
    Y.data.fill_(-3.0)
    Z = sc.ScaledTensor.make(torch.ones(n, device="cuda").bfloat16(), 1.0)
    sc.scalify_scaled_add(X, Z, Y)
    rep = sc.scalify_debug_bounds_report(reset_ranges=True, range_limit=-1)
    y = Y.data.float().cpu().numpy()
    out["capped"] = dict(rep, written=int((y == 2.0).sum()), untouched=int((y == -3.0).sum()),
                         x_ptr=X.data.data_ptr(), y_ptr=Y.data.data_ptr(), z_ptr=Z.data.data_ptr())
    out["after"] = sc.scalify_debug_bounds_report()
else:
    try:
        sc.scalify_debug_bounds_report()
        out["release_report"] = "ok"
    except sc.ScalifyError as e:
        out["release_report"] = e.code
print("RESULT" + json.dumps(out))
'''


def run_child(debug):
    env = dict(os.environ)
    env["SCALIFY_DEBUG_BUILD"] = "1" if debug else "0"
    r = subprocess.run([sys.executable, "-c", "ROOT = %r\n" % ROOT + CHILD], capture_output=True, text=True, env=env,
                       timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("RESULT")][-1]
    return json.loads(line[len("RESULT"):])


def test_debug_build_sees_no_violation_and_gives_the_same_bits_and_its_checker_works():
    rel = run_child(False)
    dbg = run_child(True)
    assert rel["release_report"] == -6          # the ordinary build has no checker
    refused = {k: v for k, v in dbg["results"].items() if k.startswith("violations_")}
    assert all(v == 0 for v in refused.values()), refused
    assert dbg["clean"]["violations"] == 0, dbg["clean"]
    for k in rel["results"]:
        assert dbg["results"][k] == rel["results"][k], k
    # with every span capped at 4 KiB, the accesses past the cap were refused and skipped: only the first
    # 2048 BF16 outputs were written, the rest kept their fill value
    cap = dbg["capped"]
    assert cap["violations"] > 0
    assert cap["written"] == 2048 and cap["untouched"] == 32768 - 2048, cap
    lo = min(cap["x_ptr"], cap["y_ptr"], cap["z_ptr"])
    assert cap["first_address"] >= lo + 4096 and cap["first_bytes"] in (16, 32)
    assert dbg["after"]["violations"] == 0
