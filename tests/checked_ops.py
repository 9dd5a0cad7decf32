"""Library calls with an optional stage-isolated oracle check.

`Ops(check=True)` runs every C-ABI call and then the oracle on the SAME inputs (downloaded bit
patterns of the library's own previous outputs), holding each call to its own tolerance.  With
`check=False` the same code only launches kernels (used to time a full-size step).

`Ops(check="sampled")` is the form for shapes the fp64 oracle cannot follow output by output
(GPT-2-small: 7e12 flop per step).  Scale words, statistic words and status words are still checked
on every call and exactly.  Matmul outputs are compared on a few thousand sampled positions plus
tile-edge positions (the oracle evaluates single outputs); row-wise and elementwise calls on large
arrays are compared in full on sampled rows (first and last rows and rows around multiples of 128
included); arrays of a few million elements (LayerNorm, residual adds, gradients of the
parameters, the optimizer) are still compared in full; the fused attention on sampled heads.
`ops.active = False` switches the checks off for a stretch of calls (a layer not under test)."""
import numpy as np
import torch

import paper_2407_17353_b200 as sc

E4, E5, F16, BF, F32 = sc.E4M3, sc.E5M2, sc.F16, sc.BF16, sc.F32
_CODE = {torch.float8_e4m3fn: E4, torch.float8_e5m2: E5, torch.float16: F16, torch.bfloat16: BF, torch.float32: F32}


def code(t: torch.Tensor) -> int:
    return _CODE[t.dtype]


class Ops:
    FULL_LIMIT = 1 << 23      # sampled mode: arrays up to this many elements are still compared in full

    def __init__(self, check, ws_bytes: int = 1 << 26, device="cuda"):
        self.mode = "sampled" if check == "sampled" else ("full" if check else "off")
        self._check = bool(check)
        self.active = True
        self.checked_calls = 0
        self.dev = device
        self.ws = sc.Workspace(ws_bytes, device)
        self.calls = 0
        if check:
            import oracle as orc
            from helpers import to_bits, ulp_diff, within
            self.orc, self.to_bits, self.ulp_diff, self.within = orc, to_bits, ulp_diff, within

    @property
    def check(self):
        on = self._check and self.active
        self.checked_calls += int(on)      # (a call may ask twice; only used as "at least so many")
        return on

    # ---------------------------------------------------------------- helpers
    def _rows(self, R, numel, k=48):
        """Row indices to compare (None: all rows)."""
        if self.mode != "sampled" or numel <= self.FULL_LIMIT or R <= 4 * k:
            return None
        rng = np.random.default_rng(7000 + self.calls)
        edge = [0, 1, R - 2, R - 1, 127, 128, R - 129, R - 128, R // 2]
        return np.unique(np.concatenate([rng.integers(0, R, k), [e for e in edge if 0 <= e < R]]))

    def _positions(self, M, N, k=2500):
        """Sampled output positions of an [M, N] product: random ones plus the corners and the first / last
        positions around multiples of the 128 x 256 tile."""
        rng = np.random.default_rng(9000 + self.calls)
        er = [r for r in (0, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1) if 0 <= r < M]
        ec = [c for c in (0, 255, 256, 511, 512, N - 513, N - 512, N - 257, N - 256, N - 1) if 0 <= c < N]
        gr, gc = np.meshgrid(er, ec, indexing="ij")
        rows = np.concatenate([rng.integers(0, M, k), gr.reshape(-1)])
        cols = np.concatenate([rng.integers(0, N, k), gc.reshape(-1)])
        return rows, cols

    def _heads_to_check(self, H):
        if self.mode != "sampled" or H <= 4:
            return range(H)
        rng = np.random.default_rng(5000 + self.calls)
        return sorted(set([0, H - 1, int(rng.integers(1, H - 1))]))

    def take(self, T, rows):
        """Bit patterns of the listed rows of T seen as [rows, last dimension] (all rows if None)."""
        t = T.data.reshape(-1, T.data.shape[-1])
        if rows is not None:
            t = t[torch.as_tensor(rows, device=t.device)]
        return self.to_bits(t, code(T.data))

    def empty(self, shape, dt):
        return sc.ScaledTensor.empty(tuple(shape), sc.TORCH_DTYPE[dt], self.dev)

    def bits(self, T):
        return self.to_bits(T.data, code(T.data))

    def _status_ok(self):
        if self.check:
            st = self.ws.check_status()
            assert st == 0, st

    # ---------------------------------------------------------------- casts and rescales
    def cast(self, X, dt):
        Y = self.empty(X.data.shape, dt)
        sc.scalify_rescale(X, Y)
        self.calls += 1
        if self.check:
            o = self.orc
            assert Y.scale_value() == X.scale_value()
            rows = self._rows(X.data.numel() // X.data.shape[-1], X.data.numel())
            assert np.array_equal(self.take(Y, rows), o.encode(o.decode(self.take(X, rows), code(X.data)), dt))
        return Y

    def rescale(self, X, stat, dt, key=None):
        """Dynamic rescale (statistic -> power of two -> rebalance).  key: a workspace of its own for this call
        site, so that the power of two predicted from the site's previous statistic holds step after step."""
        Y = self.empty(X.data.shape, dt)
        ws = self.ws
        if key is not None:
            if not hasattr(self, "ws_rescale"):
                self.ws_rescale = {}
            if key not in self.ws_rescale:
                self.ws_rescale[key] = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, X.data.numel(), 0), self.dev)
            ws = self.ws_rescale[key]
        sc.scalify_rescale(X, Y, stat=stat, ws=ws)
        self.calls += 2
        if self.check:
            o = self.orc
            assert ws.check_status() == 0
            so = o.statistic(self.bits(X).reshape(-1), code(X.data), stat)      # always over the whole array
            if stat == sc.STAT_L2 and abs(np.log2(so) - round(np.log2(so))) < 1e-5:
                return Y  # binade edge: either neighbouring scale is correct
            rows = self._rows(X.data.numel() // X.data.shape[-1], X.data.numel())
            yo, ys, _ = o.rescale(self.take(X, rows).reshape(-1), code(X.data), X.scale_value(), stat, dt,
                                  stat_override=so)
            assert Y.scale_value() == ys
            assert np.array_equal(self.take(Y, rows).reshape(-1), yo)
        return Y

    def scalar_mul(self, X, c):
        before = X.scale_value() if self.check else None
        sc.scalify_scalar_mul_pow2(X, c)
        self.calls += 1
        if self.check:
            assert X.scale_value() == before * c
        return X

    # ---------------------------------------------------------------- matmul
    def mm(self, A, B, *, transA=False, transB=False, out_dt=BF, Y=None, stat=sc.STAT_NONE, q_dt=None, key=None):
        """key: a name for this call site.  A matmul with a fused rescale to FP8 predicts its rescale factor from the
        statistic its workspace saw last, so such a call keeps a workspace of its own from step to step."""
        a, b = A.data, B.data
        M = a.shape[-1] if transA else a.shape[-2]
        N = b.shape[-2] if transB else b.shape[-1]
        shape = (M, N) if a.dim() == 2 else (a.shape[0], M, N)
        if Y is None:
            Y = self.empty(shape, out_dt)
        Yq = self.empty(shape, q_dt) if q_dt is not None else None
        ws = self.ws
        if key is not None:
            if not hasattr(self, "ws_keyed"):
                self.ws_keyed = {}
            if key not in self.ws_keyed:
                self.ws_keyed[key] = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL_SPLITK, M, N), self.dev)
            ws = self.ws_keyed[key]
        sc.scalify_scaled_matmul(A, B, Y, ws, transA=transA, transB=transB, stat=stat, Yq=Yq)
        self.calls += 1 + (1 if Yq is not None else 0)
        if self.check:
            o = self.orc
            assert ws.check_status() == 0
            a_dt, b_dt, y_dt = code(a), code(b), code(Y.data)
            K = a.shape[-2] if transA else a.shape[-1]
            if self.mode == "sampled" and a.dim() == 2 and 2.0 * M * N * K > 4e9:
                rows, cols = self._positions(M, N)
                acc, sab = o.scaled_matmul_samples(self.bits(A), a_dt, self.bits(B), b_dt, rows, cols, transA=transA,
                                                   transB=transB)
                assert Y.scale_value() == A.scale_value() * B.scale_value() * o.kf(K)
                got = self.to_bits(Y.data[torch.as_tensor(rows, device=self.dev), torch.as_tensor(cols, device=self.dev)],
                                   y_dt)
                ok = self.within(got, o.encode(acc, y_dt), y_dt, acc, sab, 1e-5)
                assert ok.all(), int((~ok).sum())
            else:
                Ab, Bb, Yb = self.bits(A), self.bits(B), self.bits(Y)
                if a.dim() == 2:
                    Ab, Bb, Yb = Ab[None], Bb[None], Yb[None]
                elif b.dim() == 2:
                    Bb = np.broadcast_to(Bb, (Ab.shape[0],) + Bb.shape)
                for i in range(Ab.shape[0]):
                    Yo, ys, acc, sab = o.scaled_matmul(Ab[i], a_dt, A.scale_value(), Bb[i], b_dt, B.scale_value(), y_dt,
                                                       transA=transA, transB=transB, want_acc=True)
                    assert Y.scale_value() == ys
                    ok = self.within(Yb[i], Yo, y_dt, acc, sab, 1e-5)
                    assert ok.all(), int((~ok).sum())
            if Yq is not None:
                so = o.statistic(self.bits(Y).reshape(-1), y_dt, stat)
                got = float(ws.statistic().item())
                assert got == so if stat == sc.STAT_AMAX else abs(got - so) <= 2e-6 * so
                qo, qs, _ = o.rescale(self.bits(Y).reshape(-1), y_dt, Y.scale_value(), stat, q_dt)
                if not (stat == sc.STAT_L2 and abs(np.log2(so) - round(np.log2(so))) < 1e-5):
                    assert Yq.scale_value() == qs
                    assert np.array_equal(self.bits(Yq).reshape(-1), qo)
        return (Y, Yq) if q_dt is not None else Y

    def linear(self, X, W, bias, out_dt=BF):
        """Y = X W + bias in one launch: [n, K] x [K, N] + [N], one rounding to out_dt (FP8 allowed)."""
        n, N = X.data.shape[0], W.data.shape[1]
        Y = self.empty((n, N), out_dt)
        sc.scalify_scaled_matmul_bias(X, W, bias, Y, self.ws)
        self.calls += 1
        if self.check:
            o = self.orc
            self._status_ok()
            K = X.data.shape[1]
            ab_s = X.scale_value() * W.scale_value() * o.kf(K)
            bs = bias.scale_value()
            ys = max(ab_s, bs)
            assert Y.scale_value() == ys
            bv = o.decode(self.bits(bias), code(bias.data))
            if self.mode == "sampled" and 2.0 * n * N * K > 4e9:
                rows, cols = self._positions(n, N)
                acc, sab = o.scaled_matmul_samples(self.bits(X), code(X.data), self.bits(W), code(W.data), rows, cols)
                exact = acc * (ab_s / ys) + bv[cols] * (bs / ys)
                mag = sab * (ab_s / ys) + np.abs(bv)[cols] * (bs / ys)
                got = self.to_bits(Y.data[torch.as_tensor(rows, device=self.dev), torch.as_tensor(cols, device=self.dev)],
                                   out_dt)
            else:
                _, ab_o, acc, sab = o.scaled_matmul(self.bits(X), code(X.data), X.scale_value(), self.bits(W),
                                                    code(W.data), W.scale_value(), F32, want_acc=True)
                assert ab_o == ab_s
                exact = acc * (ab_s / ys) + bv[None, :] * (bs / ys)
                mag = sab * (ab_s / ys) + np.abs(bv)[None, :] * (bs / ys)
                got = self.bits(Y)
            ok = self.within(got, o.encode(exact, out_dt), out_dt, exact, mag, 1e-5)
            assert ok.all(), int((~ok).sum())
        return Y

    # ---------------------------------------------------------------- add
    def add(self, A, B, subtract=False, out_dt=None):
        Y = self.empty(A.data.shape, out_dt if out_dt is not None else code(A.data))
        sc.scalify_scaled_add(A, B, Y, subtract=subtract)
        self.calls += 1
        if self.check:
            o = self.orc
            dt, ydt = code(A.data), code(Y.data)
            rows = self._rows(A.data.numel() // A.data.shape[-1], A.data.numel())
            a2 = self.take(A, rows)
            b = self.bits(B) if B.data.dim() == 1 else self.take(B, rows)
            yo, ys = o.scaled_add(a2, dt, A.scale_value(), b, dt, B.scale_value(), ydt, subtract=subtract)
            assert Y.scale_value() == ys
            fa, fb = A.scale_value() / ys, B.scale_value() / ys
            av = o.decode(a2, dt) * fa
            bv = o.decode(b, dt) * fb
            bv = bv[None, :] if b.ndim == 1 else bv
            exact = av - bv if subtract else av + bv
            ok = self.within(self.take(Y, rows), yo, ydt, exact, np.abs(av) + np.abs(bv), 2.0 ** -23)
            assert ok.all(), int((~ok).sum())
        return Y

    # ---------------------------------------------------------------- LayerNorm
    def ln(self, X, gamma, beta, eps=1e-5, out_dt=BF):
        R, d = X.data.shape
        Y = self.empty((R, d), out_dt)
        mean = torch.empty(R, dtype=torch.float32, device=self.dev)
        rinv = torch.empty(R, dtype=torch.float32, device=self.dev)
        sc.scalify_scaled_layernorm(X, gamma, beta, Y, eps=eps, mean=mean, rinv=rinv)
        self.calls += 1
        if self.check:
            o = self.orc
            xdt, gdt = code(X.data), code(gamma.data)
            gs, bs = gamma.scale_value(), beta.scale_value()
            yo, ys, _, _ = o.layernorm_fwd(self.bits(X), xdt, self.bits(gamma), gdt, gs, self.bits(beta), gdt, bs, eps,
                                           False, out_dt)
            n32, _, _, _ = o.layernorm_fwd(self.bits(X), xdt, None, 0, 1.0, None, 0, 1.0, eps, False, F32)
            nv = o.decode(n32, F32)
            g = o.decode(self.bits(gamma), gdt) * (gs / ys)
            b = o.decode(self.bits(beta), gdt) * (bs / ys)
            assert Y.scale_value() == ys
            ok = self.within(self.bits(Y), yo, out_dt, nv * g + b, np.abs(nv * g) + np.abs(b) + 1e-3, 2e-6)
            assert ok.all(), int((~ok).sum())
        return Y, mean, rinv

    def ln_bwd(self, G, X, gamma, mean, rinv, stat=sc.STAT_L2, q_dt=BF, eps=1e-5):
        R, d = X.data.shape
        dX = self.empty((R, d), BF)
        dXq = self.empty((R, d), q_dt)
        dg, db = self.empty((d,), F32), self.empty((d,), F32)
        sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, self.ws, eps=eps, stat_dx=stat, dXq=dXq,
                                        dgamma=dg, dbeta=db)
        self.calls += 3
        if self.check:
            o = self.orc
            self._status_ok()
            xdt, gdt = code(X.data), code(gamma.data)
            gb, xb, gamb = self.bits(G), self.bits(X), self.bits(gamma)
            r = o.layernorm_bwd(gb, xdt, G.scale_value(), xb, xdt, X.scale_value(), gamb, gdt, gamma.scale_value(), eps,
                                False, BF, F32, want_f64=True)
            assert dX.scale_value() == r["dX_scale"] and dg.scale_value() == r["dgamma_scale"]
            _, _, _, ro = o.layernorm_fwd(xb, xdt, None, 0, 1.0, None, 0, 1.0, eps, False, BF)
            gv = o.decode(gamb, gdt)
            ghat = o.decode(gb, xdt) * gv[None, :]
            row_mag = np.abs(ghat).max(axis=1) * ro
            got = self.bits(dX)
            ok = self.within(got, r["dX"], BF, r["dx_f64"], row_mag[:, None], 2.0 ** -18)
            assert ok.all(), int((~ok).sum())
            n32, _, _, _ = o.layernorm_fwd(xb, xdt, None, 0, 1.0, None, 0, 1.0, eps, False, F32)
            nv, Gd, f = o.decode(n32, F32), o.decode(gb, xdt), o.kf(R)
            assert np.all(np.abs(o.decode(self.bits(dg), F32) - (Gd * nv).sum(0) / f) <=
                          2e-5 * np.abs(Gd * nv).sum(0) / f + 1e-30)
            assert np.all(np.abs(o.decode(self.bits(db), F32) - Gd.sum(0) / f) <= 2e-5 * np.abs(Gd).sum(0) / f + 1e-30)
            so = o.statistic(got.reshape(-1), BF, stat)
            gstat = float(self.ws.statistic().item())
            assert gstat == so if stat == sc.STAT_AMAX else abs(gstat - so) <= 2e-6 * so
            if not (stat == sc.STAT_L2 and abs(np.log2(so) - round(np.log2(so))) < 1e-5):
                qo, qs, _ = o.rescale(got.reshape(-1), BF, r["dX_scale"], stat, q_dt)
                assert dXq.scale_value() == qs and np.array_equal(self.bits(dXq).reshape(-1), qo)
        return dXq, dg, db

    # ---------------------------------------------------------------- GELU
    def gelu(self, X, out_dt=BF):
        Y = self.empty(X.data.shape, out_dt)
        sc.scalify_scaled_gelu(X, Y)
        self.calls += 1
        if self.check:
            o = self.orc
            rows = self._rows(X.data.shape[0], X.data.numel())
            yo, ys = o.gelu_fwd(self.take(X, rows), code(X.data), X.scale_value(), out_dt)
            assert Y.scale_value() == ys and self.ulp_diff(self.take(Y, rows), yo, out_dt).max() <= 1
        return Y

    def gelu_bwd(self, G, X):
        dX = self.empty(X.data.shape, BF)
        sc.scalify_scaled_gelu_bwd(G, X, dX)
        self.calls += 1
        if self.check:
            o = self.orc
            dt = code(X.data)
            rows = self._rows(X.data.shape[0], X.data.numel())
            gb, got = self.take(G, rows), self.take(dX, rows)
            do, ds = o.gelu_bwd(gb, dt, G.scale_value(), self.take(X, rows), dt, X.scale_value(), BF)
            assert dX.scale_value() == ds
            dd = self.ulp_diff(got, do, BF)
            bad = dd > 1  # f' crosses zero near x = -0.75: absolute bound there
            if bad.any():
                err = np.abs(o.decode(got, BF) - o.decode(do, BF))
                assert np.all(err[bad] <= 2.0 ** -9 * 2e-2 * np.abs(o.decode(gb, dt))[bad] + 2.0 ** -16)
        return dX

    # ---------------------------------------------------------------- attention pieces
    def softmax(self, S, causal, p_dt):
        P = self.empty(S.data.shape, p_dt)
        sc.scalify_scaled_softmax(S, P, causal=causal)
        self.calls += 1
        if self.check:
            o = self.orc
            po, ps = o.softmax_fwd(self.bits(S), code(S.data), S.scale_value(), causal, p_dt)
            assert P.scale_value() == ps and self.ulp_diff(self.bits(P), po, p_dt).max() <= 1
        return P

    def colsum(self, X, o_dt=BF):
        """Column sums of a [R, N] matrix by the reduce-sum rule (the bias gradient)."""
        R, N = X.data.shape
        Y = self.empty((N,), o_dt)
        if not hasattr(self, "ws_col") or self.ws_col.nbytes < sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N):
            self.ws_col = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N), self.dev)
        sc.scalify_scaled_colsum(X, Y, self.ws_col)
        self.calls += 1
        if self.check:
            o = self.orc
            xv = o.decode(self.bits(X), code(X.data))
            kf = o.kf(R)
            exact, mag = xv.sum(axis=0) / kf, np.abs(xv).sum(axis=0) / kf
            assert Y.scale_value() == X.scale_value() * kf
            assert self.within(self.bits(Y), o.encode(exact, o_dt), o_dt, exact, mag, 1e-5).all()
        return Y

    def cast_colsum(self, X, dt, o_dt=BF):
        """The FP8 copy of a gradient and the column sums of that copy (the bias gradient) in one pass."""
        R, N = X.data.shape
        C = self.empty((R, N), dt)
        Y = self.empty((N,), o_dt)
        if not hasattr(self, "ws_col") or self.ws_col.nbytes < sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N):
            self.ws_col = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_COLSUM, R, N), self.dev)
        sc.scalify_scaled_cast_colsum(X, C, Y, self.ws_col)
        self.calls += 1
        if self.check:
            o = self.orc
            assert self.ws_col.check_status() == 0
            assert C.scale_value() == X.scale_value()
            rows = self._rows(R, X.data.numel())
            assert np.array_equal(self.take(C, rows), o.encode(o.decode(self.take(X, rows), code(X.data)), dt))
            cv = o.decode(self.bits(C), dt)                       # the sums are those of the library's own cast
            kf = o.kf(R)
            exact, mag = cv.sum(axis=0) / kf, np.abs(cv).sum(axis=0) / kf
            assert Y.scale_value() == X.scale_value() * kf
            assert self.within(self.bits(Y), o.encode(exact, o_dt), o_dt, exact, mag, 1e-5).all()
        return C, Y

    def attention(self, Q, K, V, O, sm_scale, causal=True):
        """Fused forward over [heads, T, 64] views; returns the E4M3 probabilities (kept for the backward).
        Checked stage by stage through the kernel's own copies of the scores and probabilities."""
        lead, Tq, Tk = tuple(Q.data.shape[:-2]), Q.data.shape[-2], K.data.shape[-2]   # [heads] or [batch, heads]
        H = int(np.prod(lead))
        # (the blocks wholly above the diagonal are never written nor read: zeroed only for the checks below)
        alloc = torch.zeros if self.check else torch.empty
        P = sc.ScaledTensor(alloc(lead + (Tq, Tk), dtype=torch.uint8, device=Q.data.device).view(torch.float8_e4m3fn),
                            torch.ones(1, dtype=torch.float32, device=Q.data.device))
        Sd = None
        if self.check:
            Sd = sc.ScaledTensor(torch.zeros(lead + (Tq, Tk), dtype=torch.bfloat16, device=Q.data.device), None)
        sc.scalify_scaled_attention(Q, K, V, O, sm_scale=sm_scale, causal=causal, S_dump=Sd, P_dump=P)
        self.calls += 1
        if self.check:
            o = self.orc
            q_dt, k_dt, v_dt, o_dt = code(Q.data), code(K.data), code(V.data), code(O.data)
            flat = lambda a: a.reshape((H,) + a.shape[-2:])
            qb, kb, vb = flat(self.bits(Q)), flat(self.bits(K)), flat(self.bits(V))
            Sg, Pg, Og = flat(self.bits(Sd)), flat(self.bits(P)), flat(self.bits(sc.ScaledTensor(O.data.contiguous(), None)))
            ii, jj = np.meshgrid(np.arange(Tq), np.arange(Tk), indexing="ij")
            vis = (jj <= ii + (Tk - Tq)) if causal else np.ones((Tq, Tk), dtype=bool)
            for h in self._heads_to_check(H):
                So, ss, acc, sab = o.scaled_matmul(qb[h], q_dt, Q.scale_value(), kb[h], k_dt, K.scale_value(), BF,
                                                   transB=True, want_acc=True)
                assert self.within(Sg[h][vis], So[vis], BF, acc[vis], sab[vis], 1e-5).all()
                Sin = np.where(vis, Sg[h], 0).astype(np.uint16)
                Po, ps = o.softmax_fwd(Sin[None], BF, ss * sm_scale, causal, E4)
                assert self.ulp_diff(Pg[h][vis], Po[0][vis], E4).max() <= 1 and np.all(Pg[h][~vis] == 0)
                Oo, os_, oacc, osab = o.scaled_matmul(Pg[h], E4, 1.0, vb[h], v_dt, V.scale_value(), o_dt, want_acc=True)
                assert O.scale_value() == os_
                assert self.within(Og[h], Oo, o_dt, oacc, osab, 1e-5).all()
        return P

    def attention_bwd(self, Q, K, V, P, dO, dQ, dK, dV, sm_scale, causal=True):
        """Fused backward over [heads, T, 64] views: dQ, dK, dV are written in place (their scale words too).
        Checked stage by stage through the kernel's own dP copy and its dS output."""
        lead, Tq, Tk = tuple(Q.data.shape[:-2]), Q.data.shape[-2], K.data.shape[-2]
        H = int(np.prod(lead))
        dev = Q.data.device
        alloc = torch.zeros if self.check else torch.empty
        dS = sc.ScaledTensor(alloc(lead + (Tq, Tk), dtype=torch.uint8, device=dev).view(torch.float8_e5m2),
                             torch.empty(1, dtype=torch.float32, device=dev))
        dPd = None
        if self.check:
            dPd = sc.ScaledTensor(torch.zeros(lead + (Tq, Tk), dtype=torch.bfloat16, device=dev), None)
        sc.scalify_scaled_attention_bwd(Q, K, V, P, dO, dS, dQ, dK, dV, sm_scale=sm_scale, causal=causal, dP_dump=dPd)
        self.calls += 1
        if self.check:
            o = self.orc
            q_dt, k_dt, v_dt, g_in, g_dt = code(Q.data), code(K.data), code(V.data), code(dO.data), code(dQ.data)
            flat = lambda a: a.reshape((H,) + a.shape[-2:])
            qb, kb, vb, gb, pb = (flat(self.bits(t)) for t in (Q, K, V, dO, P))
            dPg, dSg = flat(self.bits(dPd)), flat(self.bits(dS))
            dQg, dKg, dVg = (flat(self.bits(sc.ScaledTensor(t.data.contiguous(), None))) for t in (dQ, dK, dV))
            ii, jj = np.meshgrid(np.arange(Tq), np.arange(Tk), indexing="ij")
            shift = Tk - Tq
            vis = ((jj // 128) * 128 <= (ii // 128) * 128 + 127 + shift) if causal else np.ones((Tq, Tk), dtype=bool)
            for h in self._heads_to_check(H):
                dPo, dps, acc, sab = o.scaled_matmul(gb[h], g_in, dO.scale_value(), vb[h], v_dt, V.scale_value(), BF,
                                                     transB=True, want_acc=True)
                assert self.within(dPg[h][vis], dPo[vis], BF, acc[vis], sab[vis], 1e-5).all()
                dPin = np.where(vis, dPg[h], 0).astype(np.uint16)
                dSo, dss = o.softmax_bwd(dPin, BF, dps, pb[h], E4, P.scale_value(), E5)
                assert dS.scale_value() == dss * sm_scale
                pv, gv = o.decode(pb[h], E4), o.decode(dPin, BF)
                dot = (pv * gv).sum(-1, keepdims=True)
                mag = pv * (np.abs(gv) + np.abs(pv * gv).sum(-1, keepdims=True))
                assert self.within(dSg[h][vis], dSo[vis], E5, (pv * (gv - dot))[vis], mag[vis], 1e-5).all()
                dSin = np.where(vis, dSg[h], 0).astype(np.uint8)
                for got, (A, a_dt, a_s, B, b_dt, b_s, tA), out in (
                        (dQg[h], (dSin, E5, dS.scale_value(), kb[h], k_dt, K.scale_value(), False), dQ),
                        (dKg[h], (dSin, E5, dS.scale_value(), qb[h], q_dt, Q.scale_value(), True), dK),
                        (dVg[h], (pb[h], E4, P.scale_value(), gb[h], g_in, dO.scale_value(), True), dV)):
                    Yo, ys, a2, b2 = o.scaled_matmul(A, a_dt, a_s, B, b_dt, b_s, g_dt, transA=tA, want_acc=True)
                    assert out.scale_value() == ys
                    assert self.within(got, Yo, g_dt, a2, b2, 1e-5).all()

    def softmax_bwd(self, dP, P, o_dt):
        dS = self.empty(P.data.shape, o_dt)
        sc.scalify_scaled_softmax_bwd(dP, P, dS)
        self.calls += 1
        if self.check:
            o = self.orc
            gdt, pdt = code(dP.data), code(P.data)
            so, ss = o.softmax_bwd(self.bits(dP), gdt, dP.scale_value(), self.bits(P), pdt, P.scale_value(), o_dt)
            assert dS.scale_value() == ss
            pv, gv = o.decode(self.bits(P), pdt), o.decode(self.bits(dP), gdt)
            dot = (pv * gv).sum(-1, keepdims=True)
            mag = pv * (np.abs(gv) + np.abs(pv * gv).sum(-1, keepdims=True))
            assert self.within(self.bits(dS), so, o_dt, pv * (gv - dot), mag, 4e-6).all()
        return dS

    # ---------------------------------------------------------------- embedding and loss
    def embedding(self, ids, T, wte, wpe):
        n, d = ids.numel(), wte.data.shape[1]
        Y = self.empty((n, d), BF)
        sc.scalify_scaled_embedding(ids, T, wte, wpe, Y)
        self.calls += 1
        if self.check:
            o = self.orc
            dt = code(wte.data)
            yo, ys = o.embedding_fwd(ids.cpu().numpy(), T, self.bits(wte), dt, wte.scale_value(), self.bits(wpe), dt,
                                     wpe.scale_value(), BF)
            assert Y.scale_value() == ys and self.ulp_diff(self.bits(Y), yo, BF).max() <= 1
        return Y

    def embedding_bwd(self, ids, T, dY, vocab):
        n, d = dY.data.shape
        dwte, dwpe = self.empty((vocab, d), F32), self.empty((T, d), F32)
        sc.scalify_scaled_embedding_bwd(ids, T, dY, dwte, dwpe)
        self.calls += 2
        if self.check:
            o = self.orc
            dt = code(dY.data)
            idn = ids.cpu().numpy()
            to, s1, po, s2 = o.embedding_bwd(idn, T, vocab, self.bits(dY), dt, dY.scale_value(), F32)
            assert dwte.scale_value() == s1 and dwpe.scale_value() == s2
            g = np.abs(o.decode(self.bits(dY), dt))
            mag = np.zeros((vocab, d))
            np.add.at(mag, idn, g)
            assert np.all(np.abs(o.decode(self.bits(dwte), F32) - o.decode(to, F32)) <= 2e-6 * mag + 1e-30)
            magp = g.reshape(n // T, T, d).sum(0) / o.kf(n // T)
            assert np.all(np.abs(o.decode(self.bits(dwpe), F32) - o.decode(po, F32)) <= 2e-6 * magp + 1e-30)
        return dwte, dwpe

    def cross_entropy(self, logits, n_classes, targets, g_dt):
        n, ld = logits.data.shape
        G = self.empty((n, ld), g_dt)
        loss = torch.zeros(1, dtype=torch.float32, device=self.dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_CROSS_ENTROPY, n), self.dev)
        sc.scalify_scaled_cross_entropy(logits, n_classes, targets, loss, G, ws)
        self.calls += 2
        if self.check:
            o = self.orc
            assert ws.check_status() == 0
            ldt = code(logits.data)
            tg = targets.cpu().numpy()
            if self.mode == "sampled" and n * ld > self.FULL_LIMIT:
                # The rows are independent.  The loss needs all of them: the oracle is called on chunks of rows
                # (in parallel, it is serial inside) and the chunk means are combined.  The gradient data of a row
                # is (softmax - onehot) times the part of 1/n that is not a power of two; for n and the number of
                # sampled rows both powers of two that part is 1, so the oracle's bits for a subset of rows are
                # the bits of those rows in the full call, and only the scale word (1/n) is set by n.
                from concurrent.futures import ThreadPoolExecutor
                assert n & (n - 1) == 0
                step = 256

                def chunk_loss(r0):
                    lb = self.to_bits(logits.data[r0:r0 + step], ldt).copy()
                    lb[:, n_classes:] = 0
                    l, _, _ = o.cross_entropy(lb, ldt, logits.scale_value(), n_classes, tg[r0:r0 + step], None)
                    return l * min(step, n - r0)
                with ThreadPoolExecutor(max_workers=16) as ex:
                    lo = sum(ex.map(chunk_loss, range(0, n, step))) / n
                assert abs(float(loss.item()) - lo) <= 2e-6 * abs(lo) + 1e-6
                rng = np.random.default_rng(3000 + self.calls)
                rows = np.unique(np.concatenate([rng.integers(0, n, 58), [0, 1, 127, 128, n - 2, n - 1]]))[:64]
                while rows.size & (rows.size - 1):
                    rows = rows[:-1]
                ridx = torch.as_tensor(rows, device=self.dev)
                lb = self.to_bits(logits.data[ridx], ldt).copy()
                lb[:, n_classes:] = 0
                _, go, gs = o.cross_entropy(lb, ldt, logits.scale_value(), n_classes, tg[rows], g_dt)
                _, g64, _ = o.cross_entropy(lb, ldt, logits.scale_value(), n_classes, tg[rows], F32)
                assert G.scale_value() == o.p2f(1.0 / n) and gs == o.p2f(1.0 / rows.size)
                ex = o.decode(g64, F32)
                assert self.within(self.to_bits(G.data[ridx], g_dt), go, g_dt, ex, np.abs(ex) + 1e-6, 8e-6).all()
            else:
                lb = self.bits(logits).copy()
                lb[:, n_classes:] = 0  # padding columns hold whatever the buffer had; the call ignores them
                lo, go, gs = o.cross_entropy(lb, ldt, logits.scale_value(), n_classes, tg, g_dt)
                _, g64, _ = o.cross_entropy(lb, ldt, logits.scale_value(), n_classes, tg, F32)
                assert abs(float(loss.item()) - lo) <= 2e-6 * abs(lo) + 1e-6
                assert G.scale_value() == gs
                ex = o.decode(g64, F32)
                assert self.within(self.bits(G), go, g_dt, ex, np.abs(ex) + 1e-6, 8e-6).all()
        return loss, G
