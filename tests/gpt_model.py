"""A GPT-2-shaped training step (config 5) composed from the scalify C-ABI calls only.

All matmuls are scaled FP8 (E4M3 forward operands, E5M2 gradients, Appendix A), LayerNorm and the
residual stream are BF16, master weights and Adam state are FP16 ScaledArrays (Table 3 row 4), the
loss comes from the fused cross-entropy, and the only dynamic rescales are the L2 rescale of the
gradient leaving each LayerNorm backward (Section 4, two per layer) and the AMAX rescale of each
parameter gradient to E5M2 before the optimizer.  Gradients are always gradients with respect to
VALUES, carried as ScaledArrays.

Every call goes through `checked_ops.Ops`, which can verify each stage against the oracle."""
from collections import OrderedDict
from dataclasses import dataclass

import numpy as np
import torch

import paper_2407_17353_b200 as sc
import scalify_inputs as si
from checked_ops import BF, E4, E5, F16, F32, Ops


@dataclass
class GPTConfig:
    vocab: int = 50257
    seq: int = 1024
    d: int = 768
    heads: int = 12
    layers: int = 12
    batch: int = 8

    @property
    def vocab_padded(self):
        return (self.vocab + 63) // 64 * 64


def _dev(bits, code, dev):
    t = torch.from_numpy(np.ascontiguousarray(bits).view({1: np.int8, 2: np.int16, 4: np.int32}[bits.dtype.itemsize]))
    return t.to(dev).view(sc.TORCH_DTYPE[code])


class ScaledGPT:
    def __init__(self, cfg: GPTConfig, ops: Ops, seed: int = 5, device="cuda"):
        self.cfg, self.ops, self.dev = cfg, ops, device
        d, L = cfg.d, cfg.layers
        self.params = OrderedDict()
        tid = [0]

        def weight(name, shape, std=0.02):
            tid[0] += 1
            data = si.to_bits(si.normal(seed, tid[0], shape, std * 64.0), si.F16)  # value N(0, std) at scale 2^-6
            self.params[name] = sc.ScaledTensor.make(_dev(data, si.F16, device), 2.0 ** -6)

        def vector(name, n, mean, std, scale):
            tid[0] += 1
            data = si.to_bits((mean + std * si.normal(seed, tid[0], (n,))) / scale, si.F16)
            self.params[name] = sc.ScaledTensor.make(_dev(data, si.F16, device), scale)

        weight("wte", (cfg.vocab, d))
        weight("wpe", (cfg.seq, d))
        for l in range(L):
            p = f"h{l}."
            vector(p + "ln1.g", d, 1.0, 0.05, 1.0)
            vector(p + "ln1.b", d, 0.0, 0.02, 2.0 ** -6)
            for nm in ("q", "k", "v", "o"):
                weight(p + "w" + nm, (d, d))
                vector(p + "b" + nm, d, 0.0, 0.01, 2.0 ** -6)
            vector(p + "ln2.g", d, 1.0, 0.05, 1.0)
            vector(p + "ln2.b", d, 0.0, 0.02, 2.0 ** -6)
            weight(p + "w1", (d, 4 * d))
            vector(p + "b1", 4 * d, 0.0, 0.01, 2.0 ** -6)
            weight(p + "w2", (4 * d, d))
            vector(p + "b2", d, 0.0, 0.01, 2.0 ** -6)
        vector("lnf.g", d, 1.0, 0.05, 1.0)
        vector("lnf.b", d, 0.0, 0.02, 2.0 ** -6)
        # Adam state: FP16 zeros with scales chosen near the steady state of g ~ 2^-12
        self.m = OrderedDict((k, sc.ScaledTensor.make(torch.zeros_like(v.data), 2.0 ** -16)) for k, v in self.params.items())
        self.v = OrderedDict((k, sc.ScaledTensor.make(torch.zeros_like(v.data), 2.0 ** -24)) for k, v in self.params.items())
        n = cfg.batch * cfg.seq
        self.adam_ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, len(self.params)), device)

    def n_params(self):
        return sum(v.data.numel() for v in self.params.values())

    # ------------------------------------------------------------------ pieces
    def _heads(self, X, b):
        """[H, T, hd] view of batch element b of a [n, d] tensor (row stride d, head stride hd)."""
        c = self.cfg
        hd = c.d // c.heads
        t = X.data[b * c.seq:(b + 1) * c.seq].view(c.seq, c.heads, hd).permute(1, 0, 2)
        return sc.ScaledTensor(t, X.scale)

    def _heads4(self, X):
        """[B, H, T, hd] view of a [n, d] tensor (batch stride T*d, head stride hd, row stride d)."""
        c = self.cfg
        hd = c.d // c.heads
        return sc.ScaledTensor(X.data.view(c.batch, c.seq, c.heads, hd).permute(0, 2, 1, 3), X.scale)

    def _linear(self, x8, W8, bias, out_dt=BF):
        # [n, K] x [K, N] (B stored [K, N]) + bias in the matmul's epilogue; the sum may be written as FP8 directly
        return self.ops.linear(x8, W8, bias, out_dt=out_dt)

    def _linear_bwd(self, dy, x8, W8, name):
        """dy BF16 -> (dx BF16, dW E5M2 rescaled, db E5M2 rescaled)."""
        o = self.ops
        dy8, colsums = o.cast_colsum(dy, E5)          # the E5M2 copy and its column sums in one pass over dy
        dx = o.mm(dy8, W8, transB=True)               # dy W^T: W stored [K, N] = [N', K'] of this product
        # x^T dy with fused AMAX rescale; a workspace per weight, so that the predicted rescale holds step after step
        _, dW = o.mm(x8, dy8, transA=True, stat=sc.STAT_AMAX, q_dt=E5, key=name)
        db = o.rescale(colsums, sc.STAT_AMAX, E5, key=name + ".bias")          # the bias gradient's dynamic rescale
        return dx, dW, db

    # ------------------------------------------------------------------ one training step
    def step(self, ids, targets, t, lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8, check_layers=None):
        """One training step.  check_layers: the transformer layers whose calls the Ops object checks (None: all);
        embedding, head, loss, the parameter-gradient rescales and the optimizer are always checked."""
        c, o, P = self.cfg, self.ops, self.params
        d, H, T, B = c.d, c.heads, c.seq, c.batch
        hd = d // H
        n = B * T
        W8 = {k: o.cast(v, E4) for k, v in P.items() if v.data.dim() == 2 and k != "wpe"}   # cast_on_forward
        grads = OrderedDict()
        saved = []

        # ---------------- forward
        x = o.embedding(ids, T, P["wte"], P["wpe"])
        for l in range(c.layers):
            p = f"h{l}."
            o.active = check_layers is None or l in check_layers
            s = {"x_in": x}
            # producers write the E4M3 operand of the next matmul themselves (cast_on_forward fused in)
            s["h8"], s["mean1"], s["rinv1"] = o.ln(x, P[p + "ln1.g"], P[p + "ln1.b"], out_dt=E4)
            h8 = s["h8"]
            q8, k8, v8 = (self._linear(h8, W8[p + "w" + nm], P[p + "b" + nm], out_dt=E4) for nm in ("q", "k", "v"))
            s["q8"], s["k8"], s["v8"] = q8, k8, v8
            att = o.empty((n, d), BF)
            att.scale = None
            s["P8"] = []
            att_scale = None
            if hd == 64:
                # Q K^T, 1/sqrt(hd), causal softmax and P V of all sequences and heads in one kernel; the
                # probabilities it used are kept for the backward pass
                Oall = sc.ScaledTensor(self._heads4(sc.ScaledTensor(att.data, None)).data,
                                       torch.empty(1, dtype=torch.float32, device=self.dev))
                s["P8"] = o.attention(self._heads4(q8), self._heads4(k8), self._heads4(v8), Oall, 1.0 / float(np.sqrt(hd)))
                att_scale = Oall.scale
            for b in range(B if hd != 64 else 0):
                Ob = sc.ScaledTensor(self._heads(sc.ScaledTensor(att.data, None), b).data,
                                     torch.empty(1, dtype=torch.float32, device=self.dev))
                S = o.mm(self._heads(q8, b), self._heads(k8, b), transB=True)        # [H, T, T]
                o.scalar_mul(S, 1.0 / float(np.sqrt(hd)))                           # 1/sqrt(hd), a power of two here
                Pb = o.softmax(S, True, E4)
                o.mm(Pb, self._heads(v8, b), Y=Ob)                                   # written into the merged layout
                s["P8"].append(Pb)
                att_scale = Ob.scale  # identical for every b: static rule
            att = sc.ScaledTensor(att.data, att_scale)
            s["o8"] = o8 = o.cast(att, E4)
            x = o.add(x, self._linear(o8, W8[p + "wo"], P[p + "bo"]))
            s["x_mid"] = x
            s["h2_8"], s["mean2"], s["rinv2"] = o.ln(x, P[p + "ln2.g"], P[p + "ln2.b"], out_dt=E4)
            h2_8 = s["h2_8"]
            s["a1"] = a1 = self._linear(h2_8, W8[p + "w1"], P[p + "b1"])
            s["g8"] = g8 = o.gelu(a1, out_dt=E4)
            x = o.add(x, self._linear(g8, W8[p + "w2"], P[p + "b2"]))
            saved.append(s)
        o.active = True
        hf8, meanf, rinvf = o.ln(x, P["lnf.g"], P["lnf.b"], out_dt=E4)
        logits_buf = torch.empty((n, c.vocab_padded), dtype=torch.bfloat16, device=self.dev)
        logits = sc.ScaledTensor(logits_buf[:, :c.vocab], torch.empty(1, dtype=torch.float32, device=self.dev))
        o.mm(hf8, W8["wte"], transB=True, Y=logits)                                  # tied head: wte stored [V, d]
        loss, dlogits = o.cross_entropy(sc.ScaledTensor(logits_buf, logits.scale), c.vocab, targets, E5)

        # ---------------- backward
        dl8 = sc.ScaledTensor(dlogits.data[:, :c.vocab], dlogits.scale)              # [n, V] view, row stride padded
        dhf = o.mm(dl8, W8["wte"])                                                   # [n, V] x [V, d]
        dwte_head = o.mm(dl8, hf8, transA=True, out_dt=F32)                          # [V, n] x [n, d]
        dx, grads["lnf.g"], grads["lnf.b"] = o.ln_bwd(dhf, x, P["lnf.g"], meanf, rinvf)
        for l in reversed(range(c.layers)):
            p = f"h{l}."
            o.active = check_layers is None or l in check_layers
            s = saved[l]
            # MLP
            dg, grads[p + "w2"], grads[p + "b2"] = self._linear_bwd(dx, s["g8"], W8[p + "w2"], p + "w2")
            da1 = o.gelu_bwd(dg, s["a1"])
            dh2, grads[p + "w1"], grads[p + "b1"] = self._linear_bwd(da1, s["h2_8"], W8[p + "w1"], p + "w1")
            dln, grads[p + "ln2.g"], grads[p + "ln2.b"] = o.ln_bwd(dh2, s["x_mid"], P[p + "ln2.g"], s["mean2"], s["rinv2"])
            dx = o.add(dx, dln)
            # attention
            datt, grads[p + "wo"], grads[p + "bo"] = self._linear_bwd(dx, s["o8"], W8[p + "wo"], p + "wo")
            datt8 = o.cast(datt, E5)
            dq, dk, dv = (o.empty((n, d), BF) for _ in range(3))
            if hd == 64:
                # dO V^T, the softmax backward, 1/sqrt(hd) and the three gradient products of all sequences and
                # heads in two launches
                view4 = lambda Tn: sc.ScaledTensor(self._heads4(sc.ScaledTensor(Tn.data, None)).data, Tn.scale)
                o.attention_bwd(self._heads4(s["q8"]), self._heads4(s["k8"]), self._heads4(s["v8"]), s["P8"],
                                self._heads4(datt8), view4(dq), view4(dk), view4(dv), 1.0 / float(np.sqrt(hd)))
            for b in range(B if hd != 64 else 0):
                Pb = s["P8"][b]
                dOb = self._heads(datt8, b)
                view = lambda Tn: sc.ScaledTensor(self._heads(sc.ScaledTensor(Tn.data, None), b).data, Tn.scale)
                dPb = o.mm(dOb, self._heads(s["v8"], b), transB=True)                # dO V^T  [H, T, T]
                o.mm(Pb, dOb, transA=True, Y=view(dv))                               # P^T dO  [H, T, hd]
                dSb = o.softmax_bwd(dPb, Pb, E5)
                o.scalar_mul(dSb, 1.0 / float(np.sqrt(hd)))
                o.mm(dSb, self._heads(s["k8"], b), Y=view(dq))                       # dS K
                o.mm(dSb, self._heads(s["q8"], b), transA=True, Y=view(dk))          # dS^T Q
            dh = None
            for nm, dy in (("q", dq), ("k", dk), ("v", dv)):
                dxx, grads[p + "w" + nm], grads[p + "b" + nm] = self._linear_bwd(dy, s["h8"], W8[p + "w" + nm], p + "w" + nm)
                dh = dxx if dh is None else o.add(dh, dxx)
            dln, grads[p + "ln1.g"], grads[p + "ln1.b"] = o.ln_bwd(dh, s["x_in"], P[p + "ln1.g"], s["mean1"], s["rinv1"])
            dx = o.add(dx, dln)
        o.active = True
        dwte_emb, dwpe = o.embedding_bwd(ids, T, dx, c.vocab)
        grads["wte"] = o.rescale(o.add(dwte_head, dwte_emb), sc.STAT_AMAX, E5, key="wte")
        grads["wpe"] = o.rescale(dwpe, sc.STAT_AMAX, E5, key="wpe")
        for k in list(grads):
            if grads[k].data.dtype != torch.float8_e5m2:                              # LayerNorm dgamma / dbeta (F32)
                grads[k] = o.rescale(grads[k], sc.STAT_AMAX, E5, key=k)
        self.last_grads = grads

        # ---------------- optimizer
        names = list(P)
        G = [sc.ScaledTensor(grads[k].data.reshape(P[k].data.shape), grads[k].scale) for k in names]
        tens = sc.AdamTensors(G, [self.m[k] for k in names], [self.v[k] for k in names], [P[k] for k in names])
        self.before = None
        if o.check:
            self.before = {k: (o.bits(P[k]).copy(), P[k].scale_value(), o.bits(self.m[k]).copy(), self.m[k].scale_value(),
                               o.bits(self.v[k]).copy(), self.v[k].scale_value()) for k in names}
        sc.scalify_scaled_adam_step(tens, self.adam_ws, lr=lr, beta1=beta1, beta2=beta2, eps=eps, step=t)
        o.calls += 2
        if o.check:
            assert self.adam_ws.check_status() == 0
            orc = o.orc
            for k in names:
                w0, ws0, m0, ms0, v0, vs0 = self.before[k]
                mo, vo, wo, ms, vs, wsn = orc.adam_step(o.bits(grads[k]).reshape(-1), E5, grads[k].scale_value(),
                                                        m0.reshape(-1), v0.reshape(-1), F16, ms0, vs0, w0.reshape(-1), F16,
                                                        ws0, lr, beta1, beta2, eps, t)
                assert (self.m[k].scale_value(), self.v[k].scale_value(), P[k].scale_value()) == (ms, vs, wsn), k
                assert o.ulp_diff(o.bits(self.m[k]).reshape(-1), mo, F16).max() <= 1
                assert o.ulp_diff(o.bits(self.v[k]).reshape(-1), vo, F16).max() <= 1
                assert o.ulp_diff(o.bits(P[k]).reshape(-1), wo, F16).max() <= 1
        return loss
