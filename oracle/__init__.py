"""Scalify oracle (TEST INFRASTRUCTURE): ctypes front-end of ``scalify_oracle.cpp``.

The oracle is a plain fp64 CPU statement of the scaled operations of the
Scalify paper (arxiv 2407.17353).  It shares no code with the CUDA library and
must only be used by tests, the smoke check and the CPU-baseline leg of the
benchmark.  Arrays cross this interface as numpy arrays of raw bit patterns
(uint8 for FP8, uint16 for FP16/BF16, uint32 for FP32).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

E4M3, E5M2, F16, BF16, F32 = 0, 1, 2, 3, 4
STAT_NONE, STAT_AMAX, STAT_L2 = 0, 1, 2

_BITS_NP = {E4M3: np.uint8, E5M2: np.uint8, F16: np.uint16, BF16: np.uint16, F32: np.uint32}

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scalify_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c = ctypes
        vp, i32, i64, f32, f64 = c.c_void_p, c.c_int, c.c_int64, c.c_float, c.c_double
        pf32 = c.POINTER(c.c_float)
        L.orc_num_threads.restype = i32
        L.orc_decode.restype = f64
        L.orc_decode.argtypes = [c.c_uint32, i32]
        L.orc_encode.restype = c.c_uint32
        L.orc_encode.argtypes = [f64, i32]
        L.orc_p2f.restype = f64
        L.orc_p2f.argtypes = [f64]
        L.orc_kf.restype = f64
        L.orc_kf.argtypes = [i64]
        L.orc_decode_array.argtypes = [vp, i32, i64, vp]
        L.orc_encode_array.argtypes = [vp, i32, i64, vp]
        L.orc_statistic.restype = f64
        L.orc_statistic.argtypes = [vp, i32, i64, i32]
        L.orc_scaled_matmul.argtypes = [vp, i32, i64, i32, f32, vp, i32, i64, i32, f32, i64, i64, i64,
                                        i32, vp, i64, pf32, vp, vp]
        L.orc_scaled_matmul_delayed.restype = f64
        L.orc_scaled_matmul_delayed.argtypes = [vp, i32, i64, i32, f32, vp, i32, i64, i32, f32, i64, i64, i64, f64, i32,
                                                i32, vp, i64, pf32]
        L.orc_scaled_matmul_samples.argtypes = [vp, i32, i64, i32, vp, i32, i64, i32, i64, i64, vp, vp, vp, vp]
        L.orc_rescale.restype = f64
        L.orc_rescale.argtypes = [vp, i32, i64, f32, i32, f64, i32, vp, pf32]
        L.orc_set_scaling.argtypes = [vp, i32, i64, f32, f32, i32, vp, pf32]
        L.orc_scaled_add.argtypes = [vp, i32, f32, vp, i32, f32, i32, i32, i64, i64, i32, vp, pf32]
        L.orc_layernorm_fwd.argtypes = [vp, i32, i64, i64, vp, i32, f32, vp, i32, f32, f64, i32,
                                        i32, vp, pf32, vp, vp]
        L.orc_layernorm_bwd.argtypes = [vp, i32, f32, vp, i32, f32, vp, i32, f32, i64, i64, f64, i32,
                                        i32, vp, pf32, i32, vp, pf32, vp, pf32, vp]
        L.orc_gelu_fwd.argtypes = [vp, i32, f32, i64, i32, i32, vp, pf32]
        L.orc_gelu_bwd.argtypes = [vp, i32, f32, vp, i32, f32, i64, i32, i32, vp, pf32]
        L.orc_embedding_fwd.argtypes = [vp, i64, i64, i64, vp, i32, f32, vp, i32, f32, i32, vp, pf32]
        L.orc_embedding_bwd.argtypes = [vp, i64, i64, i64, i64, vp, i32, f32, i32, vp, pf32, vp, pf32]
        L.orc_softmax_fwd.argtypes = [vp, i32, f32, i64, i64, i64, i32, i32, vp, pf32]
        L.orc_softmax_bwd.argtypes = [vp, i32, f32, vp, i32, f32, i64, i64, i32, vp, pf32]
        L.orc_cross_entropy.restype = f64
        L.orc_cross_entropy.argtypes = [vp, i32, f32, i64, i64, i64, vp, i32, vp, pf32]
        L.orc_adam_step.argtypes = [i64, vp, i32, f32, vp, vp, i32, pf32, pf32, vp, i32, pf32,
                                    f32, f32, f32, f32, i64]
        L.orc_e8m0_decode.restype = f64
        L.orc_e8m0_decode.argtypes = [c.c_uint32]
        L.orc_mx_quantize.argtypes = [vp, i32, i64, i64, i32, vp, vp]
        L.orc_mx_matmul.argtypes = [vp, i32, vp, f32, vp, i32, vp, f32, i64, i64, i64, i32, vp, i64, pf32, vp, vp]
        _lib = L
    return _lib


def _bits(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != _BITS_NP[dtype]:
        raise TypeError(f"bit-pattern array for dtype {dtype} must be {_BITS_NP[dtype]}, got {a.dtype}")
    return a


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def decode_scalar(bits: int, dtype: int) -> float:
    return float(lib().orc_decode(int(bits), dtype))


def encode_scalar(v: float, dtype: int) -> int:
    return int(lib().orc_encode(float(v), dtype))


def p2f(x: float) -> float:
    return float(lib().orc_p2f(float(x)))


def kf(K: int) -> float:
    return float(lib().orc_kf(int(K)))


def decode(bits: np.ndarray, dtype: int) -> np.ndarray:
    b = _bits(bits, dtype)
    out = np.empty(b.shape, dtype=np.float64)
    lib().orc_decode_array(_ptr(b), dtype, b.size, _ptr(out))
    return out


def encode(values: np.ndarray, dtype: int) -> np.ndarray:
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(v.shape, dtype=_BITS_NP[dtype])
    lib().orc_encode_array(_ptr(v), dtype, v.size, _ptr(out))
    return out


def statistic(x: np.ndarray, dtype: int, stat: int) -> float:
    b = _bits(x, dtype)
    return float(lib().orc_statistic(_ptr(b), dtype, b.size, stat))


def scaled_matmul(A, a_dtype, a_scale, B, b_dtype, b_scale, y_dtype, transA=False, transB=False,
                  want_acc=False):
    """Returns (Y bits [M,N], Y scale, acc fp64 or None, sabs fp64 or None)."""
    A = _bits(A, a_dtype)
    B = _bits(B, b_dtype)
    if transA:
        K, M = A.shape
    else:
        M, K = A.shape
    if transB:
        N, Kb = B.shape
    else:
        Kb, N = B.shape
    assert K == Kb, (A.shape, B.shape, transA, transB)
    Y = np.empty((M, N), dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    acc = np.empty((M, N), dtype=np.float64) if want_acc else None
    sab = np.empty((M, N), dtype=np.float64) if want_acc else None
    lib().orc_scaled_matmul(_ptr(A), a_dtype, A.shape[1], int(transA), float(a_scale),
                            _ptr(B), b_dtype, B.shape[1], int(transB), float(b_scale),
                            M, N, K, y_dtype, _ptr(Y), N, ctypes.byref(ys), _ptr(acc), _ptr(sab))
    return Y, float(ys.value), acc, sab


def scaled_matmul_delayed(A, a_dtype, a_scale, B, b_dtype, b_scale, stat_in, stat, y_dtype, transA=False, transB=False):
    """Matmul whose output is rebalanced by p2f(stat_in) while this step's statistic is gathered.
    Returns (Y bits, Y scale, statistic of the un-rebalanced data)."""
    A = _bits(A, a_dtype)
    B = _bits(B, b_dtype)
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    N = B.shape[0] if transB else B.shape[1]
    Y = np.empty((M, N), dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    s = lib().orc_scaled_matmul_delayed(_ptr(A), a_dtype, A.shape[1], int(transA), float(a_scale), _ptr(B), b_dtype,
                                        B.shape[1], int(transB), float(b_scale), M, N, K, float(stat_in), stat,
                                        y_dtype, _ptr(Y), N, ctypes.byref(ys))
    return Y, float(ys.value), float(s)


def scaled_matmul_samples(A, a_dtype, B, b_dtype, rows, cols, transA=False, transB=False):
    """acc/kf(K) and sum|a*b|/kf(K) at the listed output positions."""
    A = _bits(A, a_dtype)
    B = _bits(B, b_dtype)
    K = A.shape[0] if transA else A.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    acc = np.empty(rows.shape, dtype=np.float64)
    sab = np.empty(rows.shape, dtype=np.float64)
    lib().orc_scaled_matmul_samples(_ptr(A), a_dtype, A.shape[1], int(transA), _ptr(B), b_dtype, B.shape[1],
                                    int(transB), K, rows.size, _ptr(rows), _ptr(cols), _ptr(acc), _ptr(sab))
    return acc, sab


def rescale(x, x_dtype, x_scale, stat, y_dtype, stat_override: float = -1.0):
    """Dynamic rescale.  Returns (Y bits, Y scale, statistic used)."""
    b = _bits(x, x_dtype)
    y = np.empty(b.shape, dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    s = lib().orc_rescale(_ptr(b), x_dtype, b.size, float(x_scale), stat, float(stat_override),
                          y_dtype, _ptr(y), ctypes.byref(ys))
    return y, float(ys.value), float(s)


def set_scaling(x, x_dtype, x_scale, new_scale, y_dtype):
    b = _bits(x, x_dtype)
    y = np.empty(b.shape, dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    lib().orc_set_scaling(_ptr(b), x_dtype, b.size, float(x_scale), float(new_scale), y_dtype, _ptr(y),
                          ctypes.byref(ys))
    return y, float(ys.value)


def scaled_add(A, a_dtype, a_scale, B, b_dtype, b_scale, y_dtype, subtract=False):
    A = _bits(A, a_dtype)
    B = _bits(B, b_dtype)
    A2 = A.reshape(-1, A.shape[-1]) if A.ndim > 1 else A.reshape(1, -1)
    M, N = A2.shape
    bcast = int(B.shape != A.shape)
    if bcast:
        assert B.shape == (N,), (A.shape, B.shape)
    Y = np.empty(A.shape, dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    lib().orc_scaled_add(_ptr(A), a_dtype, float(a_scale), _ptr(B), b_dtype, float(b_scale), bcast,
                         int(subtract), M, N, y_dtype, _ptr(Y), ctypes.byref(ys))
    return Y, float(ys.value)


def layernorm_fwd(X, x_dtype, gamma, g_dtype, g_scale, beta, b_dtype, b_scale, eps, eps_inside_sqrt, y_dtype):
    """Returns (Y bits, Y scale, mean fp64 [R], rinv fp64 [R])."""
    X = _bits(X, x_dtype)
    R, d = X.shape
    gamma = None if gamma is None else _bits(gamma, g_dtype)
    beta = None if beta is None else _bits(beta, b_dtype)
    Y = np.empty((R, d), dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    mean = np.empty(R, dtype=np.float64)
    rinv = np.empty(R, dtype=np.float64)
    lib().orc_layernorm_fwd(_ptr(X), x_dtype, R, d, _ptr(gamma), g_dtype, float(g_scale), _ptr(beta), b_dtype,
                            float(b_scale), float(eps), int(eps_inside_sqrt), y_dtype, _ptr(Y),
                            ctypes.byref(ys), _ptr(mean), _ptr(rinv))
    return Y, float(ys.value), mean, rinv


def layernorm_bwd(G, gr_dtype, gr_scale, X, x_dtype, x_scale, gamma, g_dtype, g_scale, eps, eps_inside_sqrt,
                  dx_dtype, dg_dtype, want_f64=False):
    """Returns dict(dX, dX_scale, dgamma, dgamma_scale, dbeta, dbeta_scale, dx_f64)."""
    G = _bits(G, gr_dtype)
    X = _bits(X, x_dtype)
    R, d = X.shape
    gamma = None if gamma is None else _bits(gamma, g_dtype)
    dX = np.empty((R, d), dtype=_BITS_NP[dx_dtype])
    dg = np.empty(d, dtype=_BITS_NP[dg_dtype])
    db = np.empty(d, dtype=_BITS_NP[dg_dtype])
    dxs, dgs, dbs = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_float(0)
    f64 = np.empty((R, d), dtype=np.float64) if want_f64 else None
    lib().orc_layernorm_bwd(_ptr(G), gr_dtype, float(gr_scale), _ptr(X), x_dtype, float(x_scale),
                            _ptr(gamma), g_dtype, float(g_scale), R, d, float(eps), int(eps_inside_sqrt),
                            dx_dtype, _ptr(dX), ctypes.byref(dxs), dg_dtype, _ptr(dg), ctypes.byref(dgs),
                            _ptr(db), ctypes.byref(dbs), _ptr(f64))
    return dict(dX=dX, dX_scale=float(dxs.value), dgamma=dg, dgamma_scale=float(dgs.value),
                dbeta=db, dbeta_scale=float(dbs.value), dx_f64=f64)


def gelu_fwd(X, x_dtype, x_scale, y_dtype, exact_erf=False):
    X = _bits(X, x_dtype)
    Y = np.empty(X.shape, dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    lib().orc_gelu_fwd(_ptr(X), x_dtype, float(x_scale), X.size, int(exact_erf), y_dtype, _ptr(Y),
                       ctypes.byref(ys))
    return Y, float(ys.value)


def gelu_bwd(G, g_dtype, g_scale, X, x_dtype, x_scale, y_dtype, exact_erf=False):
    G = _bits(G, g_dtype)
    X = _bits(X, x_dtype)
    Y = np.empty(X.shape, dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    lib().orc_gelu_bwd(_ptr(G), g_dtype, float(g_scale), _ptr(X), x_dtype, float(x_scale), X.size,
                       int(exact_erf), y_dtype, _ptr(Y), ctypes.byref(ys))
    return Y, float(ys.value)


def adam_step(g, g_dtype, g_scale, m, v, mv_dtype, m_scale, v_scale, w, w_dtype, w_scale,
              lr, beta1, beta2, eps, step) -> Tuple[np.ndarray, np.ndarray, np.ndarray, float, float, float]:
    """Returns new (m bits, v bits, w bits, m_scale, v_scale, w_scale); inputs are not modified."""
    g = _bits(g, g_dtype)
    m2 = _bits(m, mv_dtype).copy()
    v2 = _bits(v, mv_dtype).copy()
    w2 = _bits(w, w_dtype).copy()
    ms, vs, ws = ctypes.c_float(m_scale), ctypes.c_float(v_scale), ctypes.c_float(w_scale)
    lib().orc_adam_step(g.size, _ptr(g), g_dtype, float(g_scale), _ptr(m2), _ptr(v2), mv_dtype,
                        ctypes.byref(ms), ctypes.byref(vs), _ptr(w2), w_dtype, ctypes.byref(ws),
                        float(lr), float(beta1), float(beta2), float(eps), int(step))
    return m2, v2, w2, float(ms.value), float(vs.value), float(ws.value)


def embedding_fwd(ids, seq_len, wte, wte_dtype, wte_scale, wpe, wpe_dtype, wpe_scale, y_dtype):
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    wte = _bits(wte, wte_dtype)
    wpe = None if wpe is None else _bits(wpe, wpe_dtype)
    d = wte.shape[1]
    Y = np.empty((ids.size, d), dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    lib().orc_embedding_fwd(_ptr(ids), ids.size, int(seq_len), d, _ptr(wte), wte_dtype, float(wte_scale), _ptr(wpe),
                            wpe_dtype, float(wpe_scale), y_dtype, _ptr(Y), ctypes.byref(ys))
    return Y, float(ys.value)


def embedding_bwd(ids, seq_len, vocab, dY, dy_dtype, dy_scale, out_dtype, want_wpe=True):
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    dY = _bits(dY, dy_dtype)
    d = dY.shape[1]
    dwte = np.empty((vocab, d), dtype=_BITS_NP[out_dtype])
    dwpe = np.empty((seq_len, d), dtype=_BITS_NP[out_dtype]) if want_wpe else None
    s1, s2 = ctypes.c_float(0), ctypes.c_float(0)
    lib().orc_embedding_bwd(_ptr(ids), ids.size, int(seq_len), d, int(vocab), _ptr(dY), dy_dtype, float(dy_scale),
                            out_dtype, _ptr(dwte), ctypes.byref(s1), _ptr(dwpe), ctypes.byref(s2))
    return dwte, float(s1.value), dwpe, float(s2.value)


def softmax_fwd(S, s_dtype, s_scale, causal, p_dtype):
    S = _bits(S, s_dtype)
    Tq, Tk = S.shape[-2], S.shape[-1]
    batch = S.size // (Tq * Tk)
    P = np.empty(S.shape, dtype=_BITS_NP[p_dtype])
    ps = ctypes.c_float(0)
    lib().orc_softmax_fwd(_ptr(S), s_dtype, float(s_scale), batch, Tq, Tk, int(causal), p_dtype, _ptr(P),
                          ctypes.byref(ps))
    return P, float(ps.value)


def softmax_bwd(dP, dp_dtype, dp_scale, P, p_dtype, p_scale, ds_dtype):
    dP = _bits(dP, dp_dtype)
    P = _bits(P, p_dtype)
    Tk = P.shape[-1]
    dS = np.empty(P.shape, dtype=_BITS_NP[ds_dtype])
    ss = ctypes.c_float(0)
    lib().orc_softmax_bwd(_ptr(dP), dp_dtype, float(dp_scale), _ptr(P), p_dtype, float(p_scale), P.size // Tk, Tk,
                          ds_dtype, _ptr(dS), ctypes.byref(ss))
    return dS, float(ss.value)


def cross_entropy(logits, l_dtype, l_scale, n_classes, targets, g_dtype=None):
    """Returns (mean loss, dlogits bits or None, dlogits scale)."""
    logits = _bits(logits, l_dtype)
    n, ld = logits.shape
    targets = np.ascontiguousarray(targets, dtype=np.int64)
    g = None if g_dtype is None else np.empty((n, ld), dtype=_BITS_NP[g_dtype])
    gs = ctypes.c_float(0)
    loss = lib().orc_cross_entropy(_ptr(logits), l_dtype, float(l_scale), n, int(n_classes), ld, _ptr(targets),
                                   0 if g_dtype is None else g_dtype, _ptr(g), ctypes.byref(gs))
    return float(loss), g, float(gs.value)


def e8m0_decode(code: int) -> float:
    return float(lib().orc_e8m0_decode(int(code)))


def mx_quantize(X, x_dtype, elem_dtype):
    """Block-scale quantisation of the data component of X [R,K] (K % 32 == 0) along K.
    Returns (element bits [R,K] uint8, E8M0 codes [R,K/32] uint8)."""
    X = _bits(X, x_dtype)
    R, K = X.shape
    assert K % 32 == 0
    data = np.empty((R, K), dtype=np.uint8)
    codes = np.empty((R, K // 32), dtype=np.uint8)
    lib().orc_mx_quantize(_ptr(X), x_dtype, R, K, elem_dtype, _ptr(data), _ptr(codes))
    return data, codes


def mx_matmul(A, a_dtype, Ea, a_scale, B, b_dtype, Eb, b_scale, y_dtype, want_acc=False):
    """A [M,K], B [N,K] FP8 bits, Ea [M,K/32], Eb [N,K/32] E8M0 codes.
    Returns (Y bits [M,N], Y scale, acc or None, sabs or None)."""
    A = _bits(A, a_dtype)
    B = _bits(B, b_dtype)
    Ea = np.ascontiguousarray(Ea, dtype=np.uint8)
    Eb = np.ascontiguousarray(Eb, dtype=np.uint8)
    M, K = A.shape
    N, Kb = B.shape
    assert K == Kb and K % 32 == 0 and Ea.shape == (M, K // 32) and Eb.shape == (N, K // 32)
    Y = np.empty((M, N), dtype=_BITS_NP[y_dtype])
    ys = ctypes.c_float(0)
    acc = np.empty((M, N), dtype=np.float64) if want_acc else None
    sab = np.empty((M, N), dtype=np.float64) if want_acc else None
    lib().orc_mx_matmul(_ptr(A), a_dtype, _ptr(Ea), float(a_scale), _ptr(B), b_dtype, _ptr(Eb), float(b_scale),
                        M, N, K, y_dtype, _ptr(Y), N, ctypes.byref(ys), _ptr(acc), _ptr(sab))
    return Y, float(ys.value), acc, sab
