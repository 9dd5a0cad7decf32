"""Seeded synthetic inputs shared by the oracle-side and CUDA-side harnesses.

This module holds none of the method's arithmetic: it draws numbers from a
counter-based generator (Philox keyed by (seed, tensor id), so the stream does
not depend on thread count or call order) and narrows them to the storage
format with PyTorch's CPU casts, a library routine that neither the oracle nor
the CUDA library uses.  Everything is returned as numpy arrays of raw bit
patterns (uint8 FP8, uint16 FP16/BF16, uint32 FP32).

The workloads follow the GPT-style training shapes of the paper's experiments
(Section 4, Table 2) and the benchmark configurations: Gaussian activations,
weights N(0, 0.02) and gradients N(0,1)*2^-k, each split into unit-variance
data and a power-of-two scale.
"""
from __future__ import annotations

import numpy as np
import torch

E4M3, E5M2, F16, BF16, F32 = 0, 1, 2, 3, 4

_TORCH = {E4M3: torch.float8_e4m3fn, E5M2: torch.float8_e5m2, F16: torch.float16,
          BF16: torch.bfloat16, F32: torch.float32}
_VIEW = {E4M3: torch.uint8, E5M2: torch.uint8, F16: torch.int16, BF16: torch.int16, F32: torch.int32}
_NP = {E4M3: np.uint8, E5M2: np.uint8, F16: np.uint16, BF16: np.uint16, F32: np.uint32}
ELEM_SIZE = {E4M3: 1, E5M2: 1, F16: 2, BF16: 2, F32: 4}


def normal(seed: int, tensor_id: int, shape, std: float = 1.0) -> np.ndarray:
    """fp32 N(0, std^2) draws from Philox keyed by (seed, tensor_id)."""
    gen = np.random.Generator(np.random.Philox(key=[int(seed), int(tensor_id)]))
    x = gen.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def uniform_int(seed: int, tensor_id: int, shape, high: int) -> np.ndarray:
    gen = np.random.Generator(np.random.Philox(key=[int(seed), int(tensor_id)]))
    return gen.integers(0, high, size=shape, dtype=np.int64)


def to_bits(values: np.ndarray, dtype: int) -> np.ndarray:
    """Round-to-nearest narrowing with torch's CPU cast; returns raw bit patterns."""
    t = torch.from_numpy(np.ascontiguousarray(values, dtype=np.float32))
    if dtype in (E4M3, E5M2):
        lim = 448.0 if dtype == E4M3 else 57344.0
        t = t.clamp(-lim, lim)
    q = t.to(_TORCH[dtype]).view(_VIEW[dtype]).numpy()
    return q.view(_NP[dtype])


def from_bits(bits: np.ndarray, dtype: int) -> np.ndarray:
    """fp64 values of raw bit patterns through torch's CPU cast (library decode)."""
    b = np.ascontiguousarray(bits)
    t = torch.from_numpy(b.view({1: np.uint8, 2: np.int16, 4: np.int32}[b.dtype.itemsize]))
    return t.view(_TORCH[dtype]).to(torch.float64).numpy()


def scaled_normal(seed: int, tensor_id: int, shape, dtype: int, data_std: float = 1.0):
    """Data bits of round-to-nearest(dtype) of N(0, data_std^2)."""
    return to_bits(normal(seed, tensor_id, shape, data_std), dtype)


# ---------------------------------------------------------------------------
# benchmark / parity configurations
# ---------------------------------------------------------------------------

def config1(seed: int = 0):
    """Single scaled matmul: A, B 256x256 E4M3 data = rn(N(0,1)*2^3), scales 2^-3 and 2^2."""
    A = scaled_normal(seed, 1, (256, 256), E4M3, 8.0)
    B = scaled_normal(seed, 2, (256, 256), E4M3, 8.0)
    return dict(A=A, a_dtype=E4M3, a_scale=2.0 ** -3, B=B, b_dtype=E4M3, b_scale=2.0 ** 2)


def gemm_case(n: int, kind: str, seed: int, m: int | None = None, k: int | None = None):
    """Scaled GEMM sweep case.  kind 'fwd': E4M3 x E4M3, scales 1 and 2^-6 (weight-like);
    kind 'grad': E5M2 gradient (value N(0,1)*2^-10 => data N(0,1), scale 2^-10) x E4M3.
    A is [M,K]; B is given both as [K,N] ('B') and as its transpose [N,K] ('Bt')."""
    M = n if m is None else m
    K = n if k is None else k
    a_dtype = E4M3 if kind == "fwd" else E5M2
    a_scale = 1.0 if kind == "fwd" else 2.0 ** -10
    A = scaled_normal(seed, 1, (M, K), a_dtype)
    Bt = scaled_normal(seed, 2, (n, K), E4M3)
    return dict(A=A, a_dtype=a_dtype, a_scale=a_scale, Bt=Bt, b_dtype=E4M3, b_scale=2.0 ** -6,
                M=M, N=n, K=K)


def adam_case(n: int, seed: int = 4, w_dtype: int = F16):
    """Steady-state scaled Adam inputs: w value N(0,0.02) at scale 2^-6; g value N(0,1)*2^-12 as E5M2 data
    at scale 2^-12; m ~ 0.1*N(0,1)*2^-12 (FP16 data N(0,1)*0.1*2^4 at scale 2^-16); v ~ (N(0,1)*2^-12)^2
    (FP16 data at scale 2^-24)."""
    w = to_bits(normal(seed, 1, (n,), 0.02 * 64.0), w_dtype)
    g = scaled_normal(seed, 2, (n,), E5M2)
    m = to_bits(normal(seed, 3, (n,), 0.1 * 16.0), F16)
    vv = normal(seed, 4, (n,))
    v = to_bits(vv * vv, F16)
    return dict(w=w, w_dtype=w_dtype, w_scale=2.0 ** -6, g=g, g_dtype=E5M2, g_scale=2.0 ** -12,
                m=m, v=v, mv_dtype=F16, m_scale=2.0 ** -16, v_scale=2.0 ** -24,
                lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8, step=1000)


def gpt2_small_param_shapes():
    """The 148 parameter tensors of a GPT-2-small-shaped model (tied lm head): 124,439,808 parameters."""
    d, L, V, T = 768, 12, 50257, 1024
    shapes = [(V, d), (T, d)]
    for _ in range(L):
        shapes += [(d,), (d,), (d, 3 * d), (3 * d,), (d, d), (d,),
                   (d,), (d,), (d, 4 * d), (4 * d,), (4 * d, d), (d,)]
    shapes += [(d,), (d,)]
    return shapes


def layernorm_case(R: int, d: int, seed: int = 3, x_dtype: int = BF16):
    """x ~ N(0,1) (scale 1), gamma ~ 1 + 0.1 N(0,1), beta ~ 0.1 N(0,1), upstream gradient value
    N(0,1)*2^-10 as data N(0,1) at scale 2^-10."""
    X = scaled_normal(seed, 1, (R, d), x_dtype)
    gamma = to_bits(1.0 + 0.1 * normal(seed, 2, (d,)), BF16)
    beta = to_bits(0.1 * normal(seed, 3, (d,)), BF16)
    G = scaled_normal(seed, 4, (R, d), BF16)
    return dict(X=X, x_dtype=x_dtype, x_scale=1.0, gamma=gamma, beta=beta, gb_dtype=BF16,
                gamma_scale=1.0, beta_scale=1.0, G=G, g_dtype=BF16, g_scale=2.0 ** -10, eps=1e-5)
