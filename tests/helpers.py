"""Shared helpers of the GPU parity tests: bit-pattern transport between numpy
(oracle side) and torch CUDA tensors (library side), and ulp distances."""
import numpy as np
import torch

import oracle as orc

TORCH_DT = {orc.E4M3: torch.float8_e4m3fn, orc.E5M2: torch.float8_e5m2, orc.F16: torch.float16,
            orc.BF16: torch.bfloat16, orc.F32: torch.float32}
NP_BITS = {orc.E4M3: np.uint8, orc.E5M2: np.uint8, orc.F16: np.uint16, orc.BF16: np.uint16, orc.F32: np.uint32}
_SIGNED = {1: np.int8, 2: np.int16, 4: np.int32}
_TSIGNED = {1: torch.int8, 2: torch.int16, 4: torch.int32}
NBITS = {orc.E4M3: 8, orc.E5M2: 8, orc.F16: 16, orc.BF16: 16, orc.F32: 32}


def to_dev(bits: np.ndarray, dtype: int, device="cuda") -> torch.Tensor:
    """numpy bit patterns -> CUDA tensor of the matching torch dtype (no value conversion)."""
    b = np.ascontiguousarray(bits)
    t = torch.from_numpy(b.view(_SIGNED[b.dtype.itemsize])).to(device)
    return t.view(TORCH_DT[dtype])


def to_bits(t: torch.Tensor, dtype: int) -> np.ndarray:
    """CUDA tensor -> numpy bit patterns."""
    c = t.detach().contiguous().view(_TSIGNED[t.element_size()]).cpu().numpy()
    return c.view(NP_BITS[dtype])


def ordered(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Monotone integer image of sign-magnitude bit patterns (+0 and -0 both map to 0)."""
    n = NBITS[dtype]
    b = bits.astype(np.int64)
    mag = b & ((1 << (n - 1)) - 1)
    return np.where((b >> (n - 1)) & 1, -mag, mag)


def ulp_diff(a: np.ndarray, b: np.ndarray, dtype: int) -> np.ndarray:
    """Distance in representable values; NaN vs NaN counts as 0, NaN vs number as a huge distance."""
    va, vb = orc.decode(a, dtype), orc.decode(b, dtype)
    d = np.abs(ordered(a, dtype) - ordered(b, dtype))
    both_nan = np.isnan(va) & np.isnan(vb)
    one_nan = np.isnan(va) ^ np.isnan(vb)
    d = np.where(both_nan, 0, d)
    d = np.where(one_nan, 1 << 40, d)
    return d


def scale_of(t) -> float:
    return float(t.scale.item())


_MBITS = {orc.E4M3: 3, orc.E5M2: 2, orc.F16: 10, orc.BF16: 7, orc.F32: 23}
_EMIN = {orc.E4M3: -6, orc.E5M2: -14, orc.F16: -14, orc.BF16: -126, orc.F32: -126}


def ulp_of(x: np.ndarray, dtype: int) -> np.ndarray:
    """Spacing of the format `dtype` at magnitude |x| (the subnormal quantum below the smallest normal)."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(ax > 0, ax, 1.0)))
    e = np.maximum(np.where(ax > 0, e, _EMIN[dtype]), _EMIN[dtype])
    return np.exp2(e - _MBITS[dtype])


# Every call of within() leaves a record here: (label, elements, elements accepted ONLY by the
# cancellation clause).  conftest.py writes the totals per label at the end of a session when
# SCALIFY_TOLERANCE_LOG names a file, so the share of outputs that lean on the wider clause is a
# measured number and not an assumption.
LOOSE_LOG = []
_DT_NAME = {orc.E4M3: "e4m3", orc.E5M2: "e5m2", orc.F16: "f16", orc.BF16: "bf16", orc.F32: "f32"}

# An output may need the cancellation clause only when the fp32 rounding error of the sum (a few
# 2^-24 of its largest terms) exceeds an ulp of the RESULT, i.e. when |result| is below about
# 2^(mantissa bits) * 2^-22 of its terms: 2^-15 of them for BF16, 2^-19 / 2^-20 for FP8.  For the
# Gaussian workloads here that is far below one output in a hundred, so a kernel that is more than
# 1 ulp off on ordinary outputs exceeds the cap and fails, whatever c and err_mag are.
LOOSE_CAP = 0.01
LOOSE_FLOOR = 2   # tiny arrays: a couple of outputs near a zero crossing are not a share


def _caller_label():
    import inspect
    for fr in inspect.stack()[2:8]:
        if fr.function.startswith("test_") or fr.function in ("smoke",):
            return fr.function
    return inspect.stack()[2].function


def within(got_bits, want_bits, dtype, exact, err_mag, c, loose_cap=LOOSE_CAP, label=None):
    """Mask of acceptable outputs for a result computed in fp32 and rounded once to `dtype`:
    within 1 ulp of the oracle's encoding, or |value - exact| <= ulp(exact)/2 + c * err_mag, where
    err_mag is the magnitude of the terms that were added (a sum that cancels has an error
    relative to its terms, not to its result).  The second clause may carry at most `loose_cap` of
    the outputs (plus LOOSE_FLOOR of them): beyond that the outputs it alone accepted count as
    failures.  The number it carried is recorded in LOOSE_LOG.  An fp32 OUTPUT is the exception: it comes
    out of several fp32 operations, so it is a few fp32 ulp from the fp64 result on every element and the
    second clause (c * err_mag, a few 2^-24 of the terms) is its bar; no cap applies."""
    d = ulp_diff(got_bits, want_bits, dtype)
    err = np.abs(orc.decode(got_bits, dtype) - exact)
    tight = d <= 1
    with np.errstate(invalid="ignore"):
        loose = ~tight & (err <= 0.5 * ulp_of(exact, dtype) + c * err_mag)
    n, n_loose = int(tight.size), int(loose.sum())
    LOOSE_LOG.append(((label or _caller_label()) + ":" + _DT_NAME[dtype], n, n_loose))
    if dtype != orc.F32 and n_loose > loose_cap * n + LOOSE_FLOOR:
        return tight
    return tight | loose


def layernorm_bwd_delayed(G, gr_dtype, gr_scale, X, x_dtype, x_scale, gamma, g_dtype, g_scale, eps, eps_inside_sqrt,
                          stat_in, stat, dx_dtype, dg_dtype):
    """LayerNorm backward with DELAYED rescaling of the input gradient (Section 3.3 applied to the
    rescale site of Section 4): a composition of the oracle's pieces, no arithmetic of its own beyond
    the division by r.  The gradient is written already rebalanced by r = p2f(stat_in) (1 if stat_in
    cannot define a scale), rounded once from the oracle's fp64 derivative, and this step's statistic
    is taken on the un-rebalanced, unrounded derivative.
    Returns dict(dX, dX_scale, stat, dgamma, dgamma_scale, dbeta, dbeta_scale, dx_f64, r)."""
    o = orc.layernorm_bwd(G, gr_dtype, gr_scale, X, x_dtype, x_scale, gamma, g_dtype, g_scale, eps, eps_inside_sqrt,
                          orc.F32, dg_dtype, want_f64=True)
    usable = np.isfinite(stat_in) and stat_in >= 2.0 ** -126
    r = orc.p2f(float(stat_in)) if usable else 1.0
    dx = o["dx_f64"]
    o["dX"] = orc.encode(dx / r, dx_dtype)
    o["dX_scale"] = o["dX_scale"] * r
    o["stat"] = float(np.abs(dx).max()) if stat == orc.STAT_AMAX else float(np.sqrt(np.mean(dx * dx)))
    o["r"] = r
    return o
