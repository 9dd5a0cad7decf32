"""Python binding of the scalify C ABI (``include/scalify.h``).

Argument marshalling only: every arithmetic step runs in the CUDA library
``libscalify.so`` (hand-written sm_100a kernels).  PyTorch supplies device
memory and streams.  There is no CPU or PyTorch fallback: if the library
cannot be loaded, importing the symbols below raises.

A :class:`ScaledTensor` is the paper's ScaledArray (Section 2): ``data`` in a
low-precision dtype plus ONE fp32 power-of-two ``scale`` kept on the device,
with value = data * scale.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

from . import _build

E4M3, E5M2, F16, BF16, F32 = 0, 1, 2, 3, 4
STAT_NONE, STAT_AMAX, STAT_L2 = 0, 1, 2
OP_MATMUL, OP_RESCALE, OP_LAYERNORM_BWD, OP_ADAM, OP_STATISTIC, OP_CROSS_ENTROPY, OP_COLSUM, OP_MATMUL_SPLITK = (
    0, 1, 2, 3, 4, 5, 6, 7)
DEV_TIMEOUT, DEV_BAD_SCALE, DEV_NONFINITE_STAT, DEV_BAD_INDEX = 1, 2, 4, 8

_DTYPE_CODE = {torch.float8_e4m3fn: E4M3, torch.float8_e5m2: E5M2, torch.float16: F16,
               torch.bfloat16: BF16, torch.float32: F32}
TORCH_DTYPE = {v: k for k, v in _DTYPE_CODE.items()}


class ScalifyError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().scalify_status_string(code).decode()
        extra = f" (cudaError {lib().scalify_last_cuda_error()})" if code == -7 else ""
        super().__init__(f"{where}: {msg}{extra} [code {code}]")


class scalify_array(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("ndim", ctypes.c_int32),
                ("shape", ctypes.c_int64 * 4), ("stride", ctypes.c_int64 * 4), ("scale", ctypes.c_void_p)]


class scalify_mx_array(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("rows", ctypes.c_int64), ("K", ctypes.c_int64),
                ("sf", ctypes.c_void_p), ("scale", ctypes.c_void_p), ("transposed", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libscalify.so`` (building it with nvcc if it is not there).  Raises if neither works.
    With ``SCALIFY_DEBUG_BUILD=1`` in the environment the bounds-checking build ``libscalify_debug.so`` is loaded
    instead (see ``scalify_debug_bounds_report`` in ``include/scalify.h``)."""
    global _lib
    if _lib is None:
        debug = os.environ.get("SCALIFY_DEBUG_BUILD", "") == "1"
        path = _build.LIB_DEBUG if debug else _build.LIB
        if not os.path.exists(path):
            path = _build.build(debug=debug)
        L = ctypes.CDLL(path)
        c = ctypes
        P = c.POINTER(scalify_array)
        vp, i32, i64, f32, sz = c.c_void_p, c.c_int, c.c_int64, c.c_float, c.c_size_t
        L.scalify_version.restype = i32
        L.scalify_last_cuda_error.restype = i32
        L.scalify_status_string.restype = c.c_char_p
        L.scalify_status_string.argtypes = [i32]
        L.scalify_workspace_bytes.restype = sz
        L.scalify_workspace_bytes.argtypes = [i32, i64, i64]
        L.scalify_workspace_init.argtypes = [vp, sz, vp]
        L.scalify_check_status.argtypes = [vp, vp]
        L.scalify_scaled_matmul.argtypes = [P, i32, P, i32, P, i32, P, vp, sz, vp]
        L.scalify_scaled_matmul_speculative.argtypes = [P, i32, P, i32, P, P, vp, vp, sz, vp]
        L.scalify_statistic.argtypes = [P, i32, vp, vp, sz, vp]
        L.scalify_scaled_matmul_delayed.argtypes = [P, i32, P, i32, vp, P, i32, vp, vp, sz, vp]
        L.scalify_rescale.argtypes = [P, i32, vp, vp, P, vp, sz, vp]
        L.scalify_scaled_add.argtypes = [P, P, i32, P, vp]
        L.scalify_scaled_layernorm.argtypes = [P, P, P, f32, i32, P, vp, vp, vp]
        L.scalify_scaled_layernorm_bwd_delayed.argtypes = [P, P, P, vp, vp, f32, i32, vp, i32, P, P, P, vp, sz, vp]
        L.scalify_scaled_layernorm_bwd.argtypes = [P, P, P, vp, vp, f32, i32, i32, P, P, P, P, vp, sz, vp]
        L.scalify_scaled_gelu.argtypes = [P, i32, P, vp]
        L.scalify_scaled_gelu_bwd.argtypes = [P, P, i32, P, vp]
        L.scalify_scaled_adam_step.argtypes = [i32, P, P, P, P, f32, f32, f32, f32, i64, vp, sz, vp]
        L.scalify_scaled_attention.argtypes = [P, P, P, f32, i32, P, P, P, vp, vp]
        L.scalify_scaled_colsum.argtypes = [P, P, vp, sz, vp]
        L.scalify_scaled_cast_colsum.argtypes = [P, P, P, vp, sz, vp]
        L.scalify_scaled_matmul_bias.argtypes = [P, i32, P, i32, P, P, i32, P, vp, sz, vp]
        L.scalify_scaled_attention_bwd.argtypes = [P, P, P, P, P, f32, i32, P, P, P, P, P, vp, vp]
        L.scalify_mx_sf_bytes.restype = sz
        L.scalify_mx_sf_bytes.argtypes = [i64, i64]
        L.scalify_mx_quantize.argtypes = [P, vp, vp, vp]
        L.scalify_mx_matmul.argtypes = [vp, vp, P, i32, vp, sz, vp]
        L.scalify_scaled_adam_step_cast.argtypes = [i32, P, P, P, P, P, f32, f32, f32, f32, i64, vp, sz, vp]
        L.scalify_debug_expire_wait.argtypes = [vp, sz, c.c_uint32, vp, vp]
        L.scalify_scalar_mul_pow2.argtypes = [P, f32, vp]
        L.scalify_debug_layernorm_plan.argtypes = [i64, i64, i32, i32, vp]
        L.scalify_debug_host_state_selftest.restype = i32
        L.scalify_debug_bounds_report.argtypes = [vp, i32, i64]
        L.scalify_debug_bounds_report.restype = i32
        L.scalify_debug_bf16_round.argtypes = [vp, vp, i64, i32, vp]
        L.scalify_debug_bf16_round.restype = i32
        L.scalify_debug_tensor_map_cache.argtypes = [vp, vp]
        L.scalify_debug_tensor_map_cache.restype = i32
        L.scalify_scaled_embedding.argtypes = [vp, i64, i64, P, P, P, vp, vp]
        L.scalify_scaled_embedding_bwd.argtypes = [vp, i64, i64, P, P, P, vp]
        L.scalify_scaled_softmax.argtypes = [P, i32, P, vp]
        L.scalify_scaled_softmax_bwd.argtypes = [P, P, P, vp]
        L.scalify_scaled_cross_entropy.argtypes = [P, i64, vp, vp, P, vp, sz, vp]
        L.scalify_scaled_adam_step_static.argtypes = [i32, P, P, P, P, f32, f32, f32, f32, i64, vp, vp]
        for name in ("scalify_workspace_init", "scalify_check_status", "scalify_scaled_matmul", "scalify_scaled_matmul_delayed",
                     "scalify_statistic",
                     "scalify_rescale", "scalify_scaled_add", "scalify_scaled_layernorm",
                     "scalify_scaled_layernorm_bwd", "scalify_scaled_gelu", "scalify_scaled_gelu_bwd",
                     "scalify_scaled_adam_step", "scalify_scaled_adam_step_cast", "scalify_scaled_adam_step_static", "scalify_scaled_embedding",
                     "scalify_scaled_embedding_bwd", "scalify_scaled_softmax", "scalify_scaled_softmax_bwd",
                     "scalify_scaled_cross_entropy", "scalify_scalar_mul_pow2", "scalify_debug_expire_wait",
                     "scalify_debug_layernorm_plan",
                     "scalify_mx_quantize", "scalify_mx_matmul", "scalify_scaled_attention",
                     "scalify_scaled_attention_bwd", "scalify_scaled_colsum", "scalify_scaled_cast_colsum", "scalify_scaled_matmul_bias",
                     "scalify_scaled_matmul_speculative"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


@dataclass
class ScaledTensor:
    """ScaledArray (Section 2): value = data * scale.  ``scale`` is a 1-element fp32 CUDA tensor or None
    (unscaled: scale 1)."""
    data: torch.Tensor
    scale: Optional[torch.Tensor] = None

    @staticmethod
    def empty(shape, dtype, device="cuda") -> "ScaledTensor":
        return ScaledTensor(torch.empty(shape, dtype=dtype, device=device),
                            torch.empty(1, dtype=torch.float32, device=device))

    @staticmethod
    def make(data: torch.Tensor, scale: float) -> "ScaledTensor":
        return ScaledTensor(data, torch.full((1,), float(scale), dtype=torch.float32, device=data.device))

    def scale_value(self) -> float:
        return 1.0 if self.scale is None else float(self.scale.item())


def _desc(t: Optional[ScaledTensor]):
    """ctypes descriptor of a ScaledTensor (None -> NULL); cached on the object while its buffers stay the same."""
    if t is None:
        return None
    d = t.data
    sp = 0 if t.scale is None else t.scale.data_ptr()
    key = (d.data_ptr(), d.dtype, tuple(d.shape), d.stride(), sp)
    cached = t.__dict__.get("_desc_cache")
    if cached is not None and cached[0] == key:
        return cached[1]
    if d.dim() < 1 or d.dim() > 4:
        raise ValueError("scalify arrays have 1 to 4 dimensions")
    a = scalify_array()
    a.data = d.data_ptr()
    a.dtype = _DTYPE_CODE[d.dtype]
    a.ndim = d.dim()
    for i in range(d.dim()):
        a.shape[i] = d.shape[i]
        a.stride[i] = d.stride(i)
    if t.scale is not None:
        if t.scale.dtype != torch.float32 or t.scale.numel() != 1 or t.scale.device != d.device:
            raise ValueError("scale must be a 1-element fp32 tensor on the data's device")
        a.scale = sp
    else:
        a.scale = None
    t.__dict__["_desc_cache"] = (key, a)
    return a


def _ref(a):
    return None if a is None else ctypes.byref(a)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise ScalifyError(code, where)


class Workspace:
    """Caller-owned scratch buffer with the zeroed 256-byte header the library expects."""

    def __init__(self, nbytes: int, device="cuda", stream=None):
        nbytes = max(int(nbytes), 4096)
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.nbytes = nbytes
        _check(lib().scalify_workspace_init(self.buf.data_ptr(), nbytes, _stream(stream)), "scalify_workspace_init")

    @property
    def ptr(self) -> int:
        return self.buf.data_ptr()

    def statistic(self) -> torch.Tensor:
        """The fp32 statistic word (byte offset 16) as a 1-element tensor view."""
        return self.buf[16:20].view(torch.float32)

    def prediction(self) -> torch.Tensor:
        """The AMAX statistic of the last matmul + FP8 rescale on this workspace (byte offset 56), which the next
        such call uses as its prediction; a 1-element tensor view."""
        return self.buf[56:60].view(torch.float32)

    def check_status(self, stream=None) -> int:
        return scalify_check_status(self, stream)


def scalify_workspace_bytes(op: int, d0: int = 0, d1: int = 0) -> int:
    return int(lib().scalify_workspace_bytes(op, int(d0), int(d1)))


def scalify_check_status(ws: Workspace, stream=None) -> int:
    rc = lib().scalify_check_status(ws.ptr, _stream(stream))
    if rc < 0:
        raise ScalifyError(rc, "scalify_check_status")
    return rc


def scalify_scaled_matmul(A: ScaledTensor, B: ScaledTensor, Y: Optional[ScaledTensor], ws: Workspace, *, transA=False,
                          transB=False, stat: int = STAT_NONE, Yq: Optional[ScaledTensor] = None, stream=None) -> None:
    """Y may be None with stat=STAT_AMAX and an FP8 Yq: only the rescaled output is stored."""
    a, b, y, yq = _desc(A), _desc(B), _desc(Y), _desc(Yq)
    _check(lib().scalify_scaled_matmul(_ref(a), int(transA), _ref(b), int(transB), _ref(y), stat, _ref(yq),
                                       ws.ptr, ws.nbytes, _stream(stream)), "scalify_scaled_matmul")


def scalify_scaled_matmul_bias(A: ScaledTensor, B: ScaledTensor, bias: ScaledTensor, Y: ScaledTensor, ws: Workspace, *,
                               transA=False, transB=False, stat: int = STAT_NONE, Yq: Optional[ScaledTensor] = None,
                               stream=None) -> None:
    """Y = A B + bias (a [N] vector) in the GEMM's epilogue, by the add rule and with one rounding."""
    a, b, bi, y, yq = _desc(A), _desc(B), _desc(bias), _desc(Y), _desc(Yq)
    _check(lib().scalify_scaled_matmul_bias(_ref(a), int(transA), _ref(b), int(transB), _ref(bi), _ref(y), stat,
                                            _ref(yq), ws.ptr, ws.nbytes, _stream(stream)), "scalify_scaled_matmul_bias")


def scalify_scaled_matmul_speculative(A: ScaledTensor, B: ScaledTensor, Y: ScaledTensor, Yq: ScaledTensor,
                                      stat_hint: torch.Tensor, ws: Workspace, *, transA=False, transB=False,
                                      stream=None) -> None:
    """GEMM + exact AMAX rescale to FP8 where the GEMM already writes Yq with a predicted factor (stat_hint: a
    1-element fp32 CUDA tensor, read as the prediction and overwritten with this call's statistic)."""
    a, b, y, yq = _desc(A), _desc(B), _desc(Y), _desc(Yq)
    _check(lib().scalify_scaled_matmul_speculative(_ref(a), int(transA), _ref(b), int(transB), _ref(y), _ref(yq),
                                                   _ptr(stat_hint), ws.ptr, ws.nbytes, _stream(stream)),
           "scalify_scaled_matmul_speculative")


def scalify_scaled_matmul_delayed(A: ScaledTensor, B: ScaledTensor, stat_in: torch.Tensor, Y: ScaledTensor,
                                  ws: Workspace, *, transA=False, transB=False, stat: int = STAT_AMAX,
                                  stat_out: Optional[torch.Tensor] = None, stream=None) -> None:
    a, b, y = _desc(A), _desc(B), _desc(Y)
    _check(lib().scalify_scaled_matmul_delayed(_ref(a), int(transA), _ref(b), int(transB), _ptr(stat_in), _ref(y),
                                               stat, _ptr(stat_out), ws.ptr, ws.nbytes, _stream(stream)),
           "scalify_scaled_matmul_delayed")


def scalify_statistic(X: ScaledTensor, stat: int, ws: Workspace, out: Optional[torch.Tensor] = None, stream=None) -> None:
    x = _desc(X)
    _check(lib().scalify_statistic(_ref(x), stat, _ptr(out), ws.ptr, ws.nbytes, _stream(stream)), "scalify_statistic")


def scalify_rescale(X: ScaledTensor, Y: ScaledTensor, *, stat: int = STAT_NONE, new_scale: Optional[torch.Tensor] = None,
                    stat_in: Optional[torch.Tensor] = None, ws: Optional[Workspace] = None, stream=None) -> None:
    x, y = _desc(X), _desc(Y)
    _check(lib().scalify_rescale(_ref(x), stat, _ptr(new_scale), _ptr(stat_in), _ref(y),
                                 None if ws is None else ws.ptr, 0 if ws is None else ws.nbytes, _stream(stream)),
           "scalify_rescale")


def scalify_scaled_add(A: ScaledTensor, B: ScaledTensor, Y: ScaledTensor, *, subtract=False, stream=None) -> None:
    a, b, y = _desc(A), _desc(B), _desc(Y)
    _check(lib().scalify_scaled_add(_ref(a), _ref(b), int(subtract), _ref(y), _stream(stream)), "scalify_scaled_add")


def scalify_scaled_layernorm(X: ScaledTensor, gamma: Optional[ScaledTensor], beta: Optional[ScaledTensor],
                             Y: ScaledTensor, *, eps: float = 1e-5, eps_inside_sqrt=False,
                             mean: Optional[torch.Tensor] = None, rinv: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    x, g, b, y = _desc(X), _desc(gamma), _desc(beta), _desc(Y)
    _check(lib().scalify_scaled_layernorm(_ref(x), _ref(g), _ref(b), float(eps), int(eps_inside_sqrt), _ref(y),
                                          _ptr(mean), _ptr(rinv), _stream(stream)), "scalify_scaled_layernorm")


def scalify_scaled_layernorm_bwd(G: ScaledTensor, X: ScaledTensor, gamma: Optional[ScaledTensor], mean: torch.Tensor,
                                 rinv: torch.Tensor, dX: Optional[ScaledTensor], ws: Workspace, *, eps: float = 1e-5,
                                 eps_inside_sqrt=False, stat_dx: int = STAT_NONE, dXq: Optional[ScaledTensor] = None,
                                 dgamma: Optional[ScaledTensor] = None, dbeta: Optional[ScaledTensor] = None,
                                 stream=None) -> None:
    g, x, gm, dx, dxq, dg, db = (_desc(G), _desc(X), _desc(gamma), _desc(dX), _desc(dXq), _desc(dgamma), _desc(dbeta))
    _check(lib().scalify_scaled_layernorm_bwd(_ref(g), _ref(x), _ref(gm), _ptr(mean), _ptr(rinv), float(eps),
                                              int(eps_inside_sqrt), stat_dx, _ref(dx), _ref(dxq), _ref(dg), _ref(db),
                                              ws.ptr, ws.nbytes, _stream(stream)), "scalify_scaled_layernorm_bwd")


def scalify_scaled_layernorm_bwd_delayed(G: ScaledTensor, X: ScaledTensor, gamma: Optional[ScaledTensor],
                                         mean: torch.Tensor, rinv: torch.Tensor, stat_in: torch.Tensor, dX: ScaledTensor,
                                         ws: Workspace, *, eps: float = 1e-5, eps_inside_sqrt=False,
                                         stat_dx: int = STAT_NONE, dgamma: Optional[ScaledTensor] = None,
                                         dbeta: Optional[ScaledTensor] = None, stream=None) -> None:
    """LayerNorm backward writing the gradient already rebalanced by the power of two of an earlier statistic."""
    g, x, gm, dx, dg, db = (_desc(G), _desc(X), _desc(gamma), _desc(dX), _desc(dgamma), _desc(dbeta))
    _check(lib().scalify_scaled_layernorm_bwd_delayed(_ref(g), _ref(x), _ref(gm), _ptr(mean), _ptr(rinv), float(eps),
                                                      int(eps_inside_sqrt), _ptr(stat_in), stat_dx, _ref(dx), _ref(dg),
                                                      _ref(db), ws.ptr, ws.nbytes, _stream(stream)),
           "scalify_scaled_layernorm_bwd_delayed")


def scalify_scaled_gelu(X: ScaledTensor, Y: ScaledTensor, *, exact_erf=False, stream=None) -> None:
    x, y = _desc(X), _desc(Y)
    _check(lib().scalify_scaled_gelu(_ref(x), int(exact_erf), _ref(y), _stream(stream)), "scalify_scaled_gelu")


def scalify_scaled_gelu_bwd(G: ScaledTensor, X: ScaledTensor, dX: ScaledTensor, *, exact_erf=False, stream=None) -> None:
    g, x, dx = _desc(G), _desc(X), _desc(dX)
    _check(lib().scalify_scaled_gelu_bwd(_ref(g), _ref(x), int(exact_erf), _ref(dx), _stream(stream)),
           "scalify_scaled_gelu_bwd")


def _desc_array(ts: Sequence[ScaledTensor]):
    arr = (scalify_array * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = _desc(t)
    return arr


class AdamTensors:
    """Marshalled descriptor arrays of a fixed parameter list (built once, reused every step)."""

    def __init__(self, grads: Sequence[ScaledTensor], m: Sequence[ScaledTensor], v: Sequence[ScaledTensor],
                 w: Sequence[ScaledTensor]):
        assert len(grads) == len(m) == len(v) == len(w)
        self.n = len(grads)
        self.keep = (list(grads), list(m), list(v), list(w))
        self.g, self.m, self.v, self.w = (_desc_array(grads), _desc_array(m), _desc_array(v), _desc_array(w))


def scalify_scaled_adam_step(tensors: AdamTensors, ws: Workspace, *, lr: float, beta1: float, beta2: float, eps: float,
                             step: int, stream=None) -> None:
    _check(lib().scalify_scaled_adam_step(tensors.n, tensors.g, tensors.m, tensors.v, tensors.w, float(lr),
                                          float(beta1), float(beta2), float(eps), int(step), ws.ptr, ws.nbytes,
                                          _stream(stream)), "scalify_scaled_adam_step")


def scalify_scaled_adam_step_cast(tensors: AdamTensors, w_cast: Sequence[ScaledTensor], ws: Workspace, *, lr: float,
                                  beta1: float, beta2: float, eps: float, step: int, stream=None) -> None:
    """Adam step that also writes the low-precision compute copy of every updated weight."""
    assert len(w_cast) == tensors.n
    wc = getattr(tensors, "_wc_cache", None)
    if wc is None or wc[0] is not w_cast:
        wc = (w_cast, _desc_array(w_cast))
        tensors._wc_cache = wc
    _check(lib().scalify_scaled_adam_step_cast(tensors.n, tensors.g, tensors.m, tensors.v, tensors.w, wc[1],
                                               float(lr), float(beta1), float(beta2), float(eps), int(step), ws.ptr,
                                               ws.nbytes, _stream(stream)), "scalify_scaled_adam_step_cast")


def scalify_scaled_adam_step_static(tensors: AdamTensors, *, lr: float, beta1: float, beta2: float, eps: float,
                                    step: int, status_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """Adam step for callers that cannot allocate a workspace (their memory pool already owns the device,
    or they must not trigger cudaMalloc's synchronisation): the scratch is a fixed array inside the library.
    At most 1024 tensors.  `status_out`: optional 1-element int32/uint32 CUDA tensor that receives the device
    status bits.  Calls on one device share that array: do not let two of them overlap on the GPU, and make
    the first call on a device outside stream capture."""
    _check(lib().scalify_scaled_adam_step_static(tensors.n, tensors.g, tensors.m, tensors.v, tensors.w, float(lr),
                                                 float(beta1), float(beta2), float(eps), int(step),
                                                 _ptr(status_out), _stream(stream)),
           "scalify_scaled_adam_step_static")


def scalify_scaled_embedding(ids: torch.Tensor, seq_len: int, wte: ScaledTensor, wpe: Optional[ScaledTensor],
                             Y: ScaledTensor, *, status: Optional[torch.Tensor] = None, stream=None) -> None:
    assert ids.dtype == torch.int64 and ids.is_contiguous()
    a, b, y = _desc(wte), _desc(wpe), _desc(Y)
    _check(lib().scalify_scaled_embedding(ids.data_ptr(), ids.numel(), int(seq_len), _ref(a), _ref(b), _ref(y),
                                          _ptr(status), _stream(stream)), "scalify_scaled_embedding")


def scalify_scaled_embedding_bwd(ids: torch.Tensor, seq_len: int, dY: ScaledTensor, dwte: ScaledTensor,
                                 dwpe: Optional[ScaledTensor], *, stream=None) -> None:
    assert ids.dtype == torch.int64 and ids.is_contiguous()
    g, a, b = _desc(dY), _desc(dwte), _desc(dwpe)
    _check(lib().scalify_scaled_embedding_bwd(ids.data_ptr(), ids.numel(), int(seq_len), _ref(g), _ref(a), _ref(b),
                                              _stream(stream)), "scalify_scaled_embedding_bwd")


def scalify_scaled_softmax(S: ScaledTensor, P: ScaledTensor, *, causal=False, stream=None) -> None:
    s, p = _desc(S), _desc(P)
    _check(lib().scalify_scaled_softmax(_ref(s), int(causal), _ref(p), _stream(stream)), "scalify_scaled_softmax")


def scalify_scaled_softmax_bwd(dP: ScaledTensor, P: ScaledTensor, dS: ScaledTensor, *, stream=None) -> None:
    g, p, o = _desc(dP), _desc(P), _desc(dS)
    _check(lib().scalify_scaled_softmax_bwd(_ref(g), _ref(p), _ref(o), _stream(stream)), "scalify_scaled_softmax_bwd")


def scalify_scaled_cross_entropy(logits: ScaledTensor, n_classes: int, targets: torch.Tensor, loss: torch.Tensor,
                                 dlogits: Optional[ScaledTensor], ws: Workspace, *, stream=None) -> None:
    assert targets.dtype == torch.int64 and targets.is_contiguous() and loss.dtype == torch.float32
    l, g = _desc(logits), _desc(dlogits)
    _check(lib().scalify_scaled_cross_entropy(_ref(l), int(n_classes), targets.data_ptr(), loss.data_ptr(), _ref(g),
                                              ws.ptr, ws.nbytes, _stream(stream)), "scalify_scaled_cross_entropy")


def scalify_scalar_mul_pow2(X: ScaledTensor, c: float, *, stream=None) -> None:
    x = _desc(X)
    _check(lib().scalify_scalar_mul_pow2(_ref(x), float(c), _stream(stream)), "scalify_scalar_mul_pow2")


def scalify_debug_expire_wait(ws: Workspace, limit_us: int, waited_us: Optional[torch.Tensor] = None, *, stream=None) -> None:
    _check(lib().scalify_debug_expire_wait(ws.ptr, ws.nbytes, int(limit_us), _ptr(waited_us), _stream(stream)),
           "scalify_debug_expire_wait")


def scalify_debug_bf16_round(x: torch.Tensor, y: torch.Tensor, two_wide: bool = False, stream=None) -> None:
    """y = x rounded to the nearest BF16 value (as fp32) by the routine the attention kernels use (scalar form,
    or the two-wide form that takes the elements in pairs)."""
    assert x.dtype == y.dtype == torch.float32 and x.is_contiguous() and y.is_contiguous() and x.numel() == y.numel()
    _check(lib().scalify_debug_bf16_round(x.data_ptr(), y.data_ptr(), x.numel(), int(bool(two_wide)), _stream(stream)),
           "scalify_debug_bf16_round")


def scalify_debug_bounds_report(reset_ranges: bool = False, range_limit: int = -1) -> dict:
    """Bounds-checking build only: accesses refused since the last report (and where the first one was)."""
    out = (ctypes.c_uint64 * 3)()
    _check(lib().scalify_debug_bounds_report(ctypes.cast(out, ctypes.c_void_p), int(bool(reset_ranges)), int(range_limit)),
           "scalify_debug_bounds_report")
    return dict(violations=int(out[0]), first_address=int(out[1]), first_bytes=int(out[2]))


def scalify_debug_tensor_map_cache() -> dict:
    """Encodes saved (hits) and made (misses) by the library's tensor-map cache in this process."""
    h, m = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _check(lib().scalify_debug_tensor_map_cache(ctypes.byref(h), ctypes.byref(m)), "scalify_debug_tensor_map_cache")
    return dict(hits=int(h.value), misses=int(m.value))


def scalify_debug_layernorm_plan(R: int, d: int, x_dtype: int, backward: bool) -> dict:
    """Launch shape of the LayerNorm kernels for an [R, d] input (host only, launches nothing)."""
    out = (ctypes.c_int32 * 4)()
    _check(lib().scalify_debug_layernorm_plan(int(R), int(d), int(x_dtype), int(bool(backward)),
                                              ctypes.cast(out, ctypes.c_void_p)), "scalify_debug_layernorm_plan")
    return dict(grid=out[0], rows_per_team=out[1], team_warps=out[2], stages=out[3])


class MxTensor:
    """Block-scaled array: FP8 data [rows, K], E8M0 exponents per 32 elements of K in the tile order the
    tensor cores consume (see ``include/scalify.h``), and the tensor-wide fp32 power-of-two scale."""

    def __init__(self, rows: int, K: int, dtype: torch.dtype = torch.float8_e4m3fn, device="cuda", transposed=False):
        """transposed: the data are stored [K, rows] (blocks of 32 run down the columns); rows % 16 == 0."""
        assert dtype in (torch.float8_e4m3fn, torch.float8_e5m2) and K % 128 == 0 and rows >= 1
        assert not transposed or rows % 16 == 0
        self.rows, self.K, self.transposed = int(rows), int(K), bool(transposed)
        self.data = torch.empty((K, rows) if transposed else (rows, K), dtype=dtype, device=device)
        self.sf = torch.empty(scalify_mx_sf_bytes(rows, K), dtype=torch.uint8, device=device)
        self.scale = torch.ones(1, dtype=torch.float32, device=device)
        self._d = scalify_mx_array(self.data.data_ptr(), _DTYPE_CODE[dtype], self.rows, self.K, self.sf.data_ptr(),
                                   self.scale.data_ptr(), int(self.transposed))

    def scale_value(self) -> float:
        return float(self.scale.item())

    def exponents(self) -> torch.Tensor:
        """The E8M0 codes as a plain [rows, K/32] uint8 tensor (un-tiled copy, for inspection)."""
        kb = self.K // 32
        pr = (self.rows + 255) // 256 * 256
        t = self.sf.view(pr // 128, self.K // 128, 32, 4, 4)          # [row tile, k tile, row % 32, row / 32, blk]
        t = t.permute(0, 3, 2, 1, 4).reshape(pr, kb)                   # row = tile*128 + (row/32)*32 + row%32
        return t[: self.rows].contiguous()

    def set_exponents(self, codes: torch.Tensor, pad: int = 127) -> None:
        """Fill the tiled exponent buffer from plain [rows, K/32] codes (padding rows get `pad`)."""
        kb = self.K // 32
        pr = (self.rows + 255) // 256 * 256
        full = torch.full((pr, kb), pad, dtype=torch.uint8, device=self.sf.device)
        full[: self.rows] = codes.to(self.sf.device)
        t = full.view(pr // 128, 4, 32, self.K // 128, 4).permute(0, 3, 2, 1, 4).contiguous()
        self.sf.copy_(t.view(-1))


def scalify_mx_sf_bytes(rows: int, K: int) -> int:
    return int(lib().scalify_mx_sf_bytes(int(rows), int(K)))


def scalify_mx_quantize(X: ScaledTensor, Y: MxTensor, *, status: Optional[torch.Tensor] = None, stream=None) -> None:
    x = _desc(X)
    _check(lib().scalify_mx_quantize(_ref(x), ctypes.addressof(Y._d), _ptr(status), _stream(stream)),
           "scalify_mx_quantize")


def scalify_mx_matmul(A: MxTensor, B: MxTensor, Y: ScaledTensor, ws: Workspace, *, stat: int = STAT_NONE,
                      stream=None) -> None:
    y = _desc(Y)
    _check(lib().scalify_mx_matmul(ctypes.addressof(A._d), ctypes.addressof(B._d), _ref(y), int(stat), ws.ptr,
                                   ws.nbytes, _stream(stream)), "scalify_mx_matmul")


def scalify_scaled_attention(Q: ScaledTensor, K: ScaledTensor, V: ScaledTensor, O: ScaledTensor, *, sm_scale: float,
                             causal: bool = True, S_dump: Optional[ScaledTensor] = None,
                             P_dump: Optional[ScaledTensor] = None, status: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    """Fused attention forward over [heads, T, hd] FP8 views (hd = 64 or 128); S_dump / P_dump are optional debug copies."""
    q, k, v, o, sd, pd = _desc(Q), _desc(K), _desc(V), _desc(O), _desc(S_dump), _desc(P_dump)
    _check(lib().scalify_scaled_attention(_ref(q), _ref(k), _ref(v), float(sm_scale), int(bool(causal)), _ref(o),
                                          _ref(sd), _ref(pd), _ptr(status), _stream(stream)),
           "scalify_scaled_attention")


def scalify_scaled_cast_colsum(X: ScaledTensor, C: ScaledTensor, Y: ScaledTensor, ws: Workspace, stream=None) -> None:
    """C = static cast of X to FP8, Y = column sums of C (the bias gradient), in one pass over X."""
    x, c, y = _desc(X), _desc(C), _desc(Y)
    _check(lib().scalify_scaled_cast_colsum(_ref(x), _ref(c), _ref(y), ws.ptr, ws.nbytes, _stream(stream)),
           "scalify_scaled_cast_colsum")


def scalify_scaled_colsum(X: ScaledTensor, Y: ScaledTensor, ws: Workspace, stream=None) -> None:
    """Column sums of a [R, N] matrix into a wide [N] vector (bias gradient): Y_s = X_s kf(R)."""
    x, y = _desc(X), _desc(Y)
    _check(lib().scalify_scaled_colsum(_ref(x), _ref(y), ws.ptr, ws.nbytes, _stream(stream)), "scalify_scaled_colsum")


def scalify_scaled_attention_bwd(Q: ScaledTensor, K: ScaledTensor, V: ScaledTensor, P: ScaledTensor, dO: ScaledTensor,
                                 dS: ScaledTensor, dQ: ScaledTensor, dK: ScaledTensor, dV: ScaledTensor, *,
                                 sm_scale: float, causal: bool = True, dP_dump: Optional[ScaledTensor] = None,
                                 status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Fused attention backward: P is the forward's P_dump, dS (E5M2, dense [heads, Tq, Tk]) an output."""
    q, k, v, pp, do = _desc(Q), _desc(K), _desc(V), _desc(P), _desc(dO)
    ds, dq, dk, dv, dpd = _desc(dS), _desc(dQ), _desc(dK), _desc(dV), _desc(dP_dump)
    _check(lib().scalify_scaled_attention_bwd(_ref(q), _ref(k), _ref(v), _ref(pp), _ref(do), float(sm_scale),
                                              int(bool(causal)), _ref(ds), _ref(dq), _ref(dk), _ref(dv), _ref(dpd),
                                              _ptr(status), _stream(stream)),
           "scalify_scaled_attention_bwd")
