"""CPU-side checks of the C ABI: the shared library builds, loads and exports
every function the public header declares; argument validation rejects bad
calls on the host before anything is enqueued (no GPU needed: a call that
fails validation launches nothing)."""
import ctypes
import os
import re

import paper_2407_17353_b200 as sc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "scalify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(scalify_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    L = sc.lib()
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(L, n), n
    assert L.scalify_version() >= 100


def test_bounds_checking_build_exports_the_same_functions():
    """libscalify_debug.so (-DSCALIFY_DEBUG) is a drop-in for the ordinary library; the ordinary one answers the
    checker's report call with 'not supported'."""
    import ctypes
    from paper_2407_17353_b200 import _build
    D = ctypes.CDLL(_build.build(debug=True))
    for n in declared_functions():
        assert hasattr(D, n), n
    assert D.scalify_version() == sc.lib().scalify_version()
    if os.environ.get("SCALIFY_DEBUG_BUILD", "") != "1":
        sc.lib().scalify_debug_bounds_report.restype = ctypes.c_int
        assert sc.lib().scalify_debug_bounds_report(None, 0, -1) == -6


def test_status_strings_and_workspace_sizes():
    L = sc.lib()
    assert L.scalify_status_string(0) == b"ok"
    for code in range(-9, 0):
        assert len(L.scalify_status_string(code)) > 3
    for op in range(7):
        assert sc.scalify_workspace_bytes(op, 8192, 8192) >= 4096
    assert sc.scalify_workspace_bytes(sc.OP_ADAM, 1000) >= 1000 * 32


def _arr(ptr, dtype, shape, stride=None, scale=None):
    a = sc.scalify_array()
    a.data = ptr
    a.dtype = dtype
    a.ndim = len(shape)
    st = stride
    if st is None:
        st, n = [], 1
        for s in reversed(shape):
            st.insert(0, n)
            n *= s
    for i, (s, t) in enumerate(zip(shape, st)):
        a.shape[i] = s
        a.stride[i] = t
    a.scale = scale
    return a


def test_validation_rejects_bad_arguments_on_the_host():
    L = sc.lib()
    R = ctypes.byref
    good = _arr(4096, sc.BF16, (4, 64))
    out = _arr(8192, sc.BF16, (4, 64))
    assert L.scalify_scaled_add(None, R(good), 0, R(out), None) == -1                      # NULL
    assert L.scalify_scaled_add(R(_arr(0, sc.BF16, (4, 64))), R(good), 0, R(out), None) == -1
    assert L.scalify_scaled_add(R(_arr(4096, 9, (4, 64))), R(good), 0, R(out), None) == -2  # dtype
    assert L.scalify_scaled_add(R(_arr(4096, sc.E4M3, (4, 64))), R(_arr(4096, sc.E4M3, (4, 64))), 0, R(out), None) == -2
    assert L.scalify_scaled_add(R(good), R(_arr(4096, sc.BF16, (4, 32))), 0, R(out), None) == -3  # shape
    assert L.scalify_scaled_add(R(_arr(4098, sc.BF16, (4, 64))), R(good), 0, R(out), None) == -4  # alignment
    assert L.scalify_scaled_add(R(_arr(4096, sc.BF16, (4, 64), (64, 2))), R(good), 0, R(out), None) == -4
    assert L.scalify_scaled_add(R(_arr(4096, sc.BF16, (4, 64), scale=512)), R(good), 0,
                                R(_arr(8192, sc.BF16, (4, 64), scale=512)), None) == -8           # alias
    # matmul: dtype, shape and workspace checks
    A = _arr(4096, sc.E4M3, (128, 64))
    B = _arr(65536, sc.E4M3, (64, 256))
    Y = _arr(1 << 20, sc.BF16, (128, 256))
    assert L.scalify_scaled_matmul(R(A), 0, R(B), 0, R(Y), 0, None, None, 0, None) == -5          # workspace
    assert L.scalify_scaled_matmul(R(good), 0, R(B), 0, R(Y), 0, None, 1 << 21, 1 << 20, None) == -2
    assert L.scalify_scaled_matmul(R(A), 0, R(_arr(65536, sc.E4M3, (32, 256))), 0, R(Y), 0, None, 1 << 21, 1 << 20,
                                   None) == -3
    assert L.scalify_scaled_matmul(R(A), 0, R(B), 0, R(Y), 7, None, 1 << 21, 1 << 20, None) == -9
    Yq = _arr(1 << 22, sc.E4M3, (128, 256))
    assert L.scalify_scaled_matmul(R(A), 0, R(B), 0, R(Y), 0, R(Yq), 1 << 21, 1 << 20, None) == -9  # Yq needs a statistic
    # rescale argument combinations
    X = _arr(4096, sc.BF16, (256,))
    Z = _arr(8192, sc.E4M3, (256,))
    assert L.scalify_rescale(R(X), sc.STAT_AMAX, 64, None, R(Z), None, 0, None) == -9
    assert L.scalify_rescale(R(X), sc.STAT_AMAX, None, None, R(Z), None, 0, None) == -5
    assert L.scalify_rescale(R(X), sc.STAT_NONE, None, None, R(_arr(4096, sc.E4M3, (256,))), None, 0, None) == -8
    # adam scalar ranges
    assert L.scalify_scaled_adam_step(1, R(X), R(X), R(X), R(X), 1e-3, 1.5, 0.9, 1e-8, 1, 1 << 21, 1 << 20, None) == -9
    assert L.scalify_scaled_adam_step(1, R(X), R(X), R(X), R(X), 1e-3, 0.9, 0.9, 1e-8, 0, 1 << 21, 1 << 20, None) == -9
    assert L.scalify_scaled_adam_step(0, None, None, None, None, 1e-3, 0.9, 0.9, 1e-8, 1, None, 0, None) == 0
    # layernorm row length must be a multiple of 16 bytes
    assert L.scalify_scaled_layernorm(R(_arr(4096, sc.BF16, (4, 60), (64, 1))), None, None, 1e-5, 0,
                                      R(_arr(8192, sc.BF16, (4, 60), (64, 1))), None, None, None) == -3
    # layernorm backward: the plain call keeps a wide gradient, the delayed one needs the earlier statistic
    Xl = _arr(4096, sc.BF16, (4, 64))
    dX8 = _arr(1 << 20, sc.E5M2, (4, 64))
    assert L.scalify_scaled_layernorm_bwd(R(Xl), R(Xl), None, 64, 128, 1e-5, 0, sc.STAT_L2, R(dX8), None, None, None,
                                          1 << 21, 1 << 20, None) == -2
    assert L.scalify_scaled_layernorm_bwd_delayed(R(Xl), R(Xl), None, 64, 128, 1e-5, 0, None, sc.STAT_L2, R(dX8), None,
                                                  None, 1 << 21, 1 << 20, None) == -1
    assert L.scalify_scaled_layernorm_bwd_delayed(R(Xl), R(Xl), None, 64, 128, 1e-5, 0, 256, 7, R(dX8), None,
                                                  None, 1 << 21, 1 << 20, None) == -9
    # attention: head dimension, power-of-two scalar, batch views, required scale word of dS
    Q3 = _arr(4096, sc.E4M3, (2, 128, 64))
    O3 = _arr(1 << 20, sc.BF16, (2, 128, 64))
    assert L.scalify_scaled_attention(R(Q3), R(Q3), R(Q3), 0.125, 1, R(_arr(1 << 20, sc.BF16, (2, 128, 32))), None, None,
                                      None, None) == -3                                      # shapes differ
    Q32 = _arr(4096, sc.E4M3, (2, 128, 32))
    assert L.scalify_scaled_attention(R(Q32), R(Q32), R(Q32), 0.125, 1, R(_arr(1 << 20, sc.BF16, (2, 128, 32))), None,
                                      None, None, None) == -6                                # head dimension 32
    Q4 = _arr(4096, sc.E4M3, (3, 2, 128, 64))
    assert L.scalify_scaled_attention(R(Q4), R(Q4), R(Q4), 0.125, 1, R(O3), None, None, None, None) == -3  # batch mismatch
    P = _arr(1 << 21, sc.E4M3, (2, 128, 128))
    dS = _arr(1 << 22, sc.E5M2, (2, 128, 128), scale=1024)
    g = [_arr((3 + i) << 20, sc.BF16, (2, 128, 64)) for i in range(3)]
    args = lambda c, ds: (R(Q3), R(Q3), R(Q3), R(P), R(Q3), c, 1, R(ds), R(g[0]), R(g[1]), R(g[2]), None, None, None)
    assert L.scalify_scaled_attention_bwd(*args(0.1, dS)) == -6                              # scalar not a power of two
    assert L.scalify_scaled_attention_bwd(*args(0.125, _arr(1 << 22, sc.E5M2, (2, 128, 128)))) == -1   # dS without a scale
    assert L.scalify_scaled_attention_bwd(*args(0.125, _arr(1 << 22, sc.E4M3, (2, 128, 128), scale=1024))) == -2
    # column sums
    Xc = _arr(4096, sc.E5M2, (64, 128))
    assert L.scalify_scaled_colsum(R(Xc), R(_arr(1 << 20, sc.BF16, (64,))), 1 << 21, 1 << 22, None) == -3
    assert L.scalify_scaled_colsum(R(Xc), R(_arr(1 << 20, sc.E4M3, (128,))), 1 << 21, 1 << 22, None) == -2
    assert L.scalify_scaled_colsum(R(Xc), R(_arr(1 << 20, sc.BF16, (128,))), 1 << 21, 1024, None) == -5
    # matmul does not take four-dimensional arrays
    A4 = _arr(4096, sc.E4M3, (1, 1, 128, 64))
    assert L.scalify_scaled_matmul(R(A4), 0, R(A4), 1, R(_arr(1 << 20, sc.BF16, (1, 1, 128, 128))), 0, None, 1 << 21,
                                   1 << 20, None) == -3
    # matmul with a bias: the vector is required, wide and of length N
    Yb = _arr(1 << 20, sc.BF16, (128, 256))
    assert L.scalify_scaled_matmul_bias(R(A), 0, R(B), 0, None, R(Yb), 0, None, 1 << 21, 1 << 20, None) == -1
    assert L.scalify_scaled_matmul_bias(R(A), 0, R(B), 0, R(_arr(1 << 22, sc.BF16, (128,))), R(Yb), 0, None, 1 << 21,
                                        1 << 20, None) == -3
    assert L.scalify_scaled_matmul_bias(R(A), 0, R(B), 0, R(_arr(1 << 22, sc.E4M3, (256,))), R(Yb), 0, None, 1 << 21,
                                        1 << 20, None) == -2


def test_per_device_set_up_and_tensor_map_cache_selftest():
    """Host-side state: every kernel's one-time set-up is kept per device (a second GPU in the same process gets
    its own), and encoded tensor maps are cached by pointer / extents / strides / box.  The library's self-test
    drives both with made-up device numbers and a stand-in encoder; 0 means every check held."""
    assert sc.lib().scalify_debug_host_state_selftest() == 0
    c = sc.scalify_debug_tensor_map_cache()
    assert c["hits"] >= 0 and c["misses"] >= 0
