"""ctypes loader for oracle/w4a8_oracle.c (test infrastructure only).

``build()`` compiles the C file with gcc next to itself; ``quantize_act`` and
``linear`` mirror the numpy oracle's signatures on numpy arrays.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w4a8_oracle.c")
_LIB = os.path.join(_HERE, "libw4a8_oracle.so")
_lib = None


def build(force=False):
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.oracle_num_threads.restype = ci
        lib.oracle_quantize_act.argtypes = [vp, ci, ci, ci, vp, vp, vp]
        lib.oracle_quantize_act.restype = None
        lib.oracle_linear.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, vp]
        lib.oracle_linear.restype = None
        _lib = lib
    return _lib


def num_threads():
    return int(_load().oracle_num_threads())


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data


def quantize_act(x_bits, group):
    lib = _load()
    x, xp = _c(x_bits, np.uint16)
    M, K = x.shape
    qa = np.empty((M, K), np.int8)
    sa = np.empty((M,), np.uint16)
    asum = np.empty((M, K // group), np.int32)
    lib.oracle_quantize_act(xp, M, K, group, qa.ctypes.data, sa.ctypes.data, asum.ctypes.data)
    return qa, sa, asum


def linear(qa, sa_bits, qw, sw_bits, z, group, want_partials=False):
    """Returns (ref fp64 [M,N], D int32 [M,G,N] or None)."""
    lib = _load()
    qa, qap = _c(qa, np.int8)
    sa, sap = _c(sa_bits, np.uint16)
    qw, qwp = _c(qw, np.uint8)
    sw, swp = _c(sw_bits, np.uint16)
    z, zp = _c(z, np.uint8)
    M, K = qa.shape
    N = qw.shape[0]
    G = K // group
    assert qw.shape == (N, K) and sw.shape == (G, N) and z.shape == (G, N) and sa.shape == (M,)
    ref = np.empty((M, N), np.float64)
    D = np.empty((M, G, N), np.int32) if want_partials else None
    lib.oracle_linear(qap, sap, qwp, swp, zp, M, N, K, group, ref.ctypes.data,
                      D.ctypes.data if D is not None else None)
    return ref, D


def w4a8_linear(x_bits, qw, sw_bits, z, group, want_partials=False):
    qa, sa, asum = quantize_act(x_bits, group)
    ref, D = linear(qa, sa, qw, sw_bits, z, group, want_partials)
    return dict(qa=qa, sa=sa, asum=asum, D=D, ref=ref)
