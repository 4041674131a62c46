"""ctypes front end of the CPU oracle (``elsa_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg import this module.  It holds argument marshalling
only; every step of the method is in the C file, which cites the passage of the
paper (ELSA, arXiv 2409.09708) each function follows.  Nothing here imports the
CUDA package, and the CUDA package never imports this.

Arrays are numpy; 16-bit floats travel as their raw ``uint16`` bit patterns so
that fp16 and bf16 are handled by the same exact decoder in C.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

F16 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "elsa_oracle.c")
_LIB = os.path.join(_HERE, "libelsa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, IEEE arithmetic, OpenMP over rows)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-Wno-div-by-zero", _SRC, "-o", _LIB + ".tmp", "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        u32p = ctypes.POINTER(ctypes.c_uint32)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        f64p = ctypes.POINTER(ctypes.c_double)
        i = ctypes.c_int
        lib.oracle_nm_values_per_row.restype = ctypes.c_size_t
        lib.oracle_nm_values_per_row.argtypes = [i, i, i]
        lib.oracle_nm_index_words_per_row.restype = ctypes.c_size_t
        lib.oracle_nm_index_words_per_row.argtypes = [i, i, i]
        lib.oracle_nm_mask.restype = i
        lib.oracle_nm_mask.argtypes = [u16p, i, i, i, i, u8p]
        lib.oracle_nm_pack.restype = i
        lib.oracle_nm_pack.argtypes = [u16p, u8p, i, i, i, i, u16p, u32p]
        lib.oracle_nm_unpack.restype = i
        lib.oracle_nm_unpack.argtypes = [u16p, u32p, i, i, i, i, u16p]
        lib.oracle_linear_f64.restype = i
        lib.oracle_linear_f64.argtypes = [u16p, i, u16p, u16p, i, i, i, f64p]
        lib.oracle_best_mask_bruteforce.restype = ctypes.c_double
        lib.oracle_best_mask_bruteforce.argtypes = [u16p, i, i, i, u8p]
        lib.oracle_linear_macs.restype = ctypes.c_double
        lib.oracle_linear_macs.argtypes = [ctypes.c_double] * 3 + [i, i]
        _lib = lib
    return _lib


def _ptr(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype)) if a is not None else None


def _u16(a, shape=None):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("16-bit floats are passed as uint16 bit patterns, got %s" % a.dtype)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (shape, a.shape))
    return a


def _check(rc, what):
    if rc != 0:
        raise ValueError("oracle %s rejected its arguments (code %d)" % (what, rc))


def values_per_row(in_, N, M):
    return int(_load().oracle_nm_values_per_row(in_, N, M))


def index_words_per_row(in_, N, M):
    return int(_load().oracle_nm_index_words_per_row(in_, N, M))


def nm_mask(W, N, M):
    """uint8 [out, in] keep-mask of W (uint16 bit patterns, [out, in])."""
    W = _u16(W)
    out, in_ = W.shape
    mask = np.empty((out, in_), np.uint8)
    _check(_load().oracle_nm_mask(_ptr(W, ctypes.c_uint16), out, in_, N, M,
                                  _ptr(mask, ctypes.c_uint8)), "nm_mask")
    return mask


def nm_pack(W, mask, N, M):
    """(vals uint16 [out, in/M*N], idx uint32 [out, words_per_row]) from W and its mask."""
    W = _u16(W)
    out, in_ = W.shape
    mask = np.ascontiguousarray(mask, np.uint8)
    vals = np.empty((out, values_per_row(in_, N, M)), np.uint16)
    idx = np.empty((out, index_words_per_row(in_, N, M)), np.uint32)
    _check(_load().oracle_nm_pack(_ptr(W, ctypes.c_uint16), _ptr(mask, ctypes.c_uint8),
                                  out, in_, N, M, _ptr(vals, ctypes.c_uint16),
                                  _ptr(idx, ctypes.c_uint32) if idx.size else None), "nm_pack")
    return vals, idx


def nm_compress(W, N, M):
    """mask followed by pack: what the library's compress call must reproduce bit for bit."""
    mask = nm_mask(W, N, M)
    vals, idx = nm_pack(W, mask, N, M)
    return vals, idx, mask


def nm_unpack(vals, idx, out, in_, N, M):
    """Dense masked weight, uint16 [out, in], from the packed form."""
    vals = _u16(vals, (out, values_per_row(in_, N, M)))
    wpr = index_words_per_row(in_, N, M)
    if wpr:
        idx = np.ascontiguousarray(idx, np.uint32)
        if tuple(idx.shape) != (out, wpr):
            raise ValueError("idx shape %s, expected %s" % (idx.shape, (out, wpr)))
    Wm = np.empty((out, in_), np.uint16)
    _check(_load().oracle_nm_unpack(_ptr(vals, ctypes.c_uint16),
                                    _ptr(idx, ctypes.c_uint32) if wpr else None,
                                    out, in_, N, M, _ptr(Wm, ctypes.c_uint16)), "nm_unpack")
    return Wm


def linear_f64(X, Wm, bias, dtype):
    """fp64 Y [rows, out] = X [rows, in] . Wm[out, in]^T + bias; all inputs uint16 patterns."""
    X = _u16(X)
    Wm = _u16(Wm)
    rows, in_ = X.shape
    out = Wm.shape[0]
    if Wm.shape[1] != in_:
        raise ValueError("X and Wm disagree on the input dimension")
    if bias is not None:
        bias = _u16(bias, (out,))
    Y = np.empty((rows, out), np.float64)
    _check(_load().oracle_linear_f64(_ptr(X, ctypes.c_uint16), rows, _ptr(Wm, ctypes.c_uint16),
                                     _ptr(bias, ctypes.c_uint16), out, in_, dtype,
                                     _ptr(Y, ctypes.c_double)), "linear_f64")
    return Y


def nm_linear_f64(X, vals, idx, bias, out, in_, N, M, dtype):
    """unpack followed by the fp64 product: the reference for the library's linear call."""
    return linear_f64(X, nm_unpack(vals, idx, out, in_, N, M), bias, dtype)


def best_mask_bruteforce(group, N, dtype):
    """(mask uint8 [M], kept L1 sum) for one group, by enumeration of all C(M, N) subsets."""
    group = _u16(group)
    M = group.shape[0]
    mask = np.empty(M, np.uint8)
    s = _load().oracle_best_mask_bruteforce(_ptr(group, ctypes.c_uint16), N, M, dtype,
                                            _ptr(mask, ctypes.c_uint8))
    return mask, float(s)


def linear_macs(rows, in_, out, N, M):
    return float(_load().oracle_linear_macs(float(rows), float(in_), float(out), N, M))


def omp_threads():
    """Threads the OpenMP loops will use (what the CPU-baseline leg reports as cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))
