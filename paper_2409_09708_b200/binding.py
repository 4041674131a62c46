"""Thin ctypes binding of ``libelsa.so`` (the C ABI declared in ``include/elsa.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and streams.  There is no fallback: if
the library has not been built this module raises at import.

Functions carry the names of the C entry points.  Tensors must be CUDA,
contiguous, fp16 or bf16 (index words are int32 tensors holding the uint32
bit patterns).
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libelsa.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libelsa.so is missing: build it with `python -m paper_2409_09708_b200.build` "
        "(there is no CPU or PyTorch fallback for the sparse-linear path)")

_lib = ctypes.CDLL(LIB_PATH)

OK = 0
ERR_NAMES = {0: "ELSA_OK", 1: "ELSA_ERR_NULL", 2: "ELSA_ERR_SHAPE", 3: "ELSA_ERR_NM", 4: "ELSA_ERR_DTYPE",
             5: "ELSA_ERR_ALIGN", 6: "ELSA_ERR_WORKSPACE", 7: "ELSA_ERR_CUDA", 8: "ELSA_ERR_TIMEOUT",
             9: "ELSA_ERR_ARCH"}
F16, BF16 = 0, 1
VARIANT_AUTO, VARIANT_SIMT, VARIANT_TC_DENSE, VARIANT_TC_PAIR, VARIANT_TC_SPARSE, VARIANT_TC_SPARSE_PAIR = 0, 1, 2, 3, 4, 5
VARIANT_TC_SPARSE_WS = 6
VARIANT_TC_SPARSE_ST = 7

_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t


class ElsaLayer(ctypes.Structure):
    _fields_ = [("X", _vp), ("Y", _vp), ("vals", _vp), ("idx", _vp), ("bias", _vp),
                ("rows", _i), ("in_", _i), ("out", _i), ("N", _i), ("M", _i)]


class ElsaWeight(ctypes.Structure):
    _fields_ = [("W", _vp), ("vals", _vp), ("idx", _vp), ("out", _i), ("in_", _i), ("N", _i), ("M", _i)]


class ElsaHostLayer(ctypes.Structure):
    _fields_ = [("X", _vp), ("Y", _vp), ("W", _vp), ("bias", _vp),
                ("rows", _i), ("in_", _i), ("out", _i), ("N", _i), ("M", _i)]


def _sig(name, restype, argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = argtypes
    return fn


_values_bytes = _sig("elsa_nm_values_bytes", _sz, [_i, _i, _i, _i, _i])
_index_bytes = _sig("elsa_nm_index_bytes", _sz, [_i, _i, _i, _i])
_workspace_bytes = _sig("elsa_workspace_bytes", _sz, [_i, _i, _i, _i, _i, _i])
_compress = _sig("elsa_nm_compress", _i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _vp])
_unpack = _sig("elsa_nm_unpack", _i, [_vp, _vp, _i, _i, _i, _i, _i, _vp, _vp])
_linear = _sig("elsa_nm_linear", _i, [_vp, _i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _sz, _vp, _vp])
_linear_static = _sig("elsa_nm_linear_static", _i, [_vp, _i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp])
STATIC_SCRATCH_BYTES = 8 << 20
_compress_levels = _sig("elsa_nm_compress_levels", _i, [_vp, _i, _i, _i, ctypes.POINTER(_i), _i, _i,
                                                        ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp])
_linear_masked = _sig("elsa_nm_linear_masked", _i, [_vp, _i, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _sz, _vp, _vp])
_vit_compress = _sig("elsa_vit_compress", _i, [ctypes.POINTER(ElsaWeight), _i, _i, _vp])
_vit_ws = _sig("elsa_vit_workspace_bytes", _sz, [ctypes.POINTER(ElsaLayer), _i, _i])
_vit = _sig("elsa_vit_linears", _i, [ctypes.POINTER(ElsaLayer), _i, _i, _vp, _sz, _vp, _vp])
_vit_host_bytes = _sig("elsa_vit_host_device_bytes", _sz, [ctypes.POINTER(ElsaHostLayer), _i, _i])
_vit_host = _sig("elsa_vit_linears_host", _i, [ctypes.POINTER(ElsaHostLayer), _i, _i, _vp, _sz, _vp, _vp])
_set_variant = _sig("elsa_set_linear_variant", _i, [_i])
_set_grouping = _sig("elsa_set_grouping", None, [_i])
_get_variant = _sig("elsa_get_linear_variant", _i, [])
_launch_count = _sig("elsa_launch_count", ctypes.c_ulonglong, [])
_last_error = _sig("elsa_last_error", ctypes.c_char_p, [])
_values_bytes_i8 = _sig("elsa_nm_values_bytes_i8", _sz, [_i, _i, _i, _i])
_workspace_bytes_i8 = _sig("elsa_workspace_bytes_i8", _sz, [_i, _i, _i, _i])
_compress_i8 = _sig("elsa_nm_compress_i8", _i, [_vp, _i, _i, _i, _i, _vp, _vp, _vp])
_unpack_i8 = _sig("elsa_nm_unpack_i8", _i, [_vp, _vp, _i, _i, _i, _i, _vp, _vp])
_linear_i8 = _sig("elsa_nm_linear_i8", _i, [_vp, _i, ctypes.c_float, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _sz, _vp, _vp])


class ElsaLinearShape(ctypes.Structure):
    _fields_ = [("rows", _i), ("in_", _i), ("out", _i)]


class ElsaLevel(ctypes.Structure):
    _fields_ = [("N", _i), ("M", _i)]


_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(_i)
_cost_table = _sig("elsa_cost_table_macs", _i, [ctypes.POINTER(ElsaLinearShape), _i, ctypes.POINTER(ElsaLevel), _i, _dp])
_config_cost = _sig("elsa_config_cost", ctypes.c_double, [_dp, _i, _i, _ip, ctypes.c_double])
_two_step = _sig("elsa_two_step_sample", _i, [_dp, _i, _i, _dp, ctypes.c_double, ctypes.c_double, _i, ctypes.c_double, _dp, _ip, _ip])
_interval_masses = _sig("elsa_interval_masses", _i, [_dp, _i, _i, _dp, ctypes.c_double, ctypes.c_double, _i, ctypes.c_double, _dp])
_space_size = _sig("elsa_search_space_size", _i, [_i, _i, ctypes.c_char_p, _sz])
_config_from_index = _sig("elsa_config_from_index", _i, [ctypes.c_char_p, _i, _i, _ip])
_selftest_wait = _sig("elsa_selftest_wait_timeout", _i, [ctypes.c_ulonglong, _vp, _vp])


class ElsaBlockLinear(ctypes.Structure):
    _fields_ = [("vals", _vp), ("idx", _vp), ("bias", _vp), ("N", _i), ("M", _i)]


class ElsaBlockWeights(ctypes.Structure):
    _fields_ = [("ln1_gain", _vp), ("ln1_bias", _vp), ("ln2_gain", _vp), ("ln2_bias", _vp),
                ("qkv", ElsaBlockLinear), ("proj", ElsaBlockLinear), ("fc1", ElsaBlockLinear), ("fc2", ElsaBlockLinear),
                ("eps", ctypes.c_float)]


_backward_ws = _sig("elsa_backward_workspace_bytes", _sz, [_i, _i, _i, _i, _i, _i])
_backward = _sig("elsa_nm_linear_backward", _i, [_vp, _vp, _i, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _sz, _vp, _vp])
BLOCK_REGIONS = ("x1", "qkv", "a", "x2", "x3", "h", "t", "workspace")
_bw = ctypes.POINTER(ElsaBlockWeights)
_block_scratch = _sig("elsa_vit_block_scratch_bytes", _sz, [_i, _i, _i, _bw, _i, ctypes.POINTER(_sz)])
_block_qkv = _sig("elsa_vit_block_qkv", _i, [_vp, _i, _i, _i, _bw, _i, _vp, _sz, _vp, _vp])
_block_rest = _sig("elsa_vit_block_rest", _i, [_vp, _i, _i, _i, _bw, _i, _vp, _vp, _sz, _vp, _vp])
_block = _sig("elsa_vit_block", _i, [_vp, _i, _i, _i, _bw, _i, _vp, _vp, _sz, _vp, _vp])
_block_attn = _sig("elsa_vit_block_attn", _i, [_vp, _i, _i, _i, _i, _i, _bw, _i, _vp, _vp, _sz, _vp, _vp])
_attention = _sig("elsa_attention", _i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _vp])
_window_attention = _sig("elsa_window_attention", _i, [_vp, _i, _i, _i, _i, _vp, _i, _vp, _i, _i, _vp, _vp, _vp])
class ElsaSwinAttn(ctypes.Structure):
    _fields_ = [("H", _i), ("W", _i), ("window", _i), ("shift", _i), ("rel_bias", _vp), ("mask", _vp), ("bias_pitch", _i),
                ("pack", _i)]


_fp = ctypes.POINTER(ctypes.c_float)
_swin_mask = _sig("elsa_swin_mask", _i, [_i, _i, _i, _i, _i, _i, _fp])
_swin_pack_bias = _sig("elsa_swin_pack_bias", _i, [_fp, _i, _i, _i, _i, _fp])
_swin_block = _sig("elsa_swin_block", _i, [_vp, _i, _i, _i, _i, _bw, ctypes.POINTER(ElsaSwinAttn), _i, _vp, _vp, _sz, _vp, _vp])
_encoder_scratch = _sig("elsa_vit_encoder_scratch_bytes", _sz, [_i, _i, _i, _i, _bw, _i, _i])
_encoder = _sig("elsa_vit_encoder", _i, [_vp, _i, _i, _i, _i, _i, _bw, _i, _vp, _vp, ctypes.c_float, _i, _vp, _vp, _sz, _vp, _vp])


class ElsaKernelTime(ctypes.Structure):
    _fields_ = [("kernel", _i), ("layer", _i), ("ms", ctypes.c_float)]


KERNEL_NAMES = {0: "nm_compress", 1: "nm_unpack", 2: "linear_simt", 3: "linear_tc_dense", 4: "linear_tc_pair", 5: "nm_to_sp24", 6: "linear_tc_sp24", 7: "linear_tc_sp24_pair", 8: "weight_images",
                9: "linear_tc_sp24_ws", 10: "linear_tc_sp24_st", 11: "linear_tc_pair_i8", 12: "int8_format", 13: "block_rowwise", 14: "backward_format", 15: "attention"}
_profile_start = _sig("elsa_profile_start", _i, [])
_profile_stop = _sig("elsa_profile_stop", _i, [ctypes.POINTER(ElsaKernelTime), _i])


class ElsaError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__("%s: %s" % (ERR_NAMES.get(status, status), elsa_last_error()))


def _check(status: int):
    if status != OK:
        raise ElsaError(status)


def elsa_last_error() -> str:
    return (_last_error() or b"").decode()


# ---- INT8 form (int8 CUDA tensors; index words as int32 tensors)

def elsa_nm_compress_i8(W: torch.Tensor, N: int, M: int, stream=None):
    assert W.dtype == torch.int8 and W.is_cuda and W.is_contiguous()
    out, in_ = W.shape
    vals = torch.empty((out, in_ // M * N), dtype=torch.int8, device=W.device)
    words = elsa_nm_index_bytes(out, in_, N, M) // 4
    idx = torch.empty((out, words // out if out else 0), dtype=torch.int32, device=W.device) if words else None
    _check(_compress_i8(_ptr(W), out, in_, N, M, _ptr(vals), _ptr(idx), _stream(stream)))
    return vals, idx


def elsa_nm_unpack_i8(vals: torch.Tensor, idx, out: int, in_: int, N: int, M: int, stream=None):
    Wm = torch.empty((out, in_), dtype=torch.int8, device=vals.device)
    _check(_unpack_i8(_ptr(vals), _ptr(idx), out, in_, N, M, _ptr(Wm), _stream(stream)))
    return Wm


def elsa_nm_linear_i8(X: torch.Tensor, x_scale: float, vals: torch.Tensor, idx, w_scale: torch.Tensor, bias, out: int,
                      in_: int, N: int, M: int, out_dtype: torch.dtype, dev_status=None, stream=None):
    """Y [rows, out] (out_dtype) from int8 activations, the packed int8 weight and the scales."""
    assert X.dtype == torch.int8 and w_scale.dtype == torch.float32
    rows = X.shape[0]
    Y = torch.empty((rows, out), dtype=out_dtype, device=X.device)
    need = int(_workspace_bytes_i8(out, in_, N, M))
    ws = alloc_workspace(need) if need else None
    _check(_linear_i8(_ptr(X), rows, float(x_scale), _ptr(vals), _ptr(idx), _ptr(w_scale), _ptr(bias), out, in_, N, M,
                      dtype_code(out_dtype), _ptr(Y), _ptr(ws), need, _ptr(dev_status), _stream(stream)))
    return Y


# ---- search-side host code (lists of numbers in, lists out; argument marshalling only)

def _doubles(values):
    flat = [float(v) for v in values]
    return (ctypes.c_double * len(flat))(*flat)


def elsa_cost_table_macs(shapes, levels):
    """shapes: [(rows, in, out)], levels: [(N, M)] -> cost[l][s] as a list of lists."""
    arr = (ElsaLinearShape * len(shapes))(*[ElsaLinearShape(*s) for s in shapes])
    lev = (ElsaLevel * len(levels))(*[ElsaLevel(*s) for s in levels])
    out = (ctypes.c_double * (len(shapes) * len(levels)))()
    _check(_cost_table(arr, len(shapes), lev, len(levels), out))
    k = len(levels)
    return [[out[l * k + s] for s in range(k)] for l in range(len(shapes))]


def elsa_config_cost(cost, choice, fixed_cost=0.0):
    L, k = len(cost), len(cost[0])
    return float(_config_cost(_doubles(v for row in cost for v in row), L, k, (_i * L)(*choice), float(fixed_cost)))


def elsa_two_step_sample(cost, P, fixed_cost, c_upper, n_intervals, quantum, uniforms):
    """Returns (choice, interval)."""
    L, k = len(cost), len(cost[0])
    assert len(uniforms) == L + 1
    choice = (_i * L)()
    interval = _i(-1)
    _check(_two_step(_doubles(v for row in cost for v in row), L, k, _doubles(v for row in P for v in row), float(fixed_cost),
                     float(c_upper), int(n_intervals), float(quantum), _doubles(uniforms), choice, ctypes.byref(interval)))
    return list(choice), int(interval.value)


def elsa_interval_masses(cost, P, fixed_cost, c_upper, n_intervals, quantum):
    L, k = len(cost), len(cost[0])
    mass = (ctypes.c_double * n_intervals)()
    _check(_interval_masses(_doubles(v for row in cost for v in row), L, k, _doubles(v for row in P for v in row), float(fixed_cost),
                            float(c_upper), int(n_intervals), float(quantum), mass))
    return list(mass)


def elsa_search_space_size(n_layers, n_levels) -> int:
    buf = ctypes.create_string_buffer(4096)
    n = _space_size(n_layers, n_levels, buf, len(buf))
    if n < 0:
        raise ElsaError(2)
    return int(buf.value.decode())


def elsa_config_from_index(index: int, n_layers, n_levels):
    choice = (_i * n_layers)()
    _check(_config_from_index(str(int(index)).encode(), n_layers, n_levels, choice))
    return list(choice)


def elsa_selftest_wait_timeout(limit_ns: int, dev_status: torch.Tensor, stream=None):
    """Launches the bounded wait of the tensor-core kernels on a barrier nobody arrives at (test hook)."""
    _check(_selftest_wait(int(limit_ns), _ptr(dev_status), _stream(stream)))


def elsa_launch_count() -> int:
    return int(_launch_count())


def elsa_profile_start():
    _check(_profile_start())


def elsa_profile_stop(capacity: int = 1 << 16):
    """List of (kernel name, layer index, ms) for every launch since elsa_profile_start."""
    buf = (ElsaKernelTime * capacity)()
    n = min(int(_profile_stop(buf, capacity)), capacity)
    return [(KERNEL_NAMES.get(buf[i].kernel, str(buf[i].kernel)), buf[i].layer, float(buf[i].ms)) for i in range(n)]


def elsa_set_linear_variant(v: int):
    _check(_set_variant(v))


def elsa_set_grouping(on: bool):
    _set_grouping(1 if on else 0)


def elsa_get_linear_variant() -> int:
    return int(_get_variant())


def dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.float16:
        return F16
    if dtype == torch.bfloat16:
        return BF16
    raise TypeError("fp16 or bf16 expected, got %s" % dtype)


def _ptr(t):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("contiguous tensor expected")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def elsa_nm_values_bytes(out, in_, N, M, dtype=F16) -> int:
    return int(_values_bytes(out, in_, N, M, dtype))


def elsa_nm_index_bytes(out, in_, N, M) -> int:
    return int(_index_bytes(out, in_, N, M))


def elsa_workspace_bytes(rows, in_, out, N, M, dtype=F16) -> int:
    return int(_workspace_bytes(rows, in_, out, N, M, dtype))


def alloc_packed(out, in_, N, M, dtype: torch.dtype, device="cuda"):
    """Uninitialised (vals, idx) tensors of the packed form; idx is None when N == M."""
    vals = torch.empty((out, in_ // M * N), dtype=dtype, device=device)
    words = elsa_nm_index_bytes(out, in_, N, M) // 4 // out
    idx = torch.empty((out, words), dtype=torch.int32, device=device) if words else None
    return vals, idx


def elsa_nm_compress(W: torch.Tensor, N: int, M: int, vals=None, idx=None, stream=None):
    """Packed (vals, idx) of W [out, in] at level N:M."""
    out, in_ = W.shape
    if vals is None:
        if elsa_nm_values_bytes(out, in_, N, M, dtype_code(W.dtype)) == 0:
            _check(_compress(_ptr(W), out, in_, N, M, dtype_code(W.dtype), None, None, _stream(stream)))
        vals, idx = alloc_packed(out, in_, N, M, W.dtype, W.device)
    _check(_compress(_ptr(W), out, in_, N, M, dtype_code(W.dtype), _ptr(vals), _ptr(idx), _stream(stream)))
    return vals, idx


def elsa_nm_compress_levels(W: torch.Tensor, N_list, M: int, stream=None):
    """Packed (vals, idx) of W at every level N:M of N_list, from one read of W."""
    out, in_ = W.shape
    packed = [alloc_packed(out, in_, N, M, W.dtype, W.device) for N in N_list]
    n = len(N_list)
    Ns = (_i * n)(*N_list)
    vals = (_vp * n)(*[_ptr(v) for v, _ in packed])
    idx = (_vp * n)(*[_ptr(i) for _, i in packed])
    _check(_compress_levels(_ptr(W), out, in_, M, Ns, n, dtype_code(W.dtype), vals, idx, _stream(stream)))
    return packed


def elsa_nm_linear_masked(X: torch.Tensor, W_sup: torch.Tensor, bias, N: int, M: int, Y=None, workspace=None,
                          dev_status=None, stream=None):
    """Y = X . (W_sup projected onto N:M)^T + bias straight from the dense shared weight."""
    rows, in_ = X.shape
    out = W_sup.shape[0]
    code = dtype_code(X.dtype)
    if Y is None:
        Y = torch.empty((rows, out), dtype=X.dtype, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(elsa_workspace_bytes(rows, in_, out, N, M, code), X.device)
    _check(_linear_masked(_ptr(X), rows, _ptr(W_sup), _ptr(bias), out, in_, N, M, code, _ptr(Y), _ptr(workspace),
                          workspace.numel(), _ptr(dev_status), _stream(stream)))
    return Y


def elsa_nm_unpack(vals: torch.Tensor, idx, out: int, in_: int, N: int, M: int, W_masked=None, stream=None):
    if W_masked is None:
        W_masked = torch.empty((out, in_), dtype=vals.dtype, device=vals.device)
    _check(_unpack(_ptr(vals), _ptr(idx), out, in_, N, M, dtype_code(vals.dtype), _ptr(W_masked), _stream(stream)))
    return W_masked


def alloc_workspace(nbytes: int, device="cuda"):
    return torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=device)


def elsa_nm_linear(X: torch.Tensor, vals: torch.Tensor, idx, bias, out: int, in_: int, N: int, M: int,
                   Y=None, workspace=None, dev_status=None, stream=None):
    """Y [rows, out] = X [rows, in] . W_masked^T + bias from the packed weight."""
    rows = X.shape[0]
    code = dtype_code(X.dtype)
    if Y is None:
        Y = torch.empty((rows, out), dtype=X.dtype, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(elsa_workspace_bytes(rows, in_, out, N, M, code), X.device)
    _check(_linear(_ptr(X), rows, _ptr(vals), _ptr(idx), _ptr(bias), out, in_, N, M, code, _ptr(Y),
                   _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(stream)))
    return Y


def elsa_backward_workspace_bytes(rows, in_, out, N, M, dtype=F16) -> int:
    return int(_backward_ws(rows, in_, out, N, M, dtype))


def elsa_nm_linear_backward(dY, X, vals, idx, out, in_, N, M, want=("dX", "dW", "db"), workspace=None,
                            dev_status=None, stream=None):
    """Backward of Y = X Wm^T + b: returns (dX, dW, db), None for the ones not in `want`.  dW is dense [out, in]
    with zeros at the pruned positions."""
    rows = dY.shape[0]
    code = dtype_code(dY.dtype)
    dX = torch.empty((rows, in_), dtype=dY.dtype, device=dY.device) if "dX" in want else None
    dW = torch.empty((out, in_), dtype=dY.dtype, device=dY.device) if "dW" in want else None
    db = torch.empty((out,), dtype=dY.dtype, device=dY.device) if "db" in want else None
    if workspace is None:
        workspace = alloc_workspace(elsa_backward_workspace_bytes(rows, in_, out, N, M, code), dY.device)
    _check(_backward(_ptr(dY), _ptr(X), rows, _ptr(vals), _ptr(idx), out, in_, N, M, code, _ptr(dX), _ptr(dW), _ptr(db),
                     _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(stream)))
    return dX, dW, db


def make_block_weights(ln1_gain, ln1_bias, ln2_gain, ln2_bias, linears, eps=1e-6):
    """linears: dict name -> (vals, idx or None, bias or None, N, M) for qkv, proj, fc1, fc2 (device tensors).
    Returns (ElsaBlockWeights, the tensors it points to)."""
    w = ElsaBlockWeights()
    keep = [ln1_gain, ln1_bias, ln2_gain, ln2_bias]
    w.ln1_gain, w.ln1_bias, w.ln2_gain, w.ln2_bias = (_ptr(t) for t in keep)
    for name in ("qkv", "proj", "fc1", "fc2"):
        vals, idx, bias, N, M = linears[name]
        setattr(w, name, ElsaBlockLinear(_ptr(vals), _ptr(idx), _ptr(bias), N, M))
        keep += [vals, idx, bias]
    w.eps = eps
    return w, keep


def elsa_vit_block_scratch_bytes(rows, dim, mlp_dim, weights, dtype_c):
    """(bytes, {region name: byte offset})."""
    off = (_sz * len(BLOCK_REGIONS))()
    n = _block_scratch(rows, dim, mlp_dim, ctypes.byref(weights), dtype_c, off)
    return n, dict(zip(BLOCK_REGIONS, off))


def elsa_attention(qkv, tokens, heads, a=None, dev_status=None, stream=None):
    """a [rows, dim] = multi-head self-attention of qkv [rows, 3 dim], rows = images * tokens."""
    rows, three_dim = qkv.shape
    dim = three_dim // 3
    if a is None:
        a = torch.empty((rows, dim), dtype=qkv.dtype, device=qkv.device)
    _check(_attention(_ptr(qkv), rows // tokens, tokens, heads, dim, dtype_code(qkv.dtype), _ptr(a), _ptr(dev_status),
                      _stream(stream)))
    return a


def elsa_window_attention(qkv, tokens, heads, bias, mask=None, a=None, dev_status=None, stream=None):
    """Attention over windows of `tokens` consecutive rows of qkv [rows, 3 dim] with fp32 tables on the scores:
    bias [heads, tokens, pitch], mask [n_masks, tokens, pitch] or None (window w takes table w % n_masks)."""
    rows, three_dim = qkv.shape
    dim = three_dim // 3
    if a is None:
        a = torch.empty((rows, dim), dtype=qkv.dtype, device=qkv.device)
    _check(_window_attention(_ptr(qkv), rows // tokens, tokens, heads, dim, _ptr(bias), bias.shape[-1], _ptr(mask),
                             0 if mask is None else mask.shape[0], dtype_code(qkv.dtype), _ptr(a), _ptr(dev_status), _stream(stream)))
    return a


def pad_score_table(t):
    """fp32 table [..., T, T] with its rows padded to whole float4s, as the attention kernel reads them."""
    T = t.shape[-1]
    pitch = (T + 3) // 4 * 4
    out = torch.zeros(t.shape[:-1] + (pitch,), dtype=torch.float32, device=t.device)
    out[..., :T] = t
    return out


def elsa_swin_mask(H, W, window, shift, pitch=None, pack=1):
    """The seam mask of shifted windows as a host fp32 tensor [windows / pack, pack window^2, pitch]."""
    T = window * window * pack
    pitch = pitch or (T + 3) // 4 * 4          # rows padded to whole float4s
    n = (H // window) * (W // window) // pack
    out = torch.empty((n, T, pitch), dtype=torch.float32)
    got = _swin_mask(H, W, window, shift, pack, pitch, ctypes.cast(out.data_ptr(), _fp))
    if got != n:
        raise ValueError("elsa_swin_mask rejected its arguments")
    return out


def elsa_swin_pack_bias(rel_bias, window, pack=1, pitch=None):
    """rel_bias: host fp32 [heads, T, T] -> host fp32 [heads, pack T, pitch] (bias on the diagonal blocks, -30000 between
    tokens of different windows)."""
    rel_bias = rel_bias.detach().to(torch.float32).cpu().contiguous()
    heads, T = rel_bias.shape[0], window * window
    pitch = pitch or (pack * T + 3) // 4 * 4
    out = torch.empty((heads, pack * T, pitch), dtype=torch.float32)
    if _swin_pack_bias(ctypes.cast(rel_bias.data_ptr(), _fp), heads, window, pack, pitch, ctypes.cast(out.data_ptr(), _fp)) != 0:
        raise ValueError("elsa_swin_pack_bias rejected its arguments")
    return out


def elsa_swin_block(x, H, W, window, shift, heads, mlp_dim, weights, rel_bias, mask=None, y=None, scratch=None,
                    dev_status=None, stream=None, pack=1):
    """One Swin block over x [images * H * W, dim]; rel_bias [heads, pack T, pitch] and mask [windows / pack, pack T, pitch]
    fp32 on the device, as elsa_swin_pack_bias and elsa_swin_mask build them for `pack` windows per attention item."""
    rows, dim = x.shape
    code = dtype_code(x.dtype)
    if scratch is None:
        scratch = alloc_workspace(elsa_vit_block_scratch_bytes(rows, dim, mlp_dim, weights, code)[0], x.device)
    if y is None:
        y = torch.empty_like(x)
    attn = ElsaSwinAttn(H, W, window, shift, _ptr(rel_bias), _ptr(mask), rel_bias.shape[-1], pack)
    _check(_swin_block(_ptr(x), rows // (H * W), heads, dim, mlp_dim, ctypes.byref(weights), ctypes.byref(attn), code, _ptr(y),
                       _ptr(scratch), scratch.numel(), _ptr(dev_status), _stream(stream)))
    return y, scratch


def elsa_vit_block(x, mlp_dim, weights, y=None, scratch=None, dev_status=None, stream=None, phase="both", tokens=None,
                   heads=None):
    """One pre-norm ViT block over x [rows, dim] with the four linears in their packed N:M forms.  phase "both"
    runs the whole block, with the library's attention when tokens (per image) and heads are given and with the
    stand-in a = V otherwise; "qkv" stops after qkv (regions x1, qkv of scratch); "rest" continues from region a
    of scratch, which the caller's attention has written."""
    rows, dim = x.shape
    code = dtype_code(x.dtype)
    if scratch is None:
        scratch = alloc_workspace(elsa_vit_block_scratch_bytes(rows, dim, mlp_dim, weights, code)[0], x.device)
    if y is None and phase != "qkv":
        y = torch.empty_like(x)
    if phase == "qkv":
        _check(_block_qkv(_ptr(x), rows, dim, mlp_dim, ctypes.byref(weights), code, _ptr(scratch), scratch.numel(),
                          _ptr(dev_status), _stream(stream)))
    elif phase == "both" and tokens:
        _check(_block_attn(_ptr(x), rows // tokens, tokens, heads, dim, mlp_dim, ctypes.byref(weights), code, _ptr(y),
                           _ptr(scratch), scratch.numel(), _ptr(dev_status), _stream(stream)))
    else:
        fn = _block if phase == "both" else _block_rest
        _check(fn(_ptr(x), rows, dim, mlp_dim, ctypes.byref(weights), code, _ptr(y), _ptr(scratch), scratch.numel(),
                  _ptr(dev_status), _stream(stream)))
    return y, scratch


def make_encoder_table(block_weights):
    """ctypes array of ElsaBlockWeights from a list of them (as make_block_weights returns)."""
    return (ElsaBlockWeights * len(block_weights))(*block_weights)


def elsa_vit_encoder(x, tokens, heads, mlp_dim, table, final_gain=None, final_bias=None, final_eps=1e-6, y=None, scratch=None,
                     dev_status=None, stream=None):
    """The encoder: len(table) blocks with attention, each under its own levels, then the optional final LayerNorm."""
    rows, dim = x.shape
    code = dtype_code(x.dtype)
    n = len(table)
    if scratch is None:
        scratch = alloc_workspace(int(_encoder_scratch(rows // tokens, tokens, dim, mlp_dim, table, n, code)), x.device)
    if y is None:
        y = torch.empty_like(x)
    _check(_encoder(_ptr(x), rows // tokens, tokens, heads, dim, mlp_dim, table, n, _ptr(final_gain), _ptr(final_bias),
                    final_eps, code, _ptr(y), _ptr(scratch), scratch.numel(), _ptr(dev_status), _stream(stream)))
    return y, scratch


def block_region(scratch, offsets, name, rows, cols, dtype):
    """View of one region of a block's scratch as a [rows, cols] tensor."""
    return scratch[offsets[name]:offsets[name] + rows * cols * 2].view(dtype).view(rows, cols)


def elsa_nm_linear_static(X: torch.Tensor, vals: torch.Tensor, idx, bias, out: int, in_: int, N: int, M: int,
                          Y: torch.Tensor, dev_status=None, stream=None):
    """elsa_nm_linear without a workspace argument, for callers that cannot allocate: the weight
    image is rebuilt in the library's built-in scratch array (out * in * 2 <= STATIC_SCRATCH_BYTES).
    Y must be supplied by the caller; nothing is allocated here or in the library."""
    _check(_linear_static(_ptr(X), X.shape[0], _ptr(vals), _ptr(idx), _ptr(bias), out, in_, N, M,
                          dtype_code(X.dtype), _ptr(Y), _ptr(dev_status), _stream(stream)))
    return Y


def make_layer_table(layers):
    """ctypes array of elsa_layer from dicts / objects with X, Y, vals, idx, bias, N, M tensors."""
    arr = (ElsaLayer * len(layers))()
    for a, l in zip(arr, layers):
        X, Y = l["X"], l["Y"]
        a.X, a.Y = _ptr(X), _ptr(Y)
        a.vals, a.idx, a.bias = _ptr(l["vals"]), _ptr(l.get("idx")), _ptr(l.get("bias"))
        a.rows, a.in_, a.out = X.shape[0], X.shape[1], Y.shape[1]
        a.N, a.M = l["N"], l["M"]
    return arr


def make_weight_table(layers):
    """ctypes array of elsa_weight from dicts with W, vals, idx tensors and N, M."""
    arr = (ElsaWeight * len(layers))()
    for a, l in zip(arr, layers):
        W = l["W"]
        a.W, a.vals, a.idx = _ptr(W), _ptr(l["vals"]), _ptr(l.get("idx"))
        a.out, a.in_ = W.shape
        a.N, a.M = l["N"], l["M"]
    return arr


def elsa_vit_compress(table, dtype_c: int, stream=None):
    _check(_vit_compress(table, len(table), dtype_c, _stream(stream)))


def elsa_vit_workspace_bytes(table, dtype_c: int) -> int:
    return int(_vit_ws(table, len(table), dtype_c))


def elsa_vit_linears(table, dtype_c: int, workspace, dev_status=None, stream=None):
    _check(_vit(table, len(table), dtype_c, _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(stream)))


def make_host_layer_table(layers):
    """ctypes array of elsa_host_layer from dicts of HOST tensors X, Y, W, bias and N, M."""
    arr = (ElsaHostLayer * len(layers))()
    for a, l in zip(arr, layers):
        X, Y, W = l["X"], l["Y"], l["W"]
        a.X, a.Y, a.W, a.bias = _ptr(X), _ptr(Y), _ptr(W), _ptr(l.get("bias"))
        a.rows, a.in_, a.out = X.shape[0], X.shape[1], W.shape[0]
        a.N, a.M = l["N"], l["M"]
    return arr


def elsa_vit_host_device_bytes(table, dtype_c: int) -> int:
    return int(_vit_host_bytes(table, len(table), dtype_c))


def elsa_vit_linears_host(table, dtype_c: int, device_mem, dev_status=None, stream=None):
    _check(_vit_host(table, len(table), dtype_c, _ptr(device_mem), device_mem.numel(), _ptr(dev_status),
                     _stream(stream)))
