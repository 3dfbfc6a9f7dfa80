"""ctypes binding of libpsa.so: one Python function per C entry point of include/psa.h, same names.

Only argument marshalling happens here (tensor -> pointer, sizes, stream handle); every step of
the computation runs inside the library's CUDA kernels.  PyTorch provides device memory and
streams.  There is no fallback: if the shared library is missing, importing a symbol fails with
an explicit error.
"""
from __future__ import annotations

import ctypes
import os

import torch

FULL, SYMMETRIC, MASKED = 0, 1, 2
F32, BF16 = 0, 1
OK = 0
ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGN, ERR_SCHEME_ARGS, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NUMERIC = range(1, 10)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpsa.so")

EXPORTS = ("psa_attention", "psa_attention_f32", "psa_attention_core", "psa_attention_host", "psa_skip_count",
           "psa_last_issued", "psa_workspace_bytes", "psa_set_workspace", "psa_status_string",
           "psa_last_cuda_error", "psa_profile_begin", "psa_profile_end", "psa_attention_sym_f32_noalloc",
           "psa_attention_block", "psa_block_workspace_bytes", "psa_last_rescales", "psa_selftest_wait_expiry", "psa_measure_pipe_rates", "psa_attention_core_host", "psa_attention_block_residual")


class PsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = psa_last_cuda_error() if status == ERR_CUDA else ""
        super().__init__("%s failed: %s (status %d)%s" % (where, psa_status_string(status), status,
                                                          (": " + detail) if detail else ""))


class Counts(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint64) for k in
                ("proj_macs", "qk_macs", "pv_macs", "exps", "useful_qk_macs", "useful_pv_macs")]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class PipeRates(ctypes.Structure):
    _fields_ = [("ex2_per_clk_per_sm", ctypes.c_double), ("fma_per_clk_per_sm", ctypes.c_double),
                ("softmax_weights_per_clk_per_sm", ctypes.c_double), ("sm_count", ctypes.c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C library.  Raises if it has not been built (python -m paper_2012_01114_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libpsa.so is missing at %s: build it with `python -m paper_2012_01114_b200.build`; "
                               "there is no fallback path" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.psa_attention.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_attention_f32.argtypes = L.psa_attention.argtypes
        L.psa_attention_core.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_attention_host.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_skip_count.argtypes = [ci, ci, ci, ci, ci, ci, ci, ctypes.POINTER(Counts)]
        L.psa_last_issued.argtypes = [vp, ctypes.POINTER(Counts)]
        L.psa_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci, ci]
        L.psa_workspace_bytes.restype = ctypes.c_size_t
        L.psa_set_workspace.argtypes = [vp, ctypes.c_size_t]
        L.psa_status_string.argtypes = [ci]
        L.psa_status_string.restype = ctypes.c_char_p
        L.psa_last_cuda_error.argtypes = []
        L.psa_last_cuda_error.restype = ctypes.c_char_p
        L.psa_profile_begin.argtypes = [ci]
        L.psa_profile_begin.restype = ci
        L.psa_profile_end.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                      ctypes.POINTER(ci)]
        L.psa_profile_end.restype = ci
        L.psa_attention_block.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_attention_block.restype = ci
        L.psa_attention_block_residual.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_attention_block_residual.restype = ci
        L.psa_block_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci]
        L.psa_block_workspace_bytes.restype = ctypes.c_size_t
        L.psa_attention_core_host.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
        L.psa_attention_core_host.restype = ci
        L.psa_measure_pipe_rates.argtypes = [ctypes.POINTER(PipeRates), vp]
        L.psa_measure_pipe_rates.restype = ci
        L.psa_selftest_wait_expiry.argtypes = [ctypes.c_uint, vp]
        L.psa_selftest_wait_expiry.restype = ci
        L.psa_last_rescales.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
        L.psa_last_rescales.restype = ci
        L.psa_attention_sym_f32_noalloc.argtypes = [vp, ci, ci, ci, ci, vp, vp]
        L.psa_attention_sym_f32_noalloc.restype = ci
        for f in ("psa_attention", "psa_attention_f32", "psa_attention_core", "psa_attention_host",
                  "psa_skip_count", "psa_last_issued", "psa_set_workspace"):
            getattr(L, f).restype = ci
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check_dev(t, dtype, name):
    if t is None:
        return
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))


def psa_status_string(status: int) -> str:
    return lib().psa_status_string(int(status)).decode()


def psa_last_cuda_error() -> str:
    return lib().psa_last_cuda_error().decode()


def _layer(fn_name, dtype, X, Wq, Wk, Wv, heads, scheme, out, stream):
    for t, nm in ((X, "X"), (Wq, "Wq"), (Wk, "Wk"), (Wv, "Wv"), (out, "out")):
        _check_dev(t, dtype, nm)
    batch, n, d_model = X.shape
    hd = Wq.shape[1]
    if Wq.shape[0] != d_model or hd % heads:
        raise ValueError("Wq must be [d_model, heads*d_k]")
    d_k = hd // heads
    if out is None:
        out = torch.empty((batch, n, hd), dtype=dtype, device=X.device)
    rc = getattr(lib(), fn_name)(_ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), batch, heads, n, d_model, d_k, int(scheme),
                                 _ptr(out), _stream(stream))
    if rc != OK:
        raise PsaError(rc, fn_name)
    return out


def psa_attention(X, Wq, Wk, Wv, heads, scheme, out=None, stream=None):
    """bf16 projections + attention.  X [B,n,D], W* [D,heads*d_k] -> out [B,n,heads*d_k] (all bf16, CUDA)."""
    return _layer("psa_attention", torch.bfloat16, X, Wq, Wk, Wv, heads, scheme, out, stream)


def psa_attention_f32(X, Wq, Wk, Wv, heads, scheme, out=None, stream=None):
    """fp32 projections + attention on CUDA cores with element-exact skipping."""
    return _layer("psa_attention_f32", torch.float32, X, Wq, Wk, Wv, heads, scheme, out, stream)


def psa_attention_core(Q, K, V, scheme, out=None, stream=None):
    """Attention core with q, k, v given: Q,K,V [B,n,H,d] (bf16 or fp32) -> out [B,n,H*d]."""
    dtype = Q.dtype
    code = {torch.bfloat16: BF16, torch.float32: F32}[dtype]
    for t, nm in ((Q, "Q"), (K, "K"), (V, "V"), (out, "out")):
        _check_dev(t, dtype, nm)
    B, n, H, d = Q.shape
    if out is None:
        out = torch.empty((B, n, H * d), dtype=dtype, device=Q.device)
    rc = lib().psa_attention_core(_ptr(Q), _ptr(K), _ptr(V), B, H, n, d, int(scheme), code, _ptr(out),
                                  _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_attention_core")
    return out


def psa_attention_host(X, Wq, Wk, Wv, heads, scheme, out, stream=None):
    """The whole layer from HOST tensors (CPU, contiguous; pinned or not) into the host tensor `out`."""
    dtype = X.dtype
    code = {torch.bfloat16: BF16, torch.float32: F32}[dtype]
    for t in (X, Wq, Wk, Wv, out):
        if t is not None and (t.is_cuda or t.dtype != dtype or not t.is_contiguous()):
            raise ValueError("host tensors must be contiguous CPU tensors of one dtype")
    batch, n, d_model = X.shape
    d_k = Wq.shape[1] // heads
    rc = lib().psa_attention_host(_ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), batch, heads, n, d_model, d_k, int(scheme),
                                  code, _ptr(out), _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_attention_host")
    return out


def psa_attention_core_host(Q, K, V, scheme, out, stream=None):
    """The attention core from HOST tensors Q, K, V [B,n,H,d] (CPU, contiguous; K = V = None for the symmetric
    scheme) into the host tensor `out` [B,n,H*d]."""
    dtype = Q.dtype
    code = {torch.bfloat16: BF16, torch.float32: F32}[dtype]
    for t in (Q, K, V, out):
        if t is not None and (t.is_cuda or t.dtype != dtype or not t.is_contiguous()):
            raise ValueError("host tensors must be contiguous CPU tensors of one dtype")
    B, n, H, d = Q.shape
    rc = lib().psa_attention_core_host(_ptr(Q), _ptr(K), _ptr(V), B, H, n, d, int(scheme), code, _ptr(out),
                                       _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_attention_core_host")
    return out


def psa_skip_count(batch, heads, n, d_model, d_k, scheme, dtype) -> dict:
    """Analytic census of what a call would issue (host only).  d_model = 0: core only."""
    c = Counts()
    rc = lib().psa_skip_count(batch, heads, n, d_model, d_k, int(scheme), int(dtype), ctypes.byref(c))
    if rc != OK:
        raise PsaError(rc, "psa_skip_count")
    return c.as_dict()


def psa_last_issued(stream=None):
    """(device status, measured census) of the last call; waits for the stream."""
    c = Counts()
    rc = lib().psa_last_issued(_stream(stream), ctypes.byref(c))
    if rc not in (OK, ERR_TIMEOUT):
        raise PsaError(rc, "psa_last_issued")
    return rc, c.as_dict()


def psa_measure_pipe_rates(stream=None) -> dict:
    """Measured ex2 / fma / softmax-mix results per SM clock per SM (see include/psa.h)."""
    r = PipeRates()
    rc = lib().psa_measure_pipe_rates(ctypes.byref(r), _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_measure_pipe_rates")
    return {k: getattr(r, k) for k, _ in r._fields_}


def psa_selftest_wait_expiry(limit_us: int = 1000, stream=None):
    """Queues the miniature kernel whose bounded wait expires; psa_last_issued() then reports ERR_TIMEOUT."""
    rc = lib().psa_selftest_wait_expiry(int(limit_us), _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_selftest_wait_expiry")


def psa_last_rescales(stream=None) -> int:
    """How often the last call raised a row's running softmax maximum after the row's first key block."""
    v = ctypes.c_uint64()
    rc = lib().psa_last_rescales(_stream(stream), ctypes.byref(v))
    if rc != OK:
        raise PsaError(rc, "psa_last_rescales")
    return int(v.value)


def psa_attention_block(X, Wq, Wk, Wv, Wo, heads, scheme, out=None, stream=None, residual=None):
    """Projections + attention + output projection (+ residual).  X [B,n,D], W* [D,heads*d_k], Wo [heads*d_k,D],
    residual [B,n,D] or None -> out [B,n,D] (all bf16 or all fp32, CUDA)."""
    dtype = X.dtype
    code = {torch.bfloat16: BF16, torch.float32: F32}[dtype]
    for t, nm in ((X, "X"), (Wq, "Wq"), (Wk, "Wk"), (Wv, "Wv"), (Wo, "Wo"), (out, "out"), (residual, "residual")):
        _check_dev(t, dtype, nm)
    batch, n, d_model = X.shape
    hd = Wq.shape[1]
    if Wq.shape[0] != d_model or hd % heads or Wo is None or tuple(Wo.shape) != (hd, d_model):
        raise ValueError("Wq must be [d_model, heads*d_k] and Wo [heads*d_k, d_model]")
    if out is None:
        out = torch.empty((batch, n, d_model), dtype=dtype, device=X.device)
    if residual is not None and tuple(residual.shape) != (batch, n, d_model):
        raise ValueError("residual must be [batch, n, d_model]")
    if residual is None:
        rc = lib().psa_attention_block(_ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(Wo), batch, heads, n, d_model,
                                       hd // heads, int(scheme), code, _ptr(out), _stream(stream))
    else:
        rc = lib().psa_attention_block_residual(_ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(Wo), _ptr(residual),
                                                batch, heads, n, d_model, hd // heads, int(scheme), code, _ptr(out),
                                                _stream(stream))
    if rc != OK:
        raise PsaError(rc, "psa_attention_block")
    return out


def psa_block_workspace_bytes(batch, heads, n, d_model, d_k, scheme, dtype) -> int:
    return int(lib().psa_block_workspace_bytes(batch, heads, n, d_model, d_k, int(scheme), int(dtype)))


def psa_workspace_bytes(batch, heads, n, d_model, d_k, scheme, dtype, with_host_staging=False) -> int:
    return int(lib().psa_workspace_bytes(batch, heads, n, d_model, d_k, int(scheme), int(dtype),
                                         1 if with_host_staging else 0))


_ws_keepalive = None


def psa_set_workspace(tensor):
    """Registers a CUDA uint8 tensor as the workspace (None: back to the library's own)."""
    global _ws_keepalive
    if tensor is None:
        rc = lib().psa_set_workspace(None, 0)
    else:
        rc = lib().psa_set_workspace(_ptr(tensor), tensor.numel() * tensor.element_size())
    if rc != OK:
        raise PsaError(rc, "psa_set_workspace")
    _ws_keepalive = tensor


def psa_profile_begin(max_calls: int):
    rc = lib().psa_profile_begin(int(max_calls))
    if rc != OK:
        raise PsaError(rc, "psa_profile_begin")


def psa_profile_end():
    """(projection ms summed, attention ms summed, calls recorded) since psa_profile_begin."""
    p, a, c = ctypes.c_float(), ctypes.c_float(), ctypes.c_int()
    rc = lib().psa_profile_end(ctypes.byref(p), ctypes.byref(a), ctypes.byref(c))
    if rc != OK:
        raise PsaError(rc, "psa_profile_end")
    return p.value, a.value, c.value


def psa_attention_sym_f32_noalloc(X, out=None, stream=None):
    """Symmetric-scheme fp32 attention core (query = key = value = X [B,n,H,d]) that allocates nothing:
    its scratch is a fixed array inside the library, for callers that may not call cudaMalloc at run
    time.  Problems with B*H*n*n above the built-in limit raise PsaError(ERR_WORKSPACE).  Pass `out`
    to keep this wrapper allocation-free too."""
    _check_dev(X, torch.float32, "X")
    _check_dev(out, torch.float32, "out")
    B, n, H, d = X.shape
    if out is None:
        out = torch.empty((B, n, H * d), dtype=torch.float32, device=X.device)
    rc = lib().psa_attention_sym_f32_noalloc(_ptr(X), B, H, n, d, _ptr(out), _stream(stream))
    if rc != OK:
        detail = psa_last_cuda_error()
        err = PsaError(rc, "psa_attention_sym_f32_noalloc")
        if detail and rc == ERR_WORKSPACE:
            err.args = (err.args[0] + ": " + detail,)
        raise err
    return out
