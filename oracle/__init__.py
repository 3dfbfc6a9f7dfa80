"""fp64 CPU oracle for the self-attention hot path -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``psa_oracle.c`` (which holds all of the arithmetic and the
citations to the paper's equations).  Nothing in the product package may import this
module; the tests, the smoke check and the benchmark's CPU-baseline leg do.

Array conventions (all float64, C-contiguous):
  X        [batch, n, d_model]
  W*       [d_model, heads*d]         head h owns columns h*d .. (h+1)*d-1
  Q, K, V  [batch, n, heads, d]
  output   [batch, n, heads*d]
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

FULL, SYMMETRIC, MASKED = 0, 1, 2
SEL_MINIMAL, SEL_PAPER = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psa_oracle.c")
_LIB = os.path.join(_HERE, "libpsa_oracle.so")


def build(force: bool = False) -> str:
    """Compile psa_oracle.c with gcc (no fast-math, no FMA contraction: summation order is the source's)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Counts(ctypes.Structure):
    _fields_ = [("mac1", ctypes.c_uint64), ("eac", ctypes.c_uint64),
                ("div", ctypes.c_uint64), ("mac3", ctypes.c_uint64)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}

    @property
    def total(self):
        return int(self.mac1 + self.eac + self.div + self.mac3)


class TileCounts(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint64) for k in
                ("issued_mac1", "issued_mac3", "useful_mac1", "useful_mac3", "tiles1", "tiles3")]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        lg = ctypes.c_long
        L.psa_oracle_project.argtypes = [dp, dp, lg, lg, lg, dp]
        L.psa_oracle_project.restype = ctypes.c_int
        L.psa_oracle_round_bf16.argtypes = [dp, lg]
        L.psa_oracle_round_bf16.restype = None
        L.psa_oracle_slice.argtypes = [dp, dp, dp, lg, lg, lg, lg, lg, ctypes.c_double, ctypes.c_int,
                                       ctypes.c_int, dp, lg, dp, dp, ctypes.POINTER(Counts)]
        L.psa_oracle_slice.restype = ctypes.c_int
        L.psa_oracle_rows.argtypes = [dp, dp, dp, lg, lg, lg, lg, lg, ctypes.c_double, ctypes.c_int,
                                      ctypes.c_int, ctypes.POINTER(lg), lg, dp]
        L.psa_oracle_rows.restype = ctypes.c_int
        L.psa_oracle_tiles.argtypes = [lg, lg, ctypes.c_int, ctypes.c_int, lg, lg,
                                       ctypes.POINTER(TileCounts)]
        L.psa_oracle_tiles.restype = ctypes.c_int
        _lib = L
    return _lib


def _dp(a, offset_elems=0):
    return ctypes.cast(a.ctypes.data + 8 * offset_elems, ctypes.POINTER(ctypes.c_double))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def project(X, W):
    """out[..., c] = sum_k X[..., k] W[k, c]  (Sec. 3.1)."""
    X = _f64(X); W = _f64(W)
    D, N = W.shape
    rows = X.size // D
    out = np.empty(X.shape[:-1] + (N,), dtype=np.float64)
    rc = lib().psa_oracle_project(_dp(X), _dp(W), rows, D, N, _dp(out))
    if rc:
        raise RuntimeError("psa_oracle_project failed: %d" % rc)
    return out


def round_bf16(a):
    """Copy of `a` rounded to the nearest bfloat16 values (ties to even)."""
    out = _f64(a).copy()
    lib().psa_oracle_round_bf16(_dp(out), out.size)
    return out


def attention_slice(Q, K, V, scheme, scale, selection=SEL_MINIMAL, want_weights=False, want_scores=False):
    """One head. Q, K, V: [n, d] views (row stride may exceed d). Returns (Y, counts, W or None, S or None)."""
    n, d = Q.shape
    for a in (Q, K, V):
        assert a.dtype == np.float64 and a.strides[1] == 8 and a.strides[0] % 8 == 0
    Y = np.empty((n, d), dtype=np.float64)
    Wout = np.empty((n, n), dtype=np.float64) if want_weights else None
    Sout = np.empty((n, n), dtype=np.float64) if want_scores else None
    c = Counts()
    rc = lib().psa_oracle_slice(_dp(Q), _dp(K), _dp(V), n, d, Q.strides[0] // 8, K.strides[0] // 8,
                                V.strides[0] // 8, float(scale), int(scheme), int(selection), _dp(Y), d,
                                _dp(Wout) if want_weights else None, _dp(Sout) if want_scores else None,
                                ctypes.byref(c))
    if rc:
        raise RuntimeError("psa_oracle_slice failed: %d" % rc)
    return Y, c, Wout, Sout


def attention_core(Q, K, V, scheme, scale=None, selection=SEL_MINIMAL, slices=None):
    """All (batch, head) slices (or the listed (b, h) pairs). Q,K,V [B,n,H,d] -> out [B,n,H*d], summed Counts.

    Slices not listed are left as NaN in the output."""
    Q = _f64(Q); K = _f64(K); V = _f64(V)
    B, n, H, d = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.full((B, n, H * d), np.nan, dtype=np.float64)
    tot = Counts()
    todo = slices if slices is not None else [(b, h) for b in range(B) for h in range(H)]
    for b, h in todo:
        Y, c, _, _ = attention_slice(Q[b, :, h, :], K[b, :, h, :], V[b, :, h, :], scheme, scale, selection)
        out[b, :, h * d:(h + 1) * d] = Y
        for k, _ in Counts._fields_:
            setattr(tot, k, getattr(tot, k) + getattr(c, k))
    return out, tot


def attention_rows(Q, K, V, scheme, b, h, rows, scale=None, selection=SEL_MINIMAL):
    """Outputs of the listed query rows of slice (b, h): returns [len(rows), d]."""
    B, n, H, d = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    q, k, v = Q[b, :, h, :], K[b, :, h, :], V[b, :, h, :]
    for a in (q, k, v):
        assert a.dtype == np.float64 and a.strides[1] == 8
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    Y = np.empty((len(rows), d), dtype=np.float64)
    rc = lib().psa_oracle_rows(_dp(q), _dp(k), _dp(v), n, d, q.strides[0] // 8, k.strides[0] // 8,
                               v.strides[0] // 8, float(scale), int(scheme), int(selection),
                               rows.ctypes.data_as(ctypes.POINTER(ctypes.c_long)), len(rows), _dp(Y))
    if rc:
        raise RuntimeError("psa_oracle_rows failed: %d" % rc)
    return Y


def attention_layer(X, Wq, Wk, Wv, heads, scheme, scale=None, selection=SEL_MINIMAL, round_qkv_bf16=False,
                    slices=None):
    """Projections (Sec. 3.1) then the three phases per head. SYMMETRIC: q = k = v = X*Wq (Sec. 4.1)."""
    X = _f64(X)
    B, n, D = X.shape
    Q = project(X, Wq)
    d = Q.shape[-1] // heads
    if scheme == SYMMETRIC:
        K = V = Q
    else:
        K = project(X, Wk); V = project(X, Wv)
    if round_qkv_bf16:
        Q = round_bf16(Q); K = Q if scheme == SYMMETRIC else round_bf16(K); V = Q if scheme == SYMMETRIC else round_bf16(V)
    shp = (B, n, heads, d)
    return attention_core(Q.reshape(shp), K.reshape(shp), V.reshape(shp), scheme, scale, selection, slices)


def attention_block(X, Wq, Wk, Wv, Wo, heads, scheme, scale=None, selection=SEL_MINIMAL, round_qkv_bf16=False,
                    round_y_bf16=False, residual=None):
    """The layer followed by the output projection: z = concat_h(y^(h)) * Wo, Wo [heads*d, d_model].

    The paper stops at y (Sec. 3.2) and names the complete model as future work (Sec. 7); this is the
    standard multi-head closing step, written as one more projection of the kind Sec. 3.1 calls a typical
    matrix-vector product.  round_y_bf16 rounds y before the product (a bf16 pipeline stores y in bf16).
    `residual` [B, n, d_model], if given, is added to the product elementwise (the skip connection a transformer
    block wraps around its attention sub-layer; usually X itself): z = residual + concat_h(y^(h)) * Wo.
    Returns (z [B, n, d_model], y [B, n, heads*d], Counts of the three phases)."""
    y, cnt = attention_layer(X, Wq, Wk, Wv, heads, scheme, scale, selection, round_qkv_bf16)
    if round_y_bf16:
        y = round_bf16(y)
    z = project(y, Wo)
    if residual is not None:
        z = z + _f64(residual).reshape(z.shape)
    return z, y, cnt


def tile_counts(n, d, scheme, bm, bn, selection=SEL_MINIMAL):
    t = TileCounts()
    rc = lib().psa_oracle_tiles(n, d, int(scheme), int(selection), bm, bn, ctypes.byref(t))
    if rc:
        raise RuntimeError("psa_oracle_tiles failed: %d" % rc)
    return t
