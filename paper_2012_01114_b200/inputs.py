"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds no attention arithmetic: it only draws numbers.  Element k of tensor t
under seed s is a pure function of (s, t, k) (a 64-bit counter mixer feeding a Box-Muller
transform), so any slice of any tensor can be regenerated anywhere, and the CPU oracle and
the GPU library are always handed the very same values.  bf16 tensors are rounded to the
bf16 grid (nearest, ties to even) here, before either side sees them.

The paper uses no dataset (its experiments are SAT instances), so these tensors stand for
nothing but themselves: standard-normal activations and 1/sqrt(d_model)-scaled weights, the
shapes of the five workloads below.
"""
from __future__ import annotations

import numpy as np

FULL, SYMMETRIC, MASKED = 0, 1, 2
SCHEME_NAMES = {FULL: "full", SYMMETRIC: "symmetric", MASKED: "masked"}

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function on a uint64 array (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        x = ((x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        x = ((x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return x ^ (x >> np.uint64(31))


def _normal_chunk(key, lo, hi, out, base):
    k = np.arange(lo, hi, dtype=np.uint64)
    with np.errstate(over="ignore"):
        a = _mix64(key ^ (k * np.uint64(2)))
        b = _mix64(key ^ (k * np.uint64(2) + np.uint64(1)))
    u1 = ((a >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
    u2 = ((b >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
    out[lo - base:hi - base] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def normal(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """`count` standard-normal float64 draws for elements start .. start+count-1 of a tensor.

    Element k depends on (seed, tensor_id, k) only; large requests are drawn in chunks on a thread pool
    (numpy releases the GIL inside its loops), which changes nothing about the values."""
    out = np.empty(count, dtype=np.float64)
    key = _mix64(np.array([np.uint64(seed) * np.uint64(0x100000001B3) + np.uint64(tensor_id)], dtype=np.uint64))[0]
    step = 1 << 20
    spans = [(start + lo, start + min(count, lo + step)) for lo in range(0, count, step)]
    if len(spans) <= 2:
        for lo, hi in spans:
            _normal_chunk(key, lo, hi, out, start)
    else:
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
            list(ex.map(lambda sp: _normal_chunk(key, sp[0], sp[1], out, start), spans))
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float array -> uint16 bfloat16 bit patterns (nearest, ties to even)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> the exact float64 values they denote."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def tensor(seed: int, tensor_id: int, shape, scale: float, dtype: str, row_scale=None):
    """Returns (values, bits): float64 values exactly representable in `dtype`, and for bf16 the
    uint16 bit patterns to upload (for f32, a float32 array to upload).

    `row_scale`, if given, is one extra factor per index of axis 1 (the sequence position of a
    [batch, n, ...] tensor), applied before the rounding to `dtype`: inputs whose magnitude varies
    along the sequence, for instance keys that grow from one 128-key block to the next."""
    count = int(np.prod(shape))
    x = normal(seed, tensor_id, count) * scale
    if row_scale is not None:
        rs = np.asarray(row_scale, dtype=np.float64)
        x = (x.reshape(shape[0], shape[1], -1) * rs[None, :, None]).reshape(-1)
    if dtype == "bf16":
        bits = to_bf16_bits(x).reshape(shape)
        return bf16_bits_to_f64(bits), bits
    if dtype == "f32":
        f = x.astype(np.float32).reshape(shape)
        return f.astype(np.float64), f
    raise ValueError(dtype)


def tensor_bits(seed: int, tensor_id: int, shape, scale: float) -> np.ndarray:
    """bf16 bit patterns only (for tensors too large to also keep as float64); same numbers as `tensor`."""
    count = int(np.prod(shape))
    out = np.empty(count, dtype=np.uint16)
    step = 1 << 24
    for lo in range(0, count, step):
        hi = min(count, lo + step)
        out[lo:hi] = to_bf16_bits(normal(seed, tensor_id, hi - lo, start=lo) * scale)
    return out.reshape(shape)


# The five workloads (shape, number type, scheme, seed).  `proj` says whether X and the three
# projection matrices are the inputs (True) or q, k, v are given directly (False).
WORKLOADS = {
    "c1": dict(batch=1, heads=1, n=64, d_model=64, d_k=64, dtype="f32", scheme=MASKED, proj=True, seed=0,
               x_scale=1.0 / 8.0, w_scale=1.0 / 8.0),
    "c2": dict(batch=8, heads=12, n=512, d_model=768, d_k=64, dtype="bf16", scheme=FULL, proj=True, seed=1,
               x_scale=1.0, w_scale=768 ** -0.5),
    "c3": dict(batch=8, heads=12, n=1024, d_model=768, d_k=64, dtype="bf16", scheme=MASKED, proj=True, seed=2,
               x_scale=1.0, w_scale=768 ** -0.5),
    "c4": dict(batch=2, heads=16, n=8192, d_model=2048, d_k=128, dtype="bf16", scheme=MASKED, proj=False, seed=3,
               x_scale=1.0, w_scale=0.0),
}
# c2 / c3 followed by the output projection over the concatenated heads (Wo [heads*d_k, d_model], tensor id 7)
for _b in ("c2", "c3"):
    WORKLOADS[_b + "-block"] = dict(WORKLOADS[_b], wo=True, wo_scale=768 ** -0.5)
for _n in (256, 1024, 4096, 16384):
    for _s in (FULL, SYMMETRIC, MASKED):
        WORKLOADS["c5-n%d-%s" % (_n, SCHEME_NAMES[_s])] = dict(
            batch=65536 // _n, heads=16, n=_n, d_model=2048, d_k=128, dtype="bf16", scheme=_s, proj=False,
            seed=100 + int(np.log2(_n)), x_scale=1.0, w_scale=0.0)


def make(name: str, batch: int | None = None, **override):
    """Draw the tensors of a workload.  Returns a dict with the meta data, `values` (float64
    arrays for the oracle) and `upload` (arrays in the I/O number type for the device).
    `batch` may shrink the batch (the first `batch` items are the same numbers)."""
    w = dict(WORKLOADS[name]); w.update(override)
    if batch is not None:
        w["batch"] = batch
    B, H, n, D, d = w["batch"], w["heads"], w["n"], w["d_model"], w["d_k"]
    vals, up = {}, {}
    if w["proj"]:
        vals["X"], up["X"] = tensor(w["seed"], 0, (B, n, D), w["x_scale"], w["dtype"])
        ids = {"Wq": 1} if w["scheme"] == SYMMETRIC else {"Wq": 1, "Wk": 2, "Wv": 3}
        for k, t in ids.items():
            vals[k], up[k] = tensor(w["seed"], t, (D, H * d), w["w_scale"], w["dtype"])
        if w.get("wo"):
            vals["Wo"], up["Wo"] = tensor(w["seed"], 7, (H * d, D), w["wo_scale"], w["dtype"])
    else:
        ids = {"Q": 4} if w["scheme"] == SYMMETRIC else {"Q": 4, "K": 5, "V": 6}
        for k, t in ids.items():
            vals[k], up[k] = tensor(w["seed"], t, (B, n, H, d), w["x_scale"], w["dtype"])
    w["name"] = name
    w["values"] = vals
    w["upload"] = up
    return w
