"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.

c1-c3 are compared element by element with the oracle.  c4 and the c5 sweep are too large for that, so
the GPU computes everything and the oracle recomputes (i) sampled query rows -- first, last and the rows
around 128-row tile edges -- of a few (batch, head) slices (each output row depends only on its own query
and the keys/values of its slice), and (ii) one whole slice where that takes seconds.  The issued-MAC
census is checked bit-exactly at every size.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2
TOL_F32 = 1e-4


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _census(B, H, n, D, d, scheme):
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    assert got["qk_macs"] == B * H * t.issued_mac1 and got["pv_macs"] == B * H * t.issued_mac3
    assert got["useful_qk_macs"] == B * H * t.useful_mac1 and got["useful_pv_macs"] == B * H * t.useful_mac3
    assert got == binding.psa_skip_count(B, H, n, D, d, scheme, binding.BF16)
    return got


def test_c1_full():
    w = inputs.make("c1")
    v, u = w["values"], w["upload"]
    out = binding.psa_attention_f32(*[torch.from_numpy(u[k]).cuda() for k in ("X", "Wq", "Wk", "Wv")], 1, binding.MASKED)
    ref, cnt = oracle.attention_layer(v["X"], v["Wq"], v["Wk"], v["Wv"], 1, oracle.MASKED)
    assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= TOL_F32
    st, got = binding.psa_last_issued()
    assert st == binding.OK and (got["qk_macs"], got["pv_macs"]) == (cnt.mac1, cnt.mac3)


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_projection_workloads_full(name):
    w = inputs.make(name)
    v, u = w["values"], w["upload"]
    out = binding.psa_attention(_dev_bf16(u["X"]), _dev_bf16(u["Wq"]), _dev_bf16(u["Wk"]), _dev_bf16(u["Wv"]),
                                w["heads"], w["scheme"])
    ref, _ = oracle.attention_layer(v["X"], v["Wq"], v["Wk"], v["Wv"], w["heads"], w["scheme"])
    err = np.abs(_f64(out) - ref).max()
    assert err <= TOL_BF16, err
    _census(w["batch"], w["heads"], w["n"], w["d_model"], w["d_k"], w["scheme"])


@pytest.mark.parametrize("name", ["c2-block", "c3-block"])
def test_block_workloads_full(name):
    # the layer workloads followed by the output projection, every output element; tolerance of z: the layer's 2e-2
    # plus the rounding of z itself to bf16 (at most 2^-8 |z|)
    w = inputs.make(name)
    v, u = w["values"], w["upload"]
    out = binding.psa_attention_block(_dev_bf16(u["X"]), _dev_bf16(u["Wq"]), _dev_bf16(u["Wk"]), _dev_bf16(u["Wv"]),
                                      _dev_bf16(u["Wo"]), w["heads"], w["scheme"])
    ref, _, _ = oracle.attention_block(v["X"], v["Wq"], v["Wk"], v["Wv"], v["Wo"], w["heads"], w["scheme"])
    excess = (np.abs(_f64(out) - ref) - 2.0 ** -8 * np.abs(ref)).max()
    assert excess <= TOL_BF16, excess
    st, got = binding.psa_last_issued()
    B, H, n, D, d = w["batch"], w["heads"], w["n"], w["d_model"], w["d_k"]
    assert st == binding.OK and got["proj_macs"] == 4 * B * n * D * H * d
    t = oracle.tile_counts(n, d, w["scheme"], 128, 128)
    assert got["qk_macs"] == B * H * t.issued_mac1 and got["pv_macs"] == B * H * t.issued_mac3


def _edge_rows(n):
    rows = {0, 1, 63, 127, 128, 129, 255, 256, n // 2 - 1, n // 2, n - 257, n - 129, n - 128, n - 127, n - 2, n - 1}
    return sorted(r for r in rows if 0 <= r < n)


def _check_core(bits, B, H, n, d, scheme, slices, full_slice):
    """bits: dict of uint16 arrays [B,n,H,d] (Q, and K, V unless symmetric).  Runs the GPU on everything and
    checks sampled rows of `slices` and, if given, all rows of `full_slice` against the oracle."""
    sym = scheme == oracle.SYMMETRIC
    q = _dev_bf16(bits["Q"])
    out = binding.psa_attention_core(q, None if sym else _dev_bf16(bits["K"]), None if sym else _dev_bf16(bits["V"]),
                                     scheme)
    _census(B, H, n, 0, d, scheme)
    out = out.view(B, n, H, d)
    worst = 0.0
    for (b, h) in slices + ([full_slice] if full_slice else []):
        sl = {k: inputs.bf16_bits_to_f64(a[b, :, h, :])[None, :, None, :] for k, a in bits.items()}
        K = sl["Q"] if sym else sl["K"]
        V = sl["Q"] if sym else sl["V"]
        got = _f64(out[b, :, h, :])
        if (b, h) == full_slice:
            ref, _ = oracle.attention_core(sl["Q"], K, V, scheme)
            worst = max(worst, np.abs(got - ref[0]).max())
        else:
            rows = _edge_rows(n)
            ref = oracle.attention_rows(sl["Q"], K, V, scheme, 0, 0, rows)
            worst = max(worst, np.abs(got[rows] - ref).max())
    assert worst <= TOL_BF16, worst
    assert torch.isfinite(out.float()).all()


def test_c4_long_sequence_masked():
    w = inputs.WORKLOADS["c4"]
    B, H, n, d = w["batch"], w["heads"], w["n"], w["d_k"]
    bits = {k: inputs.tensor_bits(w["seed"], t, (B, n, H, d), 1.0) for k, t in (("Q", 4), ("K", 5), ("V", 6))}
    _check_core(bits, B, H, n, d, oracle.MASKED, [(0, 0), (1, 7), (1, 15)], (0, 3))


@pytest.mark.parametrize("n", [256, 1024, 4096, 16384])
def test_c5_sweep_all_schemes(n):
    w = inputs.WORKLOADS["c5-n%d-full" % n]
    B, H, d = w["batch"], w["heads"], w["d_k"]
    bits = {k: inputs.tensor_bits(w["seed"], t, (B, n, H, d), 1.0) for k, t in (("Q", 4), ("K", 5), ("V", 6))}
    full = (B - 1, 5) if n <= 4096 else None
    for scheme in (oracle.FULL, oracle.MASKED):
        _check_core(bits, B, H, n, d, scheme, [(0, 0), (B // 2, 9), (B - 1, 15)], full)
    _check_core({"Q": bits["Q"]}, B, H, n, d, oracle.SYMMETRIC, [(0, 0), (B - 1, 15)], full if n <= 1024 else None)
