"""fp32 CUDA-core path against the oracle: values within 1e-4, operation census bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_F32 = 1e-4   # max |gpu - oracle|, fp32 storage and arithmetic (dot products of <= 128 terms, |values| ~ 1)


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _check_counts(cnt_oracle, batch_heads_proj):
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    assert got["qk_macs"] == cnt_oracle.mac1
    assert got["pv_macs"] == cnt_oracle.mac3
    assert got["exps"] == cnt_oracle.eac
    assert got["proj_macs"] == batch_heads_proj
    return got


def test_config1_single_head_causal_n64():
    w = inputs.make("c1")
    v, u = w["values"], w["upload"]
    out = binding.psa_attention_f32(_dev(u["X"]), _dev(u["Wq"]), _dev(u["Wk"]), _dev(u["Wv"]), 1, binding.MASKED)
    ref, cnt = oracle.attention_layer(v["X"], v["Wq"], v["Wk"], v["Wv"], 1, oracle.MASKED)
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= TOL_F32, err
    got = _check_counts(cnt, 3 * 64 * 64 * 64)
    assert got["qk_macs"] == 64 * 64 * 65 // 2          # paper Sec. 5.2: d * n(n+1)/2
    assert got == dict(binding.psa_skip_count(1, 1, 64, 64, 64, binding.MASKED, binding.F32))


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.SYMMETRIC, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 1, 8, 4), (2, 3, 37, 50, 20), (1, 2, 200, 64, 128), (1, 1, 1024, 32, 64)])
def test_layer_shapes_and_schemes(scheme, B, H, n, D, d):
    rng = np.random.default_rng(n + d)
    X = (rng.standard_normal((B, n, D)) * 0.5).astype(np.float32)
    Ws = [(rng.standard_normal((D, H * d)) / np.sqrt(D)).astype(np.float32) for _ in range(3)]
    sym = scheme == oracle.SYMMETRIC
    out = binding.psa_attention_f32(_dev(X), _dev(Ws[0]), None if sym else _dev(Ws[1]), None if sym else _dev(Ws[2]),
                                    H, scheme)
    ref, cnt = oracle.attention_layer(X, Ws[0], Ws[1], Ws[2], H, scheme)
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= TOL_F32, err
    _check_counts(cnt, (1 if sym else 3) * B * n * D * H * d)


# Small layers run as one launch; with at most 32 heads the FULL and MASKED schemes spread a head over a cluster of
# 1, 2, 4 or 8 CTAs (the largest power of two that leaves every CTA a 4-row tile).  The shapes walk those cluster sizes,
# ragged last tiles, the switch back to one CTA per head at 33 heads, and d_k at both ends of the range.
@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 3, 16, 8), (1, 1, 8, 16, 8), (1, 2, 13, 24, 4), (2, 2, 17, 40, 12),
                                       (1, 1, 31, 64, 64), (1, 3, 33, 20, 128), (4, 8, 64, 64, 32), (3, 11, 45, 32, 16),
                                       (1, 1, 130, 48, 64), (1, 1, 256, 32, 32)])
def test_small_layers_on_clusters(scheme, B, H, n, D, d):
    rng = np.random.default_rng(1000 * n + d + B)
    X = (rng.standard_normal((B, n, D)) * 0.5).astype(np.float32)
    Ws = [(rng.standard_normal((D, H * d)) / np.sqrt(D)).astype(np.float32) for _ in range(3)]
    ref, cnt = oracle.attention_layer(X, Ws[0], Ws[1], Ws[2], H, scheme)
    dev = [_dev(X)] + [_dev(w) for w in Ws]
    for call in range(3):       # the two counter blocks of the workspace are used in turn: every call starts from zero
        out = binding.psa_attention_f32(dev[0], dev[1], dev[2], dev[3], H, scheme)
        err = np.abs(out.cpu().numpy().astype(np.float64) - ref).max()
        assert err <= TOL_F32, (call, err)
        _check_counts(cnt, 3 * B * n * D * H * d)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.SYMMETRIC, oracle.MASKED])
def test_core_entry(scheme):
    rng = np.random.default_rng(5)
    B, n, H, d = 2, 70, 2, 24
    Q, K, V = (rng.standard_normal((B, n, H, d)).astype(np.float32) for _ in range(3))
    if scheme == oracle.SYMMETRIC:
        out = binding.psa_attention_core(_dev(Q), None, None, scheme)
        ref, cnt = oracle.attention_core(Q, Q, Q, scheme)
    else:
        out = binding.psa_attention_core(_dev(Q), _dev(K), _dev(V), scheme)
        ref, cnt = oracle.attention_core(Q, K, V, scheme)
    assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= TOL_F32
    _check_counts(cnt, 0)


def test_host_entry_matches_device_entry():
    w = inputs.make("c1")
    u = w["upload"]
    host = [torch.from_numpy(u[k]) for k in ("X", "Wq", "Wk", "Wv")]
    out_h = torch.empty((1, 64, 64), dtype=torch.float32)
    binding.psa_attention_host(*host, 1, binding.MASKED, out_h)
    out_d = binding.psa_attention_f32(*[t.cuda() for t in host], 1, binding.MASKED)
    assert torch.equal(out_h, out_d.cpu())
