"""Head sizes other than 64 and 128 on the bf16 path.  The kernels work on 64-column boxes: a head of d_k columns
(any multiple of 8 up to 128) is described to TMA as its own axis of the tensor, so the columns between d_k and the
next multiple of 64 are out of bounds -- zero-filled when a tile is loaded, dropped when the output is stored.
Values against the oracle at the path's tolerance; the census counts what the tensor core is issued, which is the
padded width (64 for d_k <= 64, 128 up to 128, 256 above), while the useful counts are the paper's, with d_k itself.
Heads of more than 128 columns (full and masked schemes) run on a kernel of their own, one row tile per CTA."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _census(B, H, n, D, d, scheme):
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    dpad = 64 if d <= 64 else (128 if d <= 128 else 256)
    assert got["qk_macs"] == B * H * t.tiles1 * 128 * 128 * dpad
    assert got["pv_macs"] == B * H * t.tiles3 * 128 * 128 * dpad
    assert got["useful_qk_macs"] == B * H * t.useful_mac1 and got["useful_pv_macs"] == B * H * t.useful_mac3
    assert got == binding.psa_skip_count(B, H, n, D, d, scheme, binding.BF16)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,d", [(1, 2, 256, 32), (2, 3, 384, 96), (1, 1, 300, 8), (2, 2, 640, 120), (1, 4, 129, 72),
                                     (1, 2, 512, 16), (3, 50, 256, 96)])
def test_core_with_other_head_sizes(scheme, B, H, n, d):
    sym = scheme == oracle.SYMMETRIC
    vals, bits = {}, {}
    for k, tid in (("Q", 4), ("K", 5), ("V", 6)):
        vals[k], bits[k] = inputs.tensor(7 * n + d, tid, (B, n, H, d), 1.0, "bf16")
    if sym:
        out = binding.psa_attention_core(_dev(bits["Q"]), None, None, scheme)
        ref, _ = oracle.attention_core(vals["Q"], vals["Q"], vals["Q"], scheme)
    else:
        out = binding.psa_attention_core(_dev(bits["Q"]), _dev(bits["K"]), _dev(bits["V"]), scheme)
        ref, _ = oracle.attention_core(vals["Q"], vals["K"], vals["V"], scheme)
    assert tuple(out.shape) == (B, n, H * d)
    assert np.abs(_f64(out) - ref).max() <= TOL_BF16
    _census(B, H, n, 0, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,D,d", [(2, 2, 256, 128, 32), (1, 2, 384, 192, 96), (2, 8, 200, 64, 8)])
def test_layer_with_other_head_sizes(scheme, B, H, n, D, d):
    sym = scheme == oracle.SYMMETRIC
    Xv, Xb = inputs.tensor(23, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(23, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    out = binding.psa_attention(_dev(Xb), _dev(W[0][1]), None if sym else _dev(W[1][1]), None if sym else _dev(W[2][1]),
                                H, scheme)
    ref, _ = oracle.attention_layer(Xv, W[0][0], W[1][0], W[2][0], H, scheme)
    # elementwise |gpu - oracle| <= 2e-2 + 2^-8 |oracle|: with short heads the softmax of the symmetric scheme is
    # dominated by a row's own score, outputs come close to single value entries of size 2 to 4, and the rounding of
    # the output itself to bf16 (half a unit of its 8 significant bits) is no longer small beside the 2e-2
    excess = (np.abs(_f64(out) - ref) - 2.0 ** -8 * np.abs(ref)).max()
    assert excess <= TOL_BF16, excess
    _census(B, H, n, D, d, scheme)


def test_neighbouring_heads_do_not_leak_into_the_padding():
    # a head's padded columns would, without the out-of-bounds fill, hold the first columns of the next head: make
    # those huge in every head but the one under test and compare with the head computed alone
    B, H, n, d = 1, 3, 256, 96
    qv, qb = inputs.tensor(5, 4, (B, n, H, d), 1.0, "bf16")
    kv, kb = inputs.tensor(5, 5, (B, n, H, d), 1.0, "bf16")
    vv, vb = inputs.tensor(5, 6, (B, n, H, d), 1.0, "bf16")
    q, k, v = _dev(qb), _dev(kb), _dev(vb)
    base = binding.psa_attention_core(q, k, v, oracle.MASKED).clone()
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    for t in (q2, k2, v2):
        t[:, :, 1:, :] *= 64.0                      # heads 1, 2 changed; head 0 must not notice
    out = binding.psa_attention_core(q2, k2, v2, oracle.MASKED)
    assert torch.equal(out[:, :, :d].contiguous().view(torch.int16), base[:, :, :d].contiguous().view(torch.int16))


# ---- 128 < d_k <= 256: the one-row-tile kernel (full and masked schemes; the symmetric scheme stops at 128)
@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,d", [(1, 1, 128, 256), (1, 2, 256, 256), (2, 3, 384, 192), (1, 2, 640, 136), (2, 2, 1024, 256),
                                     (1, 3, 100, 256), (2, 1, 129, 200), (1, 2, 333, 248), (1, 1, 1, 256)])
def test_core_with_wide_heads(scheme, B, H, n, d):
    vals, bits = {}, {}
    for k, tid in (("Q", 4), ("K", 5), ("V", 6)):
        vals[k], bits[k] = inputs.tensor(11 * n + d, tid, (B, n, H, d), 1.0, "bf16")
    out = binding.psa_attention_core(_dev(bits["Q"]), _dev(bits["K"]), _dev(bits["V"]), scheme)
    ref, _ = oracle.attention_core(vals["Q"], vals["K"], vals["V"], scheme)
    assert tuple(out.shape) == (B, n, H * d)
    err = np.abs(_f64(out) - ref)
    assert (err <= TOL_BF16 + 2.0 ** -8 * np.abs(ref)).all(), err.max()
    _census(B, H, n, 0, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
def test_layer_with_wide_heads(scheme):
    B, H, n, D, d = 2, 2, 300, 128, 256
    Xv, Xb = inputs.tensor(29, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(29, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    out = binding.psa_attention(_dev(Xb), _dev(W[0][1]), _dev(W[1][1]), _dev(W[2][1]), H, scheme)
    ref, _ = oracle.attention_layer(Xv, W[0][0], W[1][0], W[2][0], H, scheme)
    err = np.abs(_f64(out) - ref)
    assert (err <= TOL_BF16 + 2.0 ** -8 * np.abs(ref)).all(), err.max()
    _census(B, H, n, D, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
def test_wide_heads_rescale_branch(scheme):
    # keys that grow from block to block drive the lazy rescale of the 256-column accumulator
    B, H, n, d = 1, 2, 640, 256
    row_scale = np.repeat(np.array([1.0, 24.0, 1.0, 48.0, 96.0]), 128)
    vq, bq = inputs.tensor(31, 4, (B, n, H, d), 1.0, "bf16")
    vk, bk = inputs.tensor(31, 5, (B, n, H, d), 1.0, "bf16", row_scale=row_scale)
    vv, bv = inputs.tensor(31, 6, (B, n, H, d), 1.0, "bf16")
    out = binding.psa_attention_core(_dev(bq), _dev(bk), _dev(bv), scheme)
    ref, _ = oracle.attention_core(vq, vk, vv, scheme)
    err = np.abs(_f64(out) - ref)
    assert (err <= TOL_BF16 + 2.0 ** -8 * np.abs(ref)).all(), err.max()
    assert binding.psa_last_rescales() > 0


def test_symmetric_scheme_stops_at_128_columns():
    q = torch.zeros(1, 128, 1, 256, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PsaError) as e:
        binding.psa_attention_core(q, None, None, oracle.SYMMETRIC)
    assert e.value.status == binding.ERR_UNSUPPORTED


def test_wide_heads_with_one_tensor_for_keys_and_values():
    B, H, n, d = 1, 2, 384, 256
    vq, bq = inputs.tensor(37, 4, (B, n, H, d), 1.0, "bf16")
    vk, bk = inputs.tensor(37, 5, (B, n, H, d), 1.0, "bf16")
    k = _dev(bk)
    out = binding.psa_attention_core(_dev(bq), k, k, oracle.MASKED)
    ref, _ = oracle.attention_core(vq, vk, vk, oracle.MASKED)
    err = np.abs(_f64(out) - ref)
    assert (err <= TOL_BF16 + 2.0 ** -8 * np.abs(ref)).all(), err.max()
