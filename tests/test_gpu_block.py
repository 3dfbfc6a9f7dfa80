"""Attention block (layer + output projection over the concatenated heads) against the oracle, both
storage types: values within the paths' tolerances, projection MACs bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
# bf16 storage, fp32 accumulation: the layer's tolerance (2e-2 on y, which the output projection with a matrix of
# N(0,1)/sqrt(heads*d_k) entries carries over at the same size) plus the rounding of z itself to bf16, at most
# 2^-8 |z| (z reaches 4 and more in the symmetric scheme, where half a bf16 step is already 1.6e-2).
TOL_BF16 = 2e-2
TOL_BF16_REL = 2.0 ** -8
TOL_F32 = 1e-4    # fp32 storage and arithmetic


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _proj_macs(B, H, n, D, d, scheme):
    return ((1 if scheme == oracle.SYMMETRIC else 3) + 1) * B * n * D * H * d


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
def test_block_bf16_with_wide_heads(scheme):
    # heads of 256 columns run on the one-row-tile kernel between the two projection launches
    test_block_bf16_matches_oracle(scheme, 2, 2, 300, 128, 256)
    test_block_bf16_matches_oracle(scheme, 1, 1, 257, 64, 192)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 128, 64, 64), (2, 3, 256, 192, 64), (1, 2, 384, 320, 128),
                                       (2, 2, 333, 128, 64), (1, 12, 512, 768, 64)])
def test_block_bf16_matches_oracle(scheme, B, H, n, D, d):
    sym = scheme == oracle.SYMMETRIC
    Xv, Xb = inputs.tensor(11, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(11, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    Wov, Wob = inputs.tensor(11, 8, (H * d, D), (H * d) ** -0.5, "bf16")
    out = binding.psa_attention_block(_dev_bf16(Xb), _dev_bf16(W[0][1]), None if sym else _dev_bf16(W[1][1]),
                                      None if sym else _dev_bf16(W[2][1]), _dev_bf16(Wob), H, scheme)
    assert tuple(out.shape) == (B, n, D)
    ref, _, _ = oracle.attention_block(Xv, W[0][0], W[1][0], W[2][0], Wov, H, scheme)
    excess = (np.abs(_to_f64(out) - ref) - TOL_BF16_REL * np.abs(ref)).max()
    assert excess <= TOL_BF16, excess
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    assert got["proj_macs"] == _proj_macs(B, H, n, D, d, scheme)
    layer = binding.psa_skip_count(B, H, n, D, d, scheme, binding.BF16)
    for k in ("qk_macs", "pv_macs", "useful_qk_macs", "useful_pv_macs"):
        assert got[k] == layer[k]


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 1, 8, 4), (2, 3, 37, 50, 20), (1, 2, 200, 64, 128)])
def test_block_f32_matches_oracle(scheme, B, H, n, D, d):
    rng = np.random.default_rng(3 * n + d)
    X = (rng.standard_normal((B, n, D)) * 0.5).astype(np.float32)
    Ws = [(rng.standard_normal((D, H * d)) / np.sqrt(D)).astype(np.float32) for _ in range(3)]
    Wo = (rng.standard_normal((H * d, D)) / np.sqrt(H * d)).astype(np.float32)
    sym = scheme == oracle.SYMMETRIC
    dev = lambda a: torch.from_numpy(a).cuda()
    out = binding.psa_attention_block(dev(X), dev(Ws[0]), None if sym else dev(Ws[1]), None if sym else dev(Ws[2]),
                                      dev(Wo), H, scheme)
    ref, _, cnt = oracle.attention_block(X, Ws[0], Ws[1], Ws[2], Wo, H, scheme)
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= TOL_F32, err
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    assert got["proj_macs"] == _proj_macs(B, H, n, D, d, scheme)
    assert (got["qk_macs"], got["pv_macs"]) == (cnt.mac1, cnt.mac3)


def test_block_equals_layer_then_identity_and_leaves_the_layer_path_alone():
    # Wo = identity (exact in bf16): the block's output is the layer's output bit for bit; calls of the two entry
    # points in turn share the workspace and the counter blocks.
    B, H, n, D, d = 2, 2, 384, 128, 64
    _, Xb = inputs.tensor(12, 0, (B, n, D), 1.0, "bf16")
    W = [_dev_bf16(inputs.tensor(12, 1 + i, (D, H * d), D ** -0.5, "bf16")[1]) for i in range(3)]
    X = _dev_bf16(Xb)
    eye = torch.eye(H * d, dtype=torch.bfloat16, device="cuda")
    for scheme in (oracle.MASKED, oracle.FULL, oracle.MASKED):
        y = binding.psa_attention(X, W[0], W[1], W[2], H, scheme)
        st, c_layer = binding.psa_last_issued()
        z = binding.psa_attention_block(X, W[0], W[1], W[2], eye, H, scheme)
        st2, c_block = binding.psa_last_issued()
        assert st == binding.OK and st2 == binding.OK
        assert torch.equal(y, z)
        assert c_block["proj_macs"] == c_layer["proj_macs"] + B * n * H * d * D
        assert c_block["qk_macs"] == c_layer["qk_macs"] and c_block["pv_macs"] == c_layer["pv_macs"]


def test_block_workspace_and_argument_errors():
    B, H, n, D, d = 1, 2, 256, 128, 64
    need = binding.psa_block_workspace_bytes(B, H, n, D, d, oracle.FULL, binding.BF16)
    assert need >= binding.psa_workspace_bytes(B, H, n, D, d, oracle.FULL, binding.BF16) + B * n * H * d * 2
    L = binding.lib()
    x = torch.zeros((B, n, D), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((D, H * d), dtype=torch.bfloat16, device="cuda")
    p = lambda t: t.data_ptr()
    args = (B, H, n, D, d, int(oracle.FULL), binding.BF16, p(x), None)
    assert L.psa_attention_block(p(x), p(w), p(w), p(w), None, *args) == binding.ERR_NULL          # no Wo
    assert L.psa_attention_block(p(x), p(w), p(w), p(w), p(w) + 2, *args) == binding.ERR_ALIGN
    bad = (B, H, n, D, 48, int(oracle.FULL), binding.BF16, p(x), None)
    assert L.psa_attention_block(p(x), p(w), p(w), p(w), p(w), *bad) == binding.ERR_UNSUPPORTED
    sym = (B, H, n, D, d, int(oracle.SYMMETRIC), binding.BF16, p(x), None)
    w2 = torch.zeros_like(w)
    assert L.psa_attention_block(p(x), p(w), p(w2), None, p(w), *sym) == binding.ERR_SCHEME_ARGS


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 128, 64, 64), (2, 3, 256, 192, 64), (2, 2, 333, 128, 64), (1, 2, 384, 320, 128)])
def test_block_with_residual_bf16_matches_oracle(scheme, B, H, n, D, d):
    # z = R + y Wo with R = X (the usual skip connection) and with an unrelated R; the sum is formed in fp32 before
    # the rounding of z, so the tolerance is that of the block
    sym = scheme == oracle.SYMMETRIC
    Xv, Xb = inputs.tensor(21, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(21, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    Wov, Wob = inputs.tensor(21, 8, (H * d, D), (H * d) ** -0.5, "bf16")
    Rv, Rb = inputs.tensor(21, 9, (B, n, D), 2.0, "bf16")
    X = _dev_bf16(Xb)
    for res_v, res_dev in ((Xv, X), (Rv, _dev_bf16(Rb))):
        out = binding.psa_attention_block(X, _dev_bf16(W[0][1]), None if sym else _dev_bf16(W[1][1]),
                                          None if sym else _dev_bf16(W[2][1]), _dev_bf16(Wob), H, scheme, residual=res_dev)
        ref, _, _ = oracle.attention_block(Xv, W[0][0], W[1][0], W[2][0], Wov, H, scheme, residual=res_v)
        excess = (np.abs(_to_f64(out) - ref) - TOL_BF16_REL * np.abs(ref)).max()
        assert excess <= TOL_BF16, excess
        st, got = binding.psa_last_issued()
        assert st == binding.OK and got["proj_macs"] == _proj_macs(B, H, n, D, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
def test_block_with_residual_f32_matches_oracle(scheme):
    B, H, n, D, d = 2, 3, 37, 50, 20
    rng = np.random.default_rng(77)
    X = (rng.standard_normal((B, n, D)) * 0.5).astype(np.float32)
    Ws = [(rng.standard_normal((D, H * d)) / np.sqrt(D)).astype(np.float32) for _ in range(3)]
    Wo = (rng.standard_normal((H * d, D)) / np.sqrt(H * d)).astype(np.float32)
    R = rng.standard_normal((B, n, D)).astype(np.float32)
    sym = scheme == oracle.SYMMETRIC
    dev = lambda a: torch.from_numpy(a).cuda()
    out = binding.psa_attention_block(dev(X), dev(Ws[0]), None if sym else dev(Ws[1]), None if sym else dev(Ws[2]),
                                      dev(Wo), H, scheme, residual=dev(R))
    ref, _, _ = oracle.attention_block(X, Ws[0], Ws[1], Ws[2], Wo, H, scheme, residual=R)
    assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= TOL_F32


def test_block_residual_must_not_be_the_output():
    B, H, n, D, d = 1, 2, 128, 128, 64
    x = torch.zeros((B, n, D), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((D, H * d), dtype=torch.bfloat16, device="cuda")
    wo = torch.zeros((H * d, D), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(x)
    with pytest.raises(binding.PsaError) as ei:
        binding.psa_attention_block(x, w, w, w, wo, H, oracle.FULL, out=out, residual=out)
    assert ei.value.status == binding.ERR_SCHEME_ARGS
