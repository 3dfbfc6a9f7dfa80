"""bf16 tensor-core path against the oracle: values within 2e-2, issued-MAC census bit-exact
against the oracle's independent block enumeration and against the host-side analytic twin."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2   # max |gpu - oracle| for bf16 storage with fp32 accumulation (outputs are O(1))


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _check_census(B, H, n, D, d, scheme):
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    assert got["qk_macs"] == B * H * t.tiles1 * 128 * 128 * d       # whole blocks are issued, ragged or not
    assert got["pv_macs"] == B * H * t.tiles3 * 128 * 128 * d
    assert got["useful_qk_macs"] == B * H * t.useful_mac1
    assert got["useful_pv_macs"] == B * H * t.useful_mac3
    nproj = 0 if D == 0 else (1 if scheme == oracle.SYMMETRIC else 3)
    assert got["proj_macs"] == nproj * B * n * D * H * d
    assert got == binding.psa_skip_count(B, H, n, D, d, scheme, binding.BF16)


def _core_case(B, H, n, d, scheme, seed):
    sym = scheme == oracle.SYMMETRIC
    vals, bits = {}, {}
    for k, tid in (("Q", 4), ("K", 5), ("V", 6)):
        vals[k], bits[k] = inputs.tensor(seed, tid, (B, n, H, d), 1.0, "bf16")
    if sym:
        out = binding.psa_attention_core(_dev_bf16(bits["Q"]), None, None, scheme)
        ref, _ = oracle.attention_core(vals["Q"], vals["Q"], vals["Q"], scheme)
    else:
        out = binding.psa_attention_core(_dev_bf16(bits["Q"]), _dev_bf16(bits["K"]), _dev_bf16(bits["V"]), scheme)
        ref, _ = oracle.attention_core(vals["Q"], vals["K"], vals["V"], scheme)
    err = np.abs(_to_f64(out) - ref).max()
    return err


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,d", [(1, 1, 128, 64), (1, 2, 256, 128), (2, 3, 384, 64), (1, 2, 640, 128),
                                     (2, 2, 1024, 64)])
def test_core_matches_oracle(scheme, B, H, n, d):
    err = _core_case(B, H, n, d, scheme, seed=n + d)
    assert err <= TOL_BF16, err
    _check_census(B, H, n, 0, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,D,d", [(1, 1, 128, 64, 64), (2, 3, 256, 192, 64), (1, 2, 384, 320, 128)])
def test_layer_with_projections_matches_oracle(scheme, B, H, n, D, d):
    sym = scheme == oracle.SYMMETRIC
    Xv, Xb = inputs.tensor(7, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(7, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    out = binding.psa_attention(_dev_bf16(Xb), _dev_bf16(W[0][1]), None if sym else _dev_bf16(W[1][1]),
                                None if sym else _dev_bf16(W[2][1]), H, scheme)
    ref, _ = oracle.attention_layer(Xv, W[0][0], W[1][0], W[2][0], H, scheme)
    err = np.abs(_to_f64(out) - ref).max()
    assert err <= TOL_BF16, err
    _check_census(B, H, n, D, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,d", [(2, 2, 1, 64), (1, 3, 100, 128), (2, 1, 129, 64), (1, 2, 200, 128), (1, 2, 333, 64),
                                     (2, 2, 1000, 128)])
def test_ragged_sequence_lengths(scheme, B, H, n, d):
    # n not a multiple of the 128-row block: the last block is zero-filled by TMA and its keys carry no weight
    err = _core_case(B, H, n, d, scheme, seed=7 * n + d)
    assert err <= TOL_BF16, err
    _check_census(B, H, n, 0, d, scheme)


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,d", [(4, 40, 384, 64), (2, 80, 300, 128), (3, 100, 256, 128), (5, 64, 130, 64)])
def test_more_work_items_than_sms(scheme, B, H, n, d):
    # Several hundred (head, pair of row tiles) items: every CTA of the persistent kernel walks several of them,
    # with an odd number of row tiles (a slot without rows in every other item) and ragged last blocks among them.
    err = _core_case(B, H, n, d, scheme, seed=3 * n + d)
    assert err <= TOL_BF16, err
    _check_census(B, H, n, 0, d, scheme)


def test_ragged_layer_with_projections():
    B, H, n, D, d = 2, 2, 300, 128, 64
    Xv, Xb = inputs.tensor(17, 0, (B, n, D), 1.0, "bf16")
    W = [inputs.tensor(17, 1 + i, (D, H * d), D ** -0.5, "bf16") for i in range(3)]
    out = binding.psa_attention(_dev_bf16(Xb), _dev_bf16(W[0][1]), _dev_bf16(W[1][1]), _dev_bf16(W[2][1]), H,
                                binding.MASKED)
    ref, _ = oracle.attention_layer(Xv, W[0][0], W[1][0], W[2][0], H, oracle.MASKED)
    assert np.abs(_to_f64(out) - ref).max() <= TOL_BF16
    _check_census(B, H, n, D, d, oracle.MASKED)


def test_config2_shape_reduced_batch():
    w = inputs.make("c2", batch=2)
    v, u = w["values"], w["upload"]
    out = binding.psa_attention(_dev_bf16(u["X"]), _dev_bf16(u["Wq"]), _dev_bf16(u["Wk"]), _dev_bf16(u["Wv"]),
                                12, binding.FULL)
    ref, _ = oracle.attention_layer(v["X"], v["Wq"], v["Wk"], v["Wv"], 12, oracle.FULL)
    assert np.abs(_to_f64(out) - ref).max() <= TOL_BF16
    _check_census(2, 12, 512, 768, 64, oracle.FULL)


def test_config3_shape_reduced_batch():
    w = inputs.make("c3", batch=1)
    v, u = w["values"], w["upload"]
    out = binding.psa_attention(_dev_bf16(u["X"]), _dev_bf16(u["Wq"]), _dev_bf16(u["Wk"]), _dev_bf16(u["Wv"]),
                                12, binding.MASKED)
    ref, _ = oracle.attention_layer(v["X"], v["Wq"], v["Wk"], v["Wv"], 12, oracle.MASKED)
    assert np.abs(_to_f64(out) - ref).max() <= TOL_BF16
    _check_census(1, 12, 1024, 768, 64, oracle.MASKED)


def test_reruns_are_bitwise_identical():
    _, qb = inputs.tensor(3, 4, (1, 512, 2, 128), 1.0, "bf16")
    _, kb = inputs.tensor(3, 5, (1, 512, 2, 128), 1.0, "bf16")
    _, vb = inputs.tensor(3, 6, (1, 512, 2, 128), 1.0, "bf16")
    q, k, v = _dev_bf16(qb), _dev_bf16(kb), _dev_bf16(vb)
    for scheme in (binding.FULL, binding.MASKED, binding.SYMMETRIC):
        args = (q, None, None) if scheme == binding.SYMMETRIC else (q, k, v)
        a = binding.psa_attention_core(*args, scheme).clone()
        b = binding.psa_attention_core(*args, scheme)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_census_is_exact_in_any_sequence_of_calls():
    # The FULL / MASKED path alternates between two counter blocks (the attention kernel of one call clears the block of
    # the next); the other paths clear their block themselves.  Any interleaving must leave every call's census exact.
    B, H, n, d = 2, 3, 384, 64
    _, qb = inputs.tensor(5, 4, (B, n, H, d), 1.0, "bf16")
    _, kb = inputs.tensor(5, 5, (B, n, H, d), 1.0, "bf16")
    _, vb = inputs.tensor(5, 6, (B, n, H, d), 1.0, "bf16")
    q, k, v = _dev_bf16(qb), _dev_bf16(kb), _dev_bf16(vb)
    qf = q.float()
    seq = [binding.MASKED, binding.MASKED, binding.FULL, binding.SYMMETRIC, binding.MASKED, "f32", binding.MASKED,
           binding.FULL, binding.SYMMETRIC, binding.SYMMETRIC, binding.FULL]
    for scheme in seq:
        if scheme == "f32":
            binding.psa_attention_core(qf, None, None, binding.SYMMETRIC)
            st, got = binding.psa_last_issued()
            assert st == binding.OK and got == binding.psa_skip_count(B, H, n, 0, d, binding.SYMMETRIC, binding.F32)
            continue
        args = (q, None, None) if scheme == binding.SYMMETRIC else (q, k, v)
        binding.psa_attention_core(*args, scheme)
        _check_census(B, H, n, 0, d, scheme)


def test_host_entry_matches_device_entry():
    B, H, n, D, d = 1, 2, 256, 128, 64
    _, Xb = inputs.tensor(9, 0, (B, n, D), 1.0, "bf16")
    Wb = [inputs.tensor(9, 1 + i, (D, H * d), D ** -0.5, "bf16")[1] for i in range(3)]
    host = [torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) for a in [Xb] + Wb]
    out_h = torch.empty((B, n, H * d), dtype=torch.bfloat16)
    binding.psa_attention_host(*host, H, binding.MASKED, out_h)
    out_d = binding.psa_attention(*[t.cuda() for t in host], H, binding.MASKED)
    assert torch.equal(out_h.view(torch.int16), out_d.cpu().view(torch.int16))


def test_core_host_entry_matches_device_entry():
    B, H, n, d = 2, 2, 300, 128
    bits = [inputs.tensor(19, t, (B, n, H, d), 1.0, "bf16")[1] for t in (4, 5, 6)]
    host = [torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) for a in bits]
    for scheme in (binding.FULL, binding.MASKED, binding.SYMMETRIC):
        sym = scheme == binding.SYMMETRIC
        out_h = torch.empty((B, n, H * d), dtype=torch.bfloat16)
        binding.psa_attention_core_host(host[0], None if sym else host[1], None if sym else host[2], scheme, out_h)
        _check_census(B, H, n, 0, d, scheme)
        out_d = binding.psa_attention_core(host[0].cuda(), None if sym else host[1].cuda(),
                                           None if sym else host[2].cuda(), scheme)
        assert torch.equal(out_h.view(torch.int16), out_d.cpu().view(torch.int16))


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,d", [(1, 1, 128, 64), (1, 2, 640, 128), (2, 3, 384, 64), (2, 2, 1000, 128), (1, 2, 333, 64),
                                     (3, 100, 256, 128), (4, 40, 384, 64), (1, 1, 2048, 128), (1, 2, 1536, 64)])
def test_keys_equal_values(scheme, B, H, n, d):
    # One tensor serves as keys and values (K = V != Q, the case Sec. 3.1 mentions): the kernel loads each key tile
    # once and uses it in both phases.  Same values and census as with two equal tensors.
    qv, qb = inputs.tensor(41 * n + d, 4, (B, n, H, d), 1.0, "bf16")
    kv, kb = inputs.tensor(41 * n + d, 5, (B, n, H, d), 1.0, "bf16")
    q, k = _dev_bf16(qb), _dev_bf16(kb)
    out = binding.psa_attention_core(q, k, k, scheme)
    _check_census(B, H, n, 0, d, scheme)
    if B * H * n * n <= 3 * 1024 * 1024:
        ref, _ = oracle.attention_core(qv, kv, kv, scheme)
        assert np.abs(_to_f64(out) - ref).max() <= TOL_BF16
    # two distinct tensors with the same contents take the two-ring path: bitwise the same result
    out2 = binding.psa_attention_core(q, k, k.clone(), scheme)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
