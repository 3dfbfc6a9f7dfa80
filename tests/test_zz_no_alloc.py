"""The allocation-free entry point, psa_attention_sym_f32_noalloc.

It serves callers that are not allowed to allocate device memory while running (fixed memory budgets,
plug-ins that do not own the allocator, latency-critical loops), so its scratch is an array built into
the library.  This test calls it through the C interface twice in a row -- the second call finds the
array dirty from the first -- and checks each result against the regular entry point
(psa_attention_core, symmetric scheme, fp32) within the fp32 tolerance of the other GPU tests, and the
size limit's error.  The file name sorts last so that a run stopping at the first failure has already
run everything else; the test also passes on its own in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2012_01114_b200 import binding

pytestmark = pytest.mark.gpu
TOL_F32 = 1e-4


def _x(seed, shape):
    rng = np.random.default_rng(seed)
    return torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).cuda()


def test_noalloc_matches_regular_entry_on_two_calls_in_a_row():
    cases = [(_x(1, (2, 96, 3, 40)), None), (_x(2, (1, 200, 2, 64)), None)]
    outs = []
    for X, _ in cases:                      # two calls back to back, different shapes, shared scratch
        B, n, H, d = X.shape
        out = torch.full((B, n, H * d), float("nan"), dtype=torch.float32, device="cuda")
        rc = binding.lib().psa_attention_sym_f32_noalloc(ctypes.c_void_p(X.data_ptr()), B, H, n, d,
                                                         ctypes.c_void_p(out.data_ptr()),
                                                         ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == binding.OK, binding.psa_status_string(rc)
        outs.append(out)
    torch.cuda.synchronize()
    for (X, _), out in zip(cases, outs):
        ref = binding.psa_attention_core(X, None, None, binding.SYMMETRIC)
        err = (out - ref).abs().max().item()
        assert err <= TOL_F32, err
    # same input again through the Python wrapper: the dirty scratch must not leak into the result
    again = binding.psa_attention_sym_f32_noalloc(cases[0][0])
    assert (again - outs[0]).abs().max().item() <= TOL_F32


def test_noalloc_rejects_problems_beyond_its_scratch():
    X = _x(3, (2, 1024, 1, 8))             # 2 * 1024 * 1024 scores > the built-in 2^20
    with pytest.raises(binding.PsaError) as ei:
        binding.psa_attention_sym_f32_noalloc(X)
    assert ei.value.status == binding.ERR_WORKSPACE
    assert "exceeds the built-in scratch" in str(ei.value)
    ok = _x(4, (1, 1024, 1, 8))            # exactly at the limit
    out = binding.psa_attention_sym_f32_noalloc(ok)
    ref = binding.psa_attention_core(ok, None, None, binding.SYMMETRIC)
    assert (out - ref).abs().max().item() <= TOL_F32
