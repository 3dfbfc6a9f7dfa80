"""The allocation-free entry point, psa_attention_sym_f32_noalloc.

It serves callers that are not allowed to allocate device memory while running (fixed memory budgets,
plug-ins that do not own the allocator, latency-critical loops), so its scratch is an array built into
the library.  This test calls it through the C interface twice in a row -- the second call finds the
array dirty from the first -- and checks each result against the regular entry point
(psa_attention_core, symmetric scheme, fp32) and against the fp64 oracle within the fp32 tolerance of the
other GPU tests, that the device's free memory is the same before and after a call, and the size limit's
error.  The file name sorts last so that a run stopping at the first failure has already
run everything else; the test also passes on its own in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
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
        x64 = X.cpu().numpy().astype(np.float64)
        want, _ = oracle.attention_core(x64, x64, x64, oracle.SYMMETRIC)
        assert np.abs(out.cpu().numpy().astype(np.float64) - want).max() <= TOL_F32
    # same input again through the Python wrapper: the dirty scratch must not leak into the result
    again = binding.psa_attention_sym_f32_noalloc(cases[0][0])
    assert (again - outs[0]).abs().max().item() <= TOL_F32


def test_noalloc_call_leaves_free_device_memory_unchanged():
    # the property the entry point exists for: with the output tensor made beforehand, a call changes nothing
    # about the device's memory (the first call on a device, which looks up the array's address, came earlier)
    X = _x(5, (1, 128, 2, 32))
    out = torch.empty((1, 128, 64), dtype=torch.float32, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (ctypes.c_void_p(X.data_ptr()), 1, 2, 128, 32, ctypes.c_void_p(out.data_ptr()), stream)
    assert binding.lib().psa_attention_sym_f32_noalloc(*args) == binding.OK
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        assert binding.lib().psa_attention_sym_f32_noalloc(*args) == binding.OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


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
