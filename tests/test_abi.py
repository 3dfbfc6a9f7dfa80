"""CPU-side checks of the C interface: the library loads, exports every symbol the header declares,
the host-only census agrees with the oracle's independent tile enumeration, and argument errors are
reported without touching a GPU."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2012_01114_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "psa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(psa_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations parsed"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.SYMMETRIC, oracle.MASKED])
@pytest.mark.parametrize("n,d", [(128, 64), (256, 128), (384, 64), (1024, 64), (1152, 128), (1, 64), (100, 128), (129, 64),
                                 (1000, 128)])
def test_skip_count_bf16_matches_oracle_tile_census(lib, scheme, n, d):
    # The kernels issue whole 128x128 blocks, also where the sequence ends inside a block: issued MACs are
    # (number of blocks the oracle's enumeration keeps) x 128*128*d; for n % 128 == 0 that is the oracle's
    # own issued figure.
    B, H = 3, 5
    c = binding.psa_skip_count(B, H, n, 0, d, scheme, binding.BF16)
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    assert c["qk_macs"] == B * H * t.tiles1 * 128 * 128 * d
    assert c["pv_macs"] == B * H * t.tiles3 * 128 * 128 * d
    if n % 128 == 0:
        assert (c["qk_macs"], c["pv_macs"]) == (B * H * t.issued_mac1, B * H * t.issued_mac3)
    assert c["useful_qk_macs"] == B * H * t.useful_mac1
    assert c["useful_pv_macs"] == B * H * t.useful_mac3
    assert c["proj_macs"] == 0


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.SYMMETRIC, oracle.MASKED])
@pytest.mark.parametrize("n,d", [(1, 1), (64, 64), (37, 20), (1000, 128)])
def test_skip_count_f32_is_the_element_census(lib, scheme, n, d):
    c = binding.psa_skip_count(2, 3, n, 48, d, scheme, binding.F32)
    t = oracle.tile_counts(n, d, scheme, 1, 1)
    assert c["qk_macs"] == c["useful_qk_macs"] == 6 * t.useful_mac1
    assert c["pv_macs"] == c["useful_pv_macs"] == 6 * t.useful_mac3
    nproj = 1 if scheme == oracle.SYMMETRIC else 3
    assert c["proj_macs"] == nproj * 2 * n * 48 * 3 * d


def test_skip_fractions_track_the_papers_reductions(lib):
    # Sec. 4.2 / 5.2: about 25 % and 50 % fewer operations.  At 128x128 blocks and n = 16384 the
    # issued MAC fractions are 75.2 % and 50.4 % of the original definition's.
    full = binding.psa_skip_count(1, 1, 16384, 0, 128, oracle.FULL, binding.BF16)
    sym = binding.psa_skip_count(1, 1, 16384, 0, 128, oracle.SYMMETRIC, binding.BF16)
    msk = binding.psa_skip_count(1, 1, 16384, 0, 128, oracle.MASKED, binding.BF16)
    tot = lambda c: c["qk_macs"] + c["pv_macs"]
    assert abs(tot(sym) / tot(full) - 0.752) < 1e-3
    assert abs(tot(msk) / tot(full) - 0.504) < 1e-3


def test_argument_errors_launch_nothing(lib):
    c = binding.Counts()
    assert lib.psa_skip_count(1, 1, 128, 0, 64, 7, binding.BF16, ctypes.byref(c)) == binding.ERR_SCHEME_ARGS
    assert lib.psa_skip_count(1, 1, 100, 0, 64, 0, binding.BF16, ctypes.byref(c)) == binding.OK      # ragged n is fine
    assert lib.psa_skip_count(1, 1, 128, 100, 64, 0, binding.BF16, ctypes.byref(c)) == binding.ERR_UNSUPPORTED  # d_model % 64
    assert lib.psa_skip_count(1, 1, 128, 0, 100, 0, binding.BF16, ctypes.byref(c)) == binding.ERR_UNSUPPORTED   # d_k % 8
    assert lib.psa_skip_count(1, 1, 128, 0, 256, 0, binding.BF16, ctypes.byref(c)) == binding.OK               # up to 256 columns
    assert lib.psa_skip_count(1, 1, 128, 0, 264, 0, binding.BF16, ctypes.byref(c)) == binding.ERR_UNSUPPORTED   # d_k > 256
    assert lib.psa_skip_count(1, 1, 128, 0, 256, 1, binding.BF16, ctypes.byref(c)) == binding.ERR_UNSUPPORTED   # symmetric: up to 128
    assert lib.psa_skip_count(1, 1, 128, 0, 96, 0, binding.BF16, ctypes.byref(c)) == binding.OK
    assert c.qk_macs == 128 * 128 * 128 and c.useful_qk_macs == 128 * 128 * 96    # issued at the padded width of 128
    assert lib.psa_skip_count(1, 1, 2048, 0, 64, 0, binding.F32, ctypes.byref(c)) == binding.ERR_UNSUPPORTED
    assert lib.psa_skip_count(0, 1, 128, 0, 64, 0, binding.BF16, ctypes.byref(c)) == binding.ERR_SHAPE
    assert lib.psa_skip_count(1, 1, 128, 0, 64, 0, binding.BF16, None) == binding.ERR_NULL
    # NULL data pointers and misaligned pointers are rejected before any CUDA call
    assert lib.psa_attention(None, None, None, None, 1, 1, 128, 64, 64, 0, None, None) == binding.ERR_NULL
    assert lib.psa_attention_core(None, None, None, 1, 1, 128, 64, 0, binding.BF16, None, None) == binding.ERR_NULL
    assert lib.psa_attention_core(8, 16, 16, 1, 1, 128, 64, 0, binding.BF16, 16, None) == binding.ERR_ALIGN
    assert lib.psa_attention_core(16, 32, 16, 1, 1, 128, 64, 1, binding.BF16, 16, None) == binding.ERR_SCHEME_ARGS
    assert lib.psa_attention(16, 16, 32, 16, 1, 1, 128, 64, 64, 1, 16, None) == binding.ERR_SCHEME_ARGS
    assert lib.psa_workspace_bytes(1, 1, 100, 0, 100, 0, binding.BF16, 0) == 0
    assert binding.psa_status_string(binding.ERR_TIMEOUT).startswith("a bounded")
    assert binding.psa_workspace_bytes(8, 12, 1024, 768, 64, oracle.MASKED, binding.BF16) >= 3 * 8 * 1024 * 768 * 2
