"""The online softmax of the bf16 path when a row's running maximum has to be raised after its first key block.

The kernels evaluate Eq. 2 block by block along the keys with a running row maximum m and row sum l, and raise m
only when a block's maximum exceeds it by more than 2^8; raising it multiplies the partial output (held in tensor
memory) and l by exp(m_old - m_new).  On standard-normal inputs that never happens after a row's first block, so
these cases scale the keys along the sequence (a factor per 128-key block) to force it: rising keys (every block
raises every row's maximum), a borderline ramp (only some rows of a warp are raised), falling keys (the maximum
sits in the first block and later weights underflow), and a single dominant late key (the oracle's own pin:
y_i tends to that key's value vector).  Every output element is compared with the fp64 oracle, the census must be
bit-exact, and psa_last_rescales must show that the branch ran (or did not).
"""
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


def _block_ramp(n, factors):
    """One factor per sequence position: block b of 128 positions gets factors[b]."""
    f = np.asarray(factors, dtype=np.float64)
    return f[np.minimum(np.arange(n) // 128, len(f) - 1)]


def _census(B, H, n, d, scheme):
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    assert got["qk_macs"] == B * H * t.tiles1 * 128 * 128 * d       # whole blocks are issued, ragged or not
    assert got["pv_macs"] == B * H * t.tiles3 * 128 * 128 * d
    assert got == binding.psa_skip_count(B, H, n, 0, d, scheme, binding.BF16)


def _run(B, H, n, d, scheme, key_scale, seed):
    """FULL / MASKED: only the keys are scaled, values stay N(0,1), so outputs are O(1) and the absolute tolerance of
    the other tests applies.  SYMMETRIC: query = key = value = X, so the rows of X carry the factors and the outputs
    grow with them; the error of a convex combination of value rows is linear in their size, so the tolerance is
    scaled by the largest factor."""
    sym = scheme == oracle.SYMMETRIC
    qv, qb = inputs.tensor(seed, 4, (B, n, H, d), 1.0, "bf16", row_scale=key_scale if sym else None)
    if sym:
        out = binding.psa_attention_core(_dev(qb), None, None, scheme)
        ref, _ = oracle.attention_core(qv, qv, qv, scheme)
        tol = TOL_BF16 * max(1.0, float(np.max(key_scale)))
    else:
        kv, kb = inputs.tensor(seed, 5, (B, n, H, d), 1.0, "bf16", row_scale=key_scale)
        vv, vb = inputs.tensor(seed, 6, (B, n, H, d), 1.0, "bf16")
        out = binding.psa_attention_core(_dev(qb), _dev(kb), _dev(vb), scheme)
        ref, _ = oracle.attention_core(qv, kv, vv, scheme)
        tol = TOL_BF16
    got = _f64(out)
    assert np.isfinite(got).all()
    # Elementwise |gpu - oracle| <= tol + 2^-8 |oracle|.  The second term is the rounding of the output itself to
    # bf16 (half a unit in the last of its 8 significant bits).  On standard-normal inputs outputs are averages far
    # below 1 and the term vanishes in the 2e-2; here the softmax is nearly one-hot, an output is close to a single
    # value vector entry, and those reach 4 and more, where half a bf16 step alone is 1.6e-2.
    excess = (np.abs(got - ref) - 2.0 ** -8 * np.abs(ref)).max()
    assert excess <= tol, (excess, tol, float(np.abs(got - ref).max()))
    _census(B, H, n, d, scheme)
    return binding.psa_last_rescales()


SHAPES = [(1, 2, 640, 64), (1, 2, 640, 128), (2, 1, 500, 64), (1, 1, 500, 128), (2, 40, 384, 128)]


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED, oracle.SYMMETRIC])
@pytest.mark.parametrize("B,H,n,d", SHAPES)
def test_rising_keys_rescale_every_block(scheme, B, H, n, d):
    # block maxima of scale*q.k are about 2.7 x the block's factor: each step of 3 in the factor adds about 8 to the
    # maximum in natural units (11.7 in base 2), beyond the 2^8 threshold
    T = (n + 127) // 128
    rescales = _run(B, H, n, d, scheme, _block_ramp(n, [1.0 + 3.0 * b for b in range(T)]), seed=31 * n + d)
    rows_with_later_blocks = B * H * (n - 128) if scheme != oracle.FULL else B * H * n
    assert rescales > rows_with_later_blocks // 2, rescales      # the branch ran, for most rows at least once


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,d", SHAPES[:4])
def test_borderline_ramp_rescales_only_some_rows_of_a_warp(scheme, B, H, n, d):
    # growth of about 2.7 x 1.4 = 3.8 natural units = 5.5 in base 2 per block, and the threshold compares with the
    # maximum as of the last raise: a row is raised at some blocks and not at others, and its neighbours differ
    T = (n + 127) // 128
    rescales = _run(B, H, n, d, scheme, _block_ramp(n, [1.0 + 1.4 * b for b in range(T)]), seed=17 * n + d)
    events = B * H * sum(min(128, n - 128 * t) * ((t if scheme == oracle.MASKED else T - 1)) for t in range(T))
    assert 0 < rescales < events, (rescales, events)             # some (row, block) events, not all


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("B,H,n,d", SHAPES[:4])
def test_falling_keys_keep_the_first_maximum(scheme, B, H, n, d):
    # the largest scores are in the first block: nothing is raised afterwards and the later weights underflow
    T = (n + 127) // 128
    rescales = _run(B, H, n, d, scheme, _block_ramp(n, [1.0 + 3.0 * (T - 1 - b) for b in range(T)]), seed=13 * n + d)
    assert rescales < B * H * n // 8, rescales


@pytest.mark.parametrize("scheme", [oracle.FULL, oracle.MASKED])
@pytest.mark.parametrize("d", [64, 128])
def test_one_dominant_late_key(scheme, d):
    # a single key 40 x larger than the rest, in the last block: rows whose query points its way put all their
    # weight on it (y_i -> v_j), the others none
    B, H, n = 1, 2, 512
    f = np.ones(n)
    f[n - 77] = 40.0
    rescales = _run(B, H, n, d, scheme, f, seed=5 * d)
    assert rescales > 0
