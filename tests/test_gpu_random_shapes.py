"""Seeded random shapes on the bf16 path: sampled rows of sampled (batch, head) slices against the oracle, bit-exact
census, and bitwise identical reruns.  The shapes mix both head sizes, the three schemes, ragged lengths, tile counts
that leave a row tile slot without rows, and head counts from one to several hundred work items per launch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2   # max |gpu - oracle|, bf16 storage with fp32 accumulation


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _cases():
    rng = np.random.RandomState(20121114)
    lengths = [1, 65, 127, 128, 129, 200, 256, 300, 384, 500, 512, 640, 777, 1024, 1300]
    out = []
    for i in range(24):
        n = int(lengths[rng.randint(len(lengths))])
        d = int((64, 128)[rng.randint(2)])
        scheme = int((oracle.FULL, oracle.MASKED, oracle.SYMMETRIC)[rng.randint(3)])
        B = int(rng.randint(1, 5))
        H = int(rng.randint(1, 65))
        while B * H * n * n > 2.5e8 and H > 1:
            H //= 2
        out.append((i, B, H, n, d, scheme))
    return out


@pytest.mark.parametrize("case,B,H,n,d,scheme", _cases())
def test_random_shape(case, B, H, n, d, scheme):
    sym = scheme == oracle.SYMMETRIC
    bits = {k: inputs.tensor_bits(1000 + case, t, (B, n, H, d), 1.0) for k, t in (("Q", 4), ("K", 5), ("V", 6))}
    q = _dev_bf16(bits["Q"])
    args = (q, None, None) if sym else (q, _dev_bf16(bits["K"]), _dev_bf16(bits["V"]))
    out = binding.psa_attention_core(*args, scheme)
    st, got = binding.psa_last_issued()
    assert st == binding.OK
    assert got == binding.psa_skip_count(B, H, n, 0, d, scheme, binding.BF16)
    t = oracle.tile_counts(n, d, scheme, 128, 128)
    assert got["qk_macs"] == B * H * t.tiles1 * 128 * 128 * d and got["pv_macs"] == B * H * t.tiles3 * 128 * 128 * d
    again = binding.psa_attention_core(*args, scheme)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))
    assert torch.isfinite(out.float()).all()
    # sampled rows of three slices against the oracle
    rng = np.random.RandomState(case)
    rows = sorted({0, n - 1, n // 2, min(n - 1, 127), min(n - 1, 128)} | {int(r) for r in rng.randint(0, n, size=6)})
    res = out.view(B, n, H, d).float().cpu().numpy().astype(np.float64)
    worst = 0.0
    for b, h in {(0, 0), (B - 1, H - 1), (int(rng.randint(B)), int(rng.randint(H)))}:
        sl = {k: inputs.bf16_bits_to_f64(a[b, :, h, :])[None, :, None, :] for k, a in bits.items()}
        K = sl["Q"] if sym else sl["K"]
        V = sl["Q"] if sym else sl["V"]
        ref = oracle.attention_rows(sl["Q"], K, V, scheme, 0, 0, rows)
        worst = max(worst, np.abs(res[b, rows, h, :] - ref).max())
    assert worst <= TOL_BF16, worst
