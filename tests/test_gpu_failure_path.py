"""The failure path shared by all kernels: a bounded wait that runs out must end the kernel in an orderly way and
report PSA_ERR_TIMEOUT through the device status word.  The library's self-test kernel waits on a barrier nobody
completes (nothing is broken on purpose in the production kernels, nothing traps); afterwards the same context
must run a normal call that matches the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_01114_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_expired_wait_reports_timeout_and_context_stays_usable():
    binding.psa_selftest_wait_expiry(limit_us=1000)
    st, got = binding.psa_last_issued()
    assert st == binding.ERR_TIMEOUT
    assert all(v == 0 for v in got.values()), got            # the work behind the wait was never done
    assert "wait expired" in binding.psa_status_string(st)
    # the context is intact: a normal call right after it is correct and reports PSA_OK
    qv, qb = inputs.tensor(2, 4, (1, 256, 2, 64), 1.0, "bf16")
    kv, kb = inputs.tensor(2, 5, (1, 256, 2, 64), 1.0, "bf16")
    vv, vb = inputs.tensor(2, 6, (1, 256, 2, 64), 1.0, "bf16")
    dev = [torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16) for b in (qb, kb, vb)]
    out = binding.psa_attention_core(*dev, binding.MASKED)
    ref, _ = oracle.attention_core(qv, kv, vv, oracle.MASKED)
    assert np.abs(out.float().cpu().numpy().astype(np.float64) - ref).max() <= 2e-2
    st, got = binding.psa_last_issued()
    assert st == binding.OK and got == binding.psa_skip_count(1, 2, 256, 0, 64, binding.MASKED, binding.BF16)


def test_selftest_rejects_limits_outside_its_range():
    for bad in (0, 100001):
        with pytest.raises(binding.PsaError) as ei:
            binding.psa_selftest_wait_expiry(limit_us=bad)
        assert ei.value.status == binding.ERR_SHAPE
