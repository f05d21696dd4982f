"""The error path of the bounded device-side waits, exercised without a fault: a kernel built like the compute kernels
whose barriers nothing arrives on gives up after its one-millisecond limit, reports through the status word, frees its
TMEM and leaves the context usable."""
import time

import numpy as np
import pytest
import torch

import attn_inputs as ai
import oracle
from _metrics import as_f64, max_abs, rel_fro

pytestmark = pytest.mark.gpu

ATTN_ERR_TIMEOUT = -7


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    import _gpu_util as gu
    import paper_2510_04212_b200 as attn
    torch.cuda.synchronize()
    assert attn.attn_last_device_status() == 0
    t0 = time.time()
    attn.attn_selftest_wait_timeout()
    torch.cuda.synchronize()
    assert time.time() - t0 < 1.0                         # the limit is a millisecond, not the compute kernels' two seconds
    assert attn.attn_last_device_status() == ATTN_ERR_TIMEOUT
    assert attn.attn_last_device_status() == 0            # reading the record clears it
    assert "wait" in attn.attn_strerror(ATTN_ERR_TIMEOUT)
    # the same context still computes: an ordinary forward + backward right afterwards, checked against the oracle
    t, m = ai.make("C1")
    g = gu.run_fwd_bwd(t, m, 0)                           # asserts a clean device status itself
    O, L = oracle.ref_fwd(t["q"], t["k"], t["v"], True, m["alpha"])
    dQ, dK, dV, _ = oracle.ref_bwd(t["q"], t["k"], t["v"], t["dO"], O, L, True, m["alpha"])
    for got, ref in ((g["O"], O), (g["dQ"], dQ), (g["dK"], dK), (g["dV"], dV)):
        assert max_abs(got, ref) <= 2e-2 and rel_fro(got, ref) <= 1e-2
    # twice in a row, then TMEM must still be allocatable by a full-size kernel (the self-test freed what it took)
    for _ in range(2):
        attn.attn_selftest_wait_timeout()
    torch.cuda.synchronize()
    assert attn.attn_last_device_status() == ATTN_ERR_TIMEOUT
    g2 = gu.run_fwd_bwd(t, m, 0)
    assert np.array_equal(g2["O"], g["O"]) and np.array_equal(g2["dK"], g["dK"])
