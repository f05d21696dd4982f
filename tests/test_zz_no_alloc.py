"""attn_bwd_static: the backward pass for callers that cannot allocate device memory at the point
of call (the dQ accumulator is a fixed array inside the library instead of a workspace argument).

Collected last on purpose (file name), so that a run that stops at the first failure has already
run every other test.  The check: on two calls in a row, with different inputs and shapes, the
entry point gives what attn_bwd gives with a caller-allocated workspace - dK, dV and delta bit for
bit (those kernels are deterministic), dQ within the reordering noise of its floating-point
atomics (the tolerance of the run-to-run reproducibility test).
"""
import numpy as np
import pytest
import torch

import attn_inputs as ai

pytestmark = pytest.mark.gpu


def _run_pair(B, H, N, d, causal, seed, check_no_allocation=False):
    import paper_2510_04212_b200 as attn
    from _gpu_util import to_bits, to_dev
    from _metrics import as_f64, rel_fro
    t = ai.gaussian(B, H, N, d, seed=seed)
    alpha = d ** -0.5
    dev = {n: to_dev(t[n]) for n in ("q", "k", "v", "dO")}
    o = torch.empty_like(dev["q"])
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    attn.attn_fwd(dev["q"], dev["k"], dev["v"], o, lse, B, H, N, d, causal, alpha, 0)

    def outputs():
        return [torch.empty_like(dev["q"]) for _ in range(3)] + [torch.empty_like(lse)]

    # existing entry point, caller-provided workspace (poisoned first: the library must clear it)
    dq0, dk0, dv0, delta0 = outputs()
    nbytes = attn.attn_bwd_workspace_bytes(B, H, N, d)
    ws = torch.full((nbytes,), 0x7F, dtype=torch.uint8, device="cuda")
    attn.attn_bwd(dev["q"], dev["k"], dev["v"], o, dev["dO"], lse, dq0, dk0, dv0, delta0, ws, nbytes,
                  B, H, N, d, causal, alpha, 0)
    # new entry point: no workspace argument
    dq1, dk1, dv1, delta1 = outputs()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    allocs_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    attn.attn_bwd_static(dev["q"], dev["k"], dev["v"], o, dev["dO"], lse, dq1, dk1, dv1, delta1,
                         B, H, N, d, causal, alpha, 0)
    torch.cuda.synchronize()
    if check_no_allocation:
        # what the entry point exists for: the device's free memory is what it was (the driver's own view, so an
        # allocation by the library itself would show), and torch's allocator was not asked for anything either
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == allocs_before
    assert attn.attn_last_device_status() == 0
    assert np.array_equal(to_bits(dk1), to_bits(dk0))
    assert np.array_equal(to_bits(dv1), to_bits(dv0))
    assert np.array_equal(delta1.cpu().numpy(), delta0.cpu().numpy())
    a, b = to_bits(dq1), to_bits(dq0)
    assert np.all(np.isfinite(as_f64(a)))
    assert np.mean(a != b) < 1e-2 and rel_fro(a, as_f64(b)) < 1e-3


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # the second call is smaller and differently shaped: it must not see what the first left behind
    _run_pair(2, 4, 512, 64, True, seed=31)     # the first call on the device resolves the scratch address
    _run_pair(1, 3, 256, 128, False, seed=32, check_no_allocation=True)
    _run_pair(2, 4, 512, 64, True, seed=33, check_no_allocation=True)


def test_a_call_that_uses_the_whole_scratch():
    # B*H*N*d = 8,388,608 elements: exactly the 32 MiB the library holds
    _run_pair(8, 16, 1024, 64, True, seed=34, check_no_allocation=True)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    import paper_2510_04212_b200 as attn
    p = 0x1000    # never dereferenced: the call is rejected before any device work
    # 16*12*1024*64 elements need 48 MiB > 32 MiB
    assert attn.lib.attn_bwd_static(p, p, p, p, p, p, p, p, p, p, 16, 12, 1024, 64, 1, 0.125, 0, None) == -5
    assert "workspace" in attn.attn_strerror(-5)
    # the checks come in attn_bwd's order: a NULL pointer is reported before the size
    assert attn.lib.attn_bwd_static(None, p, p, p, p, p, p, p, p, p, 16, 12, 1024, 64, 1, 0.125, 0, None) == -1
    # exactly at the limit is accepted by the size check (and then fails only on the fake pointers' alignment
    # or NULL checks, never with the workspace error): 8*16*1024*64*4 bytes = 32 MiB
    assert attn.attn_bwd_workspace_bytes(8, 16, 1024, 64) == 32 << 20
