"""Multi-GPU readiness on one GPU: the (batch, head) problems are independent, so a rank's share is a contiguous slice
of the [B*H, N, d] tensors passed to the same C ABI.  Here every rank's slice (world sizes 2, 3 and 8) goes through
attn_fwd / attn_bwd on the one GPU and the pieces must reproduce the full call: O, L, delta, dK and dV bit for bit
(each is computed by one CTA in a fixed order), dQ within the run-to-run tolerance of its floating-point reduce-adds."""
import numpy as np
import pytest
import torch

import attn_inputs as ai
from _metrics import as_f64, rel_fro

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,N,d,causal,mode", [(2, 6, 256, 64, True, 0), (3, 5, 128, 64, True, 1), (2, 4, 256, 128, False, 0)])
def test_slices_of_every_rank_reproduce_the_full_call(B, H, N, d, causal, mode):
    import _gpu_util as gu
    import paper_2510_04212_b200 as attn
    from paper_2510_04212_b200.sharding import head_slice, shard_view
    t = ai.gaussian(B, H, N, d, seed=4242 + d)
    meta = dict(B=B, H=H, N=N, d=d, causal=causal, alpha=d ** -0.5)
    full = gu.run_fwd_bwd(t, meta, mode)
    for world in (2, 3, 8):
        parts = {n: [] for n in full}
        covered = 0
        for rank in range(world):
            start, stop = head_slice(B * H, world, rank)
            covered += stop - start
            if stop == start:
                continue                                       # more ranks than problems: this rank has nothing to do
            mine = {n: np.ascontiguousarray(shard_view(t[n], B, H, world, rank)) for n in ("q", "k", "v", "dO")}
            g = gu.run_fwd_bwd(mine, dict(meta, B=1, H=stop - start), mode)
            for n in full:
                parts[n].append(g[n])
        assert covered == B * H
        for n in full:
            got = np.concatenate(parts[n], axis=1).reshape(full[n].shape)
            if n == "dQ":
                assert np.mean(got != full[n]) < 1e-2 and rel_fro(got, as_f64(full[n])) < 1e-3, (world, n)
            else:
                assert np.array_equal(got, full[n]), (world, n)
