"""The P-bar V product on the 8-bit tensor path (attn_quantize_v_e4m3 + attn_fwd_fp8pv): the FP8 setting the paper
names as future work (Sec. 5), measured against the oracle's FP8 study run on the dequantised V."""
import numpy as np
import pytest
import torch

import attn_inputs as ai
import oracle
from _metrics import as_f64, bf16_ulp, rel_fro

pytestmark = pytest.mark.gpu


def _env():
    import _gpu_util
    import paper_2510_04212_b200 as attn
    return _gpu_util, attn


from _fp8 import e4m3_table, quantize_e4m3


@pytest.mark.parametrize("d", [64, 128])
def test_v_is_quantised_and_transposed(d):
    gu, attn = _env()
    B, H, N = 2, 3, 256
    t = ai.gaussian(B, H, N, d, seed=2100 + d)
    v = gu.to_dev(t["v"])
    for scale in (1.0, 4.0):
        vt = torch.full((B, H, d, N), 0x7F, dtype=torch.uint8, device="cuda")
        attn.attn_quantize_v_e4m3(v, vt, B, H, N, d, scale)
        torch.cuda.synchronize()
        want = quantize_e4m3(as_f64(t["v"]) * scale)                    # [B][H][N][d]
        assert np.array_equal(vt.cpu().numpy(), np.transpose(want, (0, 1, 3, 2)))


@pytest.mark.parametrize("d,causal,mode,N,scale", [(64, True, 0, 384, 1.0), (64, False, 1, 256, 1.0), (128, True, 0, 384, 1.0),
                                                    (128, False, 0, 256, 2.0), (64, True, 0, 1024, 0.5)])
def test_fp8_pv_matches_the_oracle_on_the_dequantised_v(d, causal, mode, N, scale):
    gu, attn = _env()
    br, bc = attn.attn_get_tiles(d)
    B, H = 1, 2
    t = ai.gaussian(B, H, N, d, seed=2200 + d + N)
    alpha = float(d) ** -0.5
    dev = {n: gu.to_dev(t[n]) for n in ("q", "k", "v")}
    vt = torch.empty((B, H, d, N), dtype=torch.uint8, device="cuda")
    attn.attn_quantize_v_e4m3(dev["v"], vt, B, H, N, d, scale)
    o = torch.empty_like(dev["q"])
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    attn.attn_fwd_fp8pv(dev["q"], dev["k"], vt, o, lse, B, H, N, d, causal, alpha, mode, 1.0 / scale)
    torch.cuda.synchronize()
    assert attn.attn_last_device_status() == 0
    # the V the tensor core saw, times v_descale (a power of two here: exact, and it commutes with the roundings)
    vdeq = e4m3_table()[quantize_e4m3(as_f64(t["v"]) * scale)] / scale
    vbits = ai.to_bf16_bits(vdeq.astype(np.float32))
    assert np.array_equal(as_f64(vbits), vdeq)                          # E4M3 values are exact in BF16
    O, L, diag = oracle.emu_fwd(t["q"], t["k"], vbits, causal, alpha, mode, diagnostics=True, pbar_format="e4m3", Br=br, Bc=bc)
    a, b = as_f64(gu.to_bits(o)), as_f64(O)
    got_l = lse.cpu().numpy()
    assert np.all(np.isfinite(a)) and np.all(np.isfinite(got_l))
    # as for attn_fwd_pbar_format: nearly all rows to two BF16 ulp, every row within one flipped E4M3 step of one entry
    vmax = np.abs(vdeq).max()
    row_err = np.abs(a - b).max(-1)
    row_tol = 2.0 * bf16_ulp(np.maximum(np.abs(a), np.abs(b)).max(-1))
    assert float(np.mean(row_err > row_tol)) <= 0.02
    assert np.all(row_err <= 2.0 * 2.0 ** -4 * vmax / np.maximum(diag["l"], 1e-30) + row_tol), float(row_err.max())
    assert np.mean(np.abs(got_l - L) > 1e-4 + 1e-5 * np.abs(L)) <= 0.02
    assert np.all(np.abs(got_l - L) <= 2.0 * 2.0 ** -4 / np.maximum(diag["l"], 1e-30) + 1e-3)
    # against the definition on the original V: the FP8 error is visible but bounded (3 mantissa bits on both factors)
    Oref, _ = oracle.ref_fwd(t["q"], t["k"], t["v"], causal, alpha)
    assert 1e-3 < rel_fro(gu.to_bits(o), Oref) < 0.08


def test_fp8_pv_argument_checks():
    _, attn = _env()
    p = 0x1000
    assert attn.lib.attn_fwd_fp8pv(p, p, None, p, p, 1, 1, 128, 64, 1, 0.125, 0, 1.0, None) == -1
    assert attn.lib.attn_fwd_fp8pv(p, p, p, p, p, 1, 1, 128, 64, 1, 0.125, 2, 1.0, None) == -3
    assert attn.lib.attn_fwd_fp8pv(p, p, p, p, p, 1, 1, 128, 64, 1, 0.125, 0, 0.0, None) == -4
    assert attn.lib.attn_quantize_v_e4m3(p, None, 1, 1, 128, 64, 1.0, None) == -1
    assert attn.lib.attn_quantize_v_e4m3(p, p, 1, 1, 100, 64, 1.0, None) == -2
    assert attn.lib.attn_quantize_v_e4m3(p, p, 1, 1, 128, 64, -1.0, None) == -4
