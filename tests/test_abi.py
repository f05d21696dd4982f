"""Host-side checks of the C-ABI library: it loads, exports every symbol the header
declares, validates arguments before touching a device, and its host-only entry
points work without a GPU.  No compute call is made here."""
import ctypes as C
import os
import re

import pytest

import paper_2510_04212_b200 as attn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert set(attn.EXPORTS) <= set(names) and len(names) >= 9
    raw = C.CDLL(attn.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_host_only_entry_points():
    assert attn.attn_get_tiles(64) == (128, 64)
    assert attn.attn_get_tiles(128) == (128, 64)
    with pytest.raises(attn.AttnError) as e:
        attn.attn_get_tiles(96)
    assert e.value.code == -2
    assert attn.attn_bwd_workspace_bytes(16, 12, 1024, 64) == 16 * 12 * 1024 * 64 * 4
    assert attn.attn_bwd_workspace_bytes(1, 1, 100, 64) == 0       # N not a multiple of 128
    assert attn.attn_bwd_workspace_bytes(1, 1, 128, 80) == 0
    b0, e0 = attn.attn_get_mitigation()
    assert (b0, round(e0, 6)) == (2.0, 0.001)
    attn.attn_set_mitigation(4.0, 1e-2)
    b, e = attn.attn_get_mitigation()
    assert b == 4.0 and abs(e - 1e-2) < 1e-9
    for bad in ((1.0, 1e-3), (0.5, 1e-3), (2.0, 0.0), (2.0, -1.0), (float("nan"), 1e-3), (float("inf"), 1e-3)):
        with pytest.raises(attn.AttnError) as ex:
            attn.attn_set_mitigation(*bad)
        assert ex.value.code == -4
    attn.attn_set_mitigation(b0, e0)
    assert attn.attn_get_guard_max_shift() == 16.0
    attn.attn_set_guard_max_shift(32.0)
    assert attn.attn_get_guard_max_shift() == 32.0
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(attn.AttnError) as ex:
            attn.attn_set_guard_max_shift(bad)
        assert ex.value.code == -4
    assert attn.attn_get_guard_max_shift() == 32.0
    attn.attn_set_guard_max_shift(16.0)
    for code in range(0, -10, -1):
        assert attn.attn_strerror(code) != "unknown error code"
    assert attn.attn_strerror(-99) == "unknown error code"


def test_argument_validation_comes_before_any_device_work():
    lib = attn.lib
    p = 0x1000   # fake, 16-byte aligned, never dereferenced: every call below is rejected first
    fwd = lambda **kw: lib.attn_fwd(kw.get("q", p), p, p, kw.get("o", p), kw.get("lse", p), kw.get("B", 1), kw.get("H", 1),
                                    kw.get("N", 128), kw.get("d", 64), 1, kw.get("scale", 0.125), kw.get("mode", 0), None)
    assert fwd(q=None) == -1 and fwd(lse=None) == -1
    assert fwd(N=100) == -2 and fwd(N=64) == -2 and fwd(d=96) == -2 and fwd(B=0) == -2
    assert fwd(B=1 << 15, H=1 << 10, N=128) == -2          # B*H*N >= 2^31
    assert fwd(mode=4) == -3 and fwd(mode=16) == -3 and fwd(mode=-1) == -3  # forward knows bits 1, 2 and 8 only
    assert fwd(mode=8) == -3 and fwd(mode=8 | 2) == -3                      # the guarded rule needs the stabilised mode
    assert fwd(mode=8 | 1, q=None) == -1                                    # ... and is accepted with it (next check fails)
    assert lib.attn_fwd_count_ones(p, p, p, p, p, None, 1, 1, 128, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_fwd_count_ones(p, p, p, p, p, p, 1, 1, 100, 64, 1, 0.125, 0, None) == -2
    assert fwd(scale=0.0) == -4 and fwd(scale=-1.0) == -4 and fwd(scale=float("nan")) == -4
    pf = lambda **kw: lib.attn_fwd_pbar_format(p, p, p, p, p, kw.get("ones", p), 1, 1, kw.get("N", 128), 64, 1, 0.125, 0,
                                               kw.get("fmt", 1), None)
    assert pf(ones=None) == -1 and pf(fmt=3) == -3 and pf(fmt=-1) == -3 and pf(N=100) == -2
    assert fwd(q=p + 2) == -9
    bwd = lambda **kw: lib.attn_bwd(p, p, p, p, p, p, p, p, p, kw.get("delta", p), kw.get("ws", 0x1000),
                                    kw.get("ws_bytes", 1 << 30), 1, 1, kw.get("N", 128), 64, 1, 0.125,
                                    kw.get("mode", 0), None)
    assert bwd(delta=None) == -1
    assert bwd(N=130) == -2
    assert bwd(mode=8) == -3 and bwd(mode=-1) == -3        # backward accepts bits 1, 2 (ignored) and 4
    assert bwd(ws=None) == -5 and bwd(ws_bytes=16) == -5 and bwd(ws=0x1010) == -5
    assert lib.attn_bwd_delta_dp(None, p, p, p, p, p, 1, 1, 128, 64, 1, 0.125, None) == -1
    assert lib.attn_bwd_delta_dp(p, p, p, p, p, p, 1, 1, 100, 64, 1, 0.125, None) == -2
    assert lib.attn_bwd_delta_dp(p, p, p, p, p, p, 1, 1, 128, 64, 1, -1.0, None) == -4
    assert lib.attn_fwd_o_f32(p, p, p, p, p, None, 1, 1, 128, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_fwd_o_f32(p, p, p, p, p, p + 4, 1, 1, 128, 64, 1, 0.125, 0, None) == -9
    assert lib.attn_fwd_o_f32(p, p, p, p, p, p, 1, 1, 100, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_bwd_delta_f32(None, p, p, 1, 1, 128, 64, None) == -1
    assert lib.attn_bwd_delta_f32(p, p, p, 1, 1, 128, 96, None) == -2
    assert lib.attn_fwd_packed(p, p, p, p, p, None, p, 1 << 30, 2, 4, 2, 300, 256, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_fwd_packed(p, p, p, p, p, p, p, 16, 2, 4, 2, 300, 256, 64, 1, 0.125, 0, None) == -5
    assert lib.attn_bwd_packed(p, p, p, p, p, p, p, p, p, None, p, p, 1 << 30, 2, 4, 2, 300, 256, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_bwd_packed(p, p, p, p, p, p, p, p, p, p, p, p, 1 << 20, 2, 4, 2, 300, 200, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_bwd_preprocess(None, p, p, 1, 1, 128, 64, None) == -1
    assert lib.attn_bwd_preprocess(p, p, p, 1, 1, 128, 32, None) == -2


def test_argument_validation_of_the_grouped_padded_and_varlen_entry_points():
    lib = attn.lib
    p = 0x1000   # fake, aligned, never dereferenced: every call below is rejected by a check that comes first
    # grouped-query: H must be a multiple of H_kv >= 1
    assert lib.attn_fwd_gqa(p, p, p, p, p, 1, 4, 3, 128, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_fwd_gqa(p, p, p, p, p, 1, 4, 0, 128, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_fwd_gqa(p, p, p, p, None, 1, 4, 2, 128, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_bwd_gqa(p, p, p, p, p, p, p, p, p, p, p, 1 << 30, 1, 4, 8, 128, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_bwd_gqa(p, p, p, p, p, p, p, p, p, p, p, 16, 1, 4, 2, 128, 64, 1, 0.125, 0, None) == -5
    # padded: 1 <= seqlen <= N, N still a multiple of 128
    assert lib.attn_fwd_padded(p, p, p, p, p, 1, 1, 1, 128, 0, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_fwd_padded(p, p, p, p, p, 1, 1, 1, 128, 129, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_fwd_padded(p, p, p, p, p, 1, 1, 1, 100, 50, 64, 1, 0.125, 0, None) == -2
    assert lib.attn_fwd_padded(p, p, p, p, p, 1, 1, 1, 128, 50, 64, 1, 0.125, 16, None) == -3
    assert lib.attn_bwd_padded(p, p, p, p, p, p, p, p, p, p, p, 1 << 30, 1, 1, 1, 128, 200, 64, 1, 0.125, 0, None) == -2
    # one length per batch element: the array is required
    assert lib.attn_fwd_varlen(p, p, p, p, p, None, 1, 1, 1, 128, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_bwd_varlen(p, p, p, p, p, p, p, p, p, p, p, 1 << 30, None, 1, 1, 1, 128, 64, 1, 0.125, 0, None) == -1
    assert lib.attn_fwd_varlen(p, p, p, p, p, p, 1, 4, 3, 128, 64, 1, 0.125, 0, None) == -2


def test_compute_entry_points_refuse_to_run_without_a_b200():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present; the parity tests cover the compute path")
    p = 0x1000
    rc = attn.lib.attn_fwd(p, p, p, p, p, 1, 1, 128, 64, 1, 0.125, 0, None)
    assert rc in (-6, -8)         # no CUDA device / not sm_100: an error, never a fallback
