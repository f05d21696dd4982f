"""Packed variable-length batches (attn_fwd_packed / attn_bwd_packed): sequences stored one after the other with
cumulative offsets, token-major tensors.  Every sequence is compared with the oracle run on that sequence alone
(the oracle takes any length), and the rows of the packed outputs are checked to be exactly the rows of the
sequences (nothing else written)."""
import numpy as np
import pytest
import torch

import attn_inputs as ai
import oracle
from _metrics import as_f64, max_abs, rel_fro, ulp_violations

pytestmark = pytest.mark.gpu


def _env():
    import _gpu_util
    import paper_2510_04212_b200 as attn
    return _gpu_util, attn


def _pack(per_seq, lens, heads, d):
    """per-sequence [1][heads][n][d] bit arrays -> token-major [T][heads][d]"""
    rows = [np.transpose(a[0, :, :n], (1, 0, 2)) for a, n in zip(per_seq, lens) if n > 0]
    return np.ascontiguousarray(np.concatenate(rows, axis=0)).reshape(-1, heads, d)


@pytest.mark.parametrize("d,causal,Hkv,mode,lens", [
    (64, True, 2, 0, [512, 300, 77, 129, 0, 1]),
    (64, False, 4, 1, [200, 128, 5]),
    (128, True, 4, 0, [384, 130, 64]),
    (128, False, 2, 0, [256, 33]),
])
def test_packed_sequences_against_the_oracle(d, causal, Hkv, mode, lens):
    gu, attn = _env()
    br, bc = attn.attn_get_tiles(d)
    H, B = 4, len(lens)
    Nmax = -(-max(lens) // 128) * 128
    T = sum(lens)
    alpha = d ** -0.5
    seqs = [ai.gaussian(1, H, max(n, 1), d, seed=1700 + 10 * i + d) for i, n in enumerate(lens)]
    for s in seqs:
        s["k"], s["v"] = np.ascontiguousarray(s["k"][:, :Hkv]), np.ascontiguousarray(s["v"][:, :Hkv])
    packed = {n: _pack([s[n] for s in seqs], lens, H if n in ("q", "dO") else Hkv, d) for n in ("q", "k", "v", "dO")}
    dev = {n: gu.to_dev(packed[n]) for n in packed}
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    sentinel = 0x7FC1
    o = torch.full_like(dev["q"].view(torch.int16), sentinel).view(torch.bfloat16)
    lse = torch.full((H, T), float("nan"), dtype=torch.float32, device="cuda")
    nb_f = attn.attn_packed_workspace_bytes(B, H, Hkv, Nmax, d, False)
    nb_b = attn.attn_packed_workspace_bytes(B, H, Hkv, Nmax, d, True)
    assert 0 < nb_f < nb_b
    ws = torch.full((nb_b,), 0x7F, dtype=torch.uint8, device="cuda")           # poisoned: the call must not rely on its contents
    attn.attn_fwd_packed(dev["q"], dev["k"], dev["v"], o, lse, cu, ws, nb_f, B, H, Hkv, T, Nmax, d, causal, alpha, mode)
    dq = torch.full_like(dev["q"].view(torch.int16), sentinel).view(torch.bfloat16)
    dk = torch.full_like(dev["k"].view(torch.int16), sentinel).view(torch.bfloat16)
    dv = torch.full_like(dev["v"].view(torch.int16), sentinel).view(torch.bfloat16)
    delta = torch.full((H, T), float("nan"), dtype=torch.float32, device="cuda")
    ws.fill_(0x7F)
    attn.attn_bwd_packed(dev["q"], dev["k"], dev["v"], o, dev["dO"], lse, dq, dk, dv, delta, cu, ws, nb_b,
                         B, H, Hkv, T, Nmax, d, causal, alpha, mode)
    torch.cuda.synchronize()
    assert attn.attn_last_device_status() == 0
    got = dict(O=gu.to_bits(o), dQ=gu.to_bits(dq), dK=gu.to_bits(dk), dV=gu.to_bits(dv),
               L=lse.cpu().numpy(), delta=delta.cpu().numpy())
    for name in ("O", "dQ", "dK", "dV"):                           # every token row written
        assert not np.any(got[name] == sentinel), name
    assert np.all(np.isfinite(got["L"])) and np.all(np.isfinite(got["delta"]))
    start = 0
    for b, n in enumerate(lens):
        if n == 0:
            continue
        u = {x: np.ascontiguousarray(seqs[b][x][:, :, :n]) for x in ("q", "k", "v", "dO")}
        rows = slice(start, start + n)
        g = {x: np.ascontiguousarray(np.transpose(got[x][rows], (1, 0, 2)))[None] for x in ("O", "dQ", "dK", "dV")}
        g["L"] = got["L"][None, :, rows]
        g["delta"] = got["delta"][None, :, rows]
        start += n
        Oe, Le = oracle.emu_fwd_gqa(u["q"], u["k"], u["v"], causal, alpha, mode, Br=br, Bc=bc)
        O, L = oracle.ref_fwd_gqa(u["q"], u["k"], u["v"], causal, alpha)
        absv = ai.to_bf16_bits(np.abs(ai.bf16_bits_to_f32(u["v"])))
        A, _ = oracle.ref_fwd_gqa(u["q"], u["k"], absv, causal, alpha)
        viol, strict, worst = ulp_violations(g["O"], Oe, A)
        assert viol <= max(1.0, 1e-4 * g["O"].size) and worst <= 2.0, (b, viol, strict, worst)
        assert np.max(np.abs(g["L"] - Le)) <= 2e-3 and max_abs(g["O"], O) <= 2e-2, b
        d_want = (as_f64(u["dO"]) * as_f64(g["O"])).sum(-1)
        assert np.all(np.abs(g["delta"] - d_want) <= 1e-5 * (np.abs(as_f64(u["dO"])) * np.abs(as_f64(g["O"]))).sum(-1) + 1e-30), b
        dqe, dke, dve = oracle.emu_bwd(u["q"], u["k"], u["v"], u["dO"], np.ascontiguousarray(g["L"]),
                                       np.ascontiguousarray(g["delta"]), causal, alpha)
        dQ, dK, dV, _ = oracle.ref_bwd_gqa(u["q"], u["k"], u["v"], u["dO"], O, L, causal, alpha)
        for name, e, r in (("dQ", dqe, dQ), ("dK", dke, dK), ("dV", dve, dV)):
            denom = np.linalg.norm(as_f64(e).ravel())
            assert np.linalg.norm((as_f64(g[name]) - as_f64(e)).ravel()) <= 2e-3 * denom + 1e-6, (b, name)
            assert max_abs(g[name], r) <= 2e-2, (b, name)
            if np.linalg.norm(r.ravel()) > 0:                         # a one-token sequence has dQ = dK = 0 exactly
                assert rel_fro(g[name], r) <= 1e-2, (b, name)


def test_packed_equals_the_plain_call_on_equal_full_length_sequences():
    """B sequences of length N, packed: the same numbers as attn_fwd / attn_bwd on the [B][H][N][d] tensors."""
    gu, attn = _env()
    B, H, N, d = 2, 3, 256, 64
    t = ai.gaussian(B, H, N, d, seed=1800)
    alpha = d ** -0.5
    dev = {n: gu.to_dev(t[n]) for n in ("q", "k", "v", "dO")}
    o = torch.empty_like(dev["q"])
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    attn.attn_fwd(dev["q"], dev["k"], dev["v"], o, lse, B, H, N, d, True, alpha, 0)
    dq, dk, dv = (torch.empty_like(dev["q"]) for _ in range(3))
    delta = torch.empty_like(lse)
    nb = attn.attn_bwd_workspace_bytes(B, H, N, d)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    attn.attn_bwd(dev["q"], dev["k"], dev["v"], o, dev["dO"], lse, dq, dk, dv, delta, ws, nb, B, H, N, d, True, alpha, 0)
    # packed: token-major [B*N][H][d]
    pk = {n: dev[n].permute(0, 2, 1, 3).reshape(B * N, H, d).contiguous() for n in dev}
    cu = torch.tensor([0, N, 2 * N], dtype=torch.int32, device="cuda")
    po = torch.empty_like(pk["q"])
    plse = torch.empty((H, B * N), dtype=torch.float32, device="cuda")
    nbp = attn.attn_packed_workspace_bytes(B, H, H, N, d, True)
    pws = torch.empty(nbp, dtype=torch.uint8, device="cuda")
    attn.attn_fwd_packed(pk["q"], pk["k"], pk["v"], po, plse, cu, pws, nbp, B, H, H, B * N, N, d, True, alpha, 0)
    pdq, pdk, pdv = (torch.empty_like(pk["q"]) for _ in range(3))
    pdelta = torch.empty_like(plse)
    attn.attn_bwd_packed(pk["q"], pk["k"], pk["v"], po, pk["dO"], plse, pdq, pdk, pdv, pdelta, cu, pws, nbp,
                         B, H, H, B * N, N, d, True, alpha, 0)
    torch.cuda.synchronize()
    unpack = lambda x: x.reshape(B, N, H, d).permute(0, 2, 1, 3)
    assert torch.equal(unpack(po).view(torch.int16), o.view(torch.int16))
    assert torch.equal(plse.reshape(H, B, N).permute(1, 0, 2), lse)
    assert torch.equal(unpack(pdk).view(torch.int16), dk.view(torch.int16))
    assert torch.equal(unpack(pdv).view(torch.int16), dv.view(torch.int16))
    assert torch.equal(pdelta.reshape(H, B, N).permute(1, 0, 2), delta)
    a, b = gu.to_bits(unpack(pdq).contiguous()), gu.to_bits(dq)
    assert np.mean(a != b) < 1e-2 and rel_fro(a, as_f64(b)) < 1e-3           # dQ: floating-point atomics, order varies


def test_packed_argument_checks():
    _, attn = _env()
    p = 0x1000
    f = lambda **kw: attn.lib.attn_fwd_packed(p, p, p, p, p, kw.get("cu", p), kw.get("ws", p), kw.get("wsb", 1 << 40),
                                              kw.get("B", 2), 4, kw.get("Hkv", 2), kw.get("T", 300), kw.get("N", 256), 64, 1,
                                              0.125, 0, None)
    assert f(cu=None) == -1 and f(N=200) == -2 and f(Hkv=3) == -2 and f(T=0) == -2
    assert f(ws=None) == -5 and f(ws=0x1010) == -5 and f(wsb=1024) == -5
    assert attn.attn_packed_workspace_bytes(2, 4, 3, 256, 64, 0) == 0
    assert attn.attn_packed_workspace_bytes(2, 4, 2, 256, 64, 1) > attn.attn_packed_workspace_bytes(2, 4, 2, 256, 64, 0) > 0
