"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same
seeded inputs.

Tolerances (floating point):
  O, dQ, dK, dV against fp64:          max abs <= 2e-2 and relative Frobenius <= 1e-2
  O against the BF16-emulating oracle:  within one BF16 ulp taken at the condition scale
                                        sum_t P|V| of the dot product (two correct FP32
                                        summation orders cannot agree more closely on outputs
                                        that are small through cancellation).  Observed on the
                                        GPU: no element beyond one ulp on C1, C2, C3 (standard
                                        mode), C4 and every multi-tile shape; 6 of 2.1 M elements
                                        on C5 (10 of 0.5 M on its head (0,0)) and 65 of 6.3 M on C3
                                        in the stabilised mode reach two ulp (O is rounded twice,
                                        O-bar and then O-bar / l, and each rounding can move by one
                                        ulp when the FP32 sums differ in their last bits).  The bar:
                                        at most 4e-5 of the elements beyond one ulp (twice the
                                        largest fraction observed), none beyond two.
                                        The strict count (one ulp at |O| itself, no condition
                                        scale) is reported and bounded per configuration by about
                                        twice its observed fraction (STRICT_BOUND below)
  L against the emulating oracle:       1e-4 + 1e-5 |L| on at least 98 % of the rows (same
                                        algorithm, FP32 noise only); a row where one P-bar entry
                                        rounds to the neighbouring BF16 value moves l by up to
                                        2^-8 of that entry, so every row is within 2^-8 + 1e-4
  L against fp64:                       2^-8 + 1e-4  (l sums BF16-rounded P-bar values)
  delta against fp64 rowsum of the same BF16 O and dO: 1e-5 relative
  gradients against the emulating oracle: relative Frobenius <= 2e-3 (where the fp64 bars are reachable)
Where the inputs make the fp64 bars unreachable for any BF16 implementation (the
emulating oracle itself misses them), the bar for that tensor becomes
"GPU error <= 1.25 x the emulating oracle's error".
"""
import numpy as np
import pytest
import torch

import attn_inputs as ai
import oracle
from _metrics import as_f64, bias_statistic, max_abs, rel_fro, ulp_violations

pytestmark = pytest.mark.gpu

MAX_ABS, REL_FRO = 2e-2, 1e-2
L_TOL_FP64 = 2 ** -8 + 1e-4
# Fraction of O elements that differ from the emulating oracle by more than one BF16 ulp of their own magnitude
# (outputs that are small through cancellation).  Observed: C1 0, multi-tile shapes <= 3.9e-4, C2 3.9e-4, C3 1.6e-7
# (standard) / 3.6e-5 (stabilised), C4 2.2e-3, C5 6e-4 to 2.0e-3 per head.  A regression that doubles these fails.
STRICT_BOUND = {"C1": 2e-4, "C2": 8e-4, "C3": 8e-5, "C4": 4.5e-3, "C5": 4e-3, "shape": 1.1e-3}
OBSERVED = []          # (label, violations, strict count, worst ratio, elements): printed at the end of the module


def _gpu():
    import _gpu_util
    return _gpu_util


def _tiles(d):
    import paper_2510_04212_b200 as attn
    br, bc = attn.attn_get_tiles(d)
    return dict(Br=br, Bc=bc)      # the key-tile size is part of the numerical contract in mode 1


def _oracle_all(t, meta, mode):
    c, a = meta["causal"], meta["alpha"]
    tl = _tiles(meta["d"])
    O, L = oracle.ref_fwd(t["q"], t["k"], t["v"], c, a)
    dQ, dK, dV, delta = oracle.ref_bwd(t["q"], t["k"], t["v"], t["dO"], O, L, c, a)
    Oe, Le = oracle.emu_fwd(t["q"], t["k"], t["v"], c, a, mode, **tl)
    de = oracle.emu_delta(Oe, t["dO"])
    dqe, dke, dve = oracle.emu_bwd(t["q"], t["k"], t["v"], t["dO"], Le, de, c, a)
    absv = ai.to_bf16_bits(np.abs(ai.bf16_bits_to_f32(t["v"])))
    A, _ = oracle.ref_fwd(t["q"], t["k"], absv, c, a)
    return dict(O=O, L=L, dQ=dQ, dK=dK, dV=dV, Oe=Oe, Le=Le, dQe=dqe, dKe=dke, dVe=dve, A=A)


def _check_against_oracle(g, r, t, label, strict_key=None):
    """Returns (violations of the one-ulp rule, strict count, worst ratio) of O against the emulating oracle."""
    # forward
    assert np.all(np.isfinite(as_f64(g["O"]))) and np.all(np.isfinite(g["L"])), label
    if max_abs(r["Oe"], r["O"]) <= MAX_ABS and rel_fro(r["Oe"], r["O"]) <= REL_FRO:
        assert max_abs(g["O"], r["O"]) <= MAX_ABS and rel_fro(g["O"], r["O"]) <= REL_FRO, label
    else:
        # the emulating oracle itself misses a bar on these inputs (|O| large enough that BF16 quantisation alone
        # exceeds 2e-2 on some element): no implementation of these rounding points can meet it; bound the GPU by the
        # oracle's own error instead
        assert max_abs(g["O"], r["O"]) <= 1.25 * max_abs(r["Oe"], r["O"]), (label, max_abs(g["O"], r["O"]), max_abs(r["Oe"], r["O"]))
        assert rel_fro(g["O"], r["O"]) <= 1.25 * rel_fro(r["Oe"], r["O"]), label
    viol, strict, worst = ulp_violations(g["O"], r["Oe"], r["A"])
    OBSERVED.append((label, viol, strict, worst, g["O"].size))
    assert viol <= 4e-5 * g["O"].size and worst <= 2.0, (label, viol, strict, worst)
    if strict_key is not None:
        assert strict <= max(1.0, STRICT_BOUND[strict_key] * g["O"].size), (label, viol, strict, worst)
    dL = np.abs(g["L"] - r["Le"])
    assert np.mean(dL > 1e-4 + 1e-5 * np.abs(r["Le"])) <= 0.02 and np.max(dL) <= L_TOL_FP64, label
    assert np.max(np.abs(g["L"] - r["L"])) <= L_TOL_FP64, label
    # delta: FP32 sum of exact products of the GPU's own BF16 O and dO
    want = (as_f64(t["dO"]) * as_f64(g["O"])).sum(-1)
    scale = np.abs(as_f64(t["dO"]) * as_f64(g["O"])).sum(-1)
    assert np.max(np.abs(g["delta"] - want) / (scale + 1e-30)) <= 1e-5, label
    # gradients
    for n in ("dQ", "dK", "dV"):
        got, ref, emu = g[n], r[n], r[n + "e"]
        assert np.all(np.isfinite(as_f64(got))), (label, n)
        if not np.any(ref):                                   # an exactly zero gradient (degenerate inputs) stays exactly zero
            assert not np.any(got & 0x7FFF) and not np.any(emu & 0x7FFF), (label, n)
            continue
        if np.max(np.abs(ref)) <= 1e-6:
            # a gradient that vanishes up to 1e-6 in exact arithmetic (e.g. dQ when P is one-hot: dP - delta = 0):
            # what an FP32 implementation returns there is the difference of two FP32 sums taken in different orders
            # (delta sequentially, dP on the tensor cores), i.e. noise of relative size 2^-23 of their terms; or, when the
            # cancellation is across BF16-rounded dS values (identical keys: sum_t dS_t = 0), the emulation's own residue
            assert max_abs(got, ref) <= max(1e-5, 1.25 * max_abs(emu, ref)), (label, n)
            continue
        feasible = max_abs(emu, ref) <= MAX_ABS and rel_fro(emu, ref) <= REL_FRO
        if feasible:
            assert max_abs(got, ref) <= MAX_ABS and rel_fro(got, ref) <= REL_FRO, (label, n)
            denom = np.linalg.norm(as_f64(emu).ravel())
            assert np.linalg.norm((as_f64(got) - as_f64(emu)).ravel()) <= 2e-3 * denom + 1e-6, (label, n)
        else:
            # rounding noise dominates this tensor in any BF16 implementation (e.g. dQ of the
            # tied-maximum case, whose exact value is ~1e-5): bound the GPU by the oracle's own error
            assert max_abs(got, ref) <= 1.25 * max_abs(emu, ref), (label, n)
            assert rel_fro(got, ref) <= 1.25 * rel_fro(emu, ref), (label, n)
    return viol, strict, worst


def teardown_module(module):
    # what was observed, for the record (shown with pytest -s or -rA)
    for label, viol, strict, worst, size in OBSERVED:
        print(f"[O vs emulating oracle] {label}: beyond one ulp {viol}, strict {strict} of {size} ({strict / size:.2e}), worst {worst:.2f}")


@pytest.mark.parametrize("mode", [0, 1])
def test_c1_single_tile(mode):
    t, m = ai.make("C1")
    g = _gpu().run_fwd_bwd(t, m, mode)
    viol, strict, worst = _check_against_oracle(g, _oracle_all(t, m, mode), t, f"C1 mode {mode}", "C1")
    assert viol == 0


@pytest.mark.parametrize("B,H,N,d,causal,mode", [
    (1, 2, 384, 64, True, 0),       # three tiles, causal
    (1, 2, 384, 64, False, 0),      # three tiles, full
    (2, 3, 640, 64, True, 1),       # five tiles, stabilised mode, more heads than fit one wave of a tile
    (1, 2, 256, 128, True, 0),      # d = 128
    (1, 2, 384, 128, False, 1),     # d = 128, full, stabilised
    (5, 7, 128, 64, True, 0),       # many single-tile heads
    (1, 1, 1152, 64, True, 0),      # nine tiles: odd count through the two-stage rings
    (40, 12, 128, 64, True, 0),     # 480 one-pair work items: every CTA of the persistent backward crosses item boundaries
    (9, 20, 256, 64, False, 1),     # 360 two-pair items, full attention (head-by-head item order)
    (3, 5, 512, 128, True, 0),      # d = 128, 60 CTAs of up to four pairs
])
def test_multi_tile_shapes(B, H, N, d, causal, mode):
    t = ai.gaussian(B, H, N, d, seed=100 + N + d + B)
    m = dict(B=B, H=H, N=N, d=d, causal=causal, alpha=d ** -0.5)
    g = _gpu().run_fwd_bwd(t, m, mode)
    viol, strict, worst = _check_against_oracle(g, _oracle_all(t, m, mode), t,
                                                f"{B}x{H}x{N}x{d} causal={causal} mode={mode}", "shape")
    assert viol == 0


def test_results_are_reproducible_run_to_run():
    # a missing barrier shows up as run-to-run differences; dQ is reduced with floating-point
    # atomics whose order may differ, so it is compared within FP32-reordering noise only
    t = ai.gaussian(2, 4, 512, 64, seed=21)
    m = dict(B=2, H=4, N=512, d=64, causal=True, alpha=0.125)
    runs = [_gpu().run_fwd_bwd(t, m, 0) for _ in range(3)]
    for r in runs[1:]:
        for n in ("O", "dK", "dV"):
            assert np.array_equal(r[n], runs[0][n]), n
        assert np.array_equal(r["L"], runs[0]["L"]) and np.array_equal(r["delta"], runs[0]["delta"])
        assert np.mean(r["dQ"] != runs[0]["dQ"]) < 1e-2
        assert rel_fro(r["dQ"], as_f64(runs[0]["dQ"])) < 1e-3


@pytest.mark.parametrize("causal", [False, True])
def test_forward_d128_is_bitwise_reproducible_on_long_sequences(causal):
    """Many CTAs with many key tiles each (two score buffers: warps of a CTA run up to a tile apart): a hand-off that
    lets a warp read the accumulator early shows up as run-to-run differences in a few 32-row blocks."""
    import paper_2510_04212_b200 as attn
    B, H, N, d = 2, 16, 4096, 128
    g = torch.Generator(device="cuda").manual_seed(5)
    q, k, v = (torch.randn(B, H, N, d, device="cuda", generator=g).to(torch.bfloat16) for _ in range(3))
    o = torch.empty_like(q)
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    first = None
    for _ in range(5):
        o.zero_()
        attn.attn_fwd(q, k, v, o, lse, B, H, N, d, causal, d ** -0.5, 0)
        torch.cuda.synchronize()
        assert attn.attn_last_device_status() == 0
        if first is None:
            first = (o.clone(), lse.clone())
        else:
            assert torch.equal(o.view(torch.int16), first[0].view(torch.int16)) and torch.equal(lse, first[1])
    ref = torch.nn.functional.scaled_dot_product_attention(q[:1, :2].float(), k[:1, :2].float(), v[:1, :2].float(),
                                                           is_causal=causal)
    assert (first[0][:1, :2].float() - ref).abs().max().item() <= 2e-2


def test_mitigation_parameters_are_honoured():
    import paper_2510_04212_b200 as attn
    t, m = ai.make("C3", B=1, H=2)
    try:
        attn.attn_set_mitigation(3.0, 2e-3)
        dev, o, lse = _gpu().run_fwd(t, m, 1)
        Oe, Le = oracle.emu_fwd(t["q"], t["k"], t["v"], True, m["alpha"], 1, beta=3.0, eps=2e-3, **_tiles(m["d"]))
    finally:
        attn.attn_set_mitigation(2.0, 1e-3)
    absv = ai.to_bf16_bits(np.abs(ai.bf16_bits_to_f32(t["v"])))
    A, _ = oracle.ref_fwd(t["q"], t["k"], absv, True, m["alpha"])
    viol, strict, worst = ulp_violations(_gpu().to_bits(o), Oe, A)
    assert viol == 0, (viol, strict, worst)
    assert np.max(np.abs(lse.cpu().numpy() - Le)) <= 1e-3


@pytest.fixture(scope="module")
def c3_runs():
    # tied-maximum stress case at the configuration's size: B = 8, all 96 heads (the recipe is per head)
    t, m = ai.make("C3")
    O, L = oracle.ref_fwd(t["q"], t["k"], t["v"], True, m["alpha"])
    out = {}
    for mode in (0, 1):
        g = _gpu().run_fwd_bwd(t, m, mode)
        Oe, Le = oracle.emu_fwd(t["q"], t["k"], t["v"], True, m["alpha"], mode, **_tiles(m["d"]))
        out[mode] = (g, Oe, Le)
    return t, m, O, L, out


def test_c3_rounding_bias_statistic(c3_runs):
    t, m, O, L, out = c3_runs
    st = {}
    for mode in (0, 1):
        g, Oe, Le = out[mode]
        st[mode] = (bias_statistic(g["O"], O, t["dO"], t["tied"], t["mu_sign"]),
                    bias_statistic(Oe, O, t["dO"], t["tied"], t["mu_sign"]))
    (g0, e0), (g1, e1) = st[0], st[1]
    # standard mode: biased, and the GPU statistic equals the oracle's to 3 significant digits
    assert e0["E_O"] > 2e-4 and e0["E_delta"] > 5e-4
    assert abs(g0["E_O"] - e0["E_O"]) <= 5e-4 * abs(e0["E_O"])
    assert abs(g0["E_delta"] - e0["E_delta"]) <= 5e-4 * abs(e0["E_delta"])
    # stabilised mode: an order of magnitude smaller, and compared on the scale of the standard-mode bias.
    # Observed at B = 8 (96 heads, 63,106 tied rows): E_O 4.549e-5 on the GPU against 4.655e-5 (oracle), E_delta 1.499e-4
    # against 1.539e-4: 1.7e-3 and 2.0e-3 of the standard-mode values.  No P-bar entry differs from the oracle's (L agrees
    # to 7.6e-6 on all 98,304 rows; one flipped entry of a tied row would move it by 4e-3); what differs is the FP32
    # accumulation of O-bar: here a tied row sums k = 2 or 4 equal products p v with p = bf16(exp(-(beta-1) r_m)), 16-bit
    # products whose FP32 sum the tensor core does not round as a sequence of IEEE additions, and 2,112 of the 98,304
    # rows hold an element whose O-bar then rounds to the other BF16 neighbour (362 rows in the standard mode, where
    # p = 1 and the sums are exact).  The bar is 3e-3 of the standard-mode statistic.
    assert abs(g1["E_O"]) <= 0.1 * abs(g0["E_O"]) and abs(g1["E_delta"]) <= 0.1 * abs(g0["E_delta"])
    assert abs(g1["E_O"] - e1["E_O"]) <= 3e-3 * abs(e0["E_O"])
    assert abs(g1["E_delta"] - e1["E_delta"]) <= 3e-3 * abs(e0["E_delta"])


def test_c3_outputs_and_gradients(c3_runs):
    t, m, O, L, out = c3_runs
    dQ, dK, dV, _ = oracle.ref_bwd(t["q"], t["k"], t["v"], t["dO"], O, L, True, m["alpha"])
    absv = ai.to_bf16_bits(np.abs(ai.bf16_bits_to_f32(t["v"])))
    A, _ = oracle.ref_fwd(t["q"], t["k"], absv, True, m["alpha"])
    for mode in (0, 1):
        g, Oe, Le = out[mode]
        de = oracle.emu_delta(Oe, t["dO"])
        dqe, dke, dve = oracle.emu_bwd(t["q"], t["k"], t["v"], t["dO"], Le, de, True, m["alpha"])
        r = dict(O=O, L=L, dQ=dQ, dK=dK, dV=dV, Oe=Oe, Le=Le, dQe=dqe, dKe=dke, dVe=dve, A=A)
        viol, strict, worst = _check_against_oracle(g, r, t, f"C3 mode {mode}", "C3")
        if mode == 0:
            assert viol == 0


def _sampled_heads_check(name, heads, mode, B=None):
    """Run the full-size configuration on the GPU, check sampled (b, h) heads against the
    oracle run on those heads alone (heads are independent problems)."""
    t, m = ai.make(name, B=B)
    g = _gpu().run_fwd_bwd(t, m, mode)
    for n in ("O", "dQ", "dK", "dV"):
        assert np.all(np.isfinite(as_f64(g[n]))), n
    assert np.all(np.isfinite(g["L"])) and np.all(np.isfinite(g["delta"]))
    for (b, h) in heads:
        sub = {n: np.ascontiguousarray(t[n][b:b + 1, h:h + 1]) for n in ("q", "k", "v", "dO")}
        ms = dict(m, B=1, H=1)
        gs = {n: np.ascontiguousarray(g[n][b:b + 1, h:h + 1]) for n in g}
        viol, strict, worst = _check_against_oracle(gs, _oracle_all(sub, ms, mode), sub,
                                                    f"{name} head ({b},{h}) mode {mode}", name)
        if name != "C5":
            assert viol == 0


@pytest.mark.parametrize("mode", [0, 1])
def test_c2_full_size_sampled_heads(mode):
    _sampled_heads_check("C2", [(0, 0), (7, 5), (15, 11)], mode)


def test_c4_long_context_sampled_head():
    _sampled_heads_check("C4", [(1, 9)], 0)


def test_c5_peaked_non_causal_sampled_head():
    _sampled_heads_check("C5", [(3, 31), (0, 0)], 0)


def _degenerate(kind, B, H, N, d, seed):
    """Seeded inputs for the degenerate cases of the method."""
    t = ai.gaussian(B, H, N, d, seed=seed)
    f32 = {n: ai.bf16_bits_to_f32(t[n]).copy() for n in ("q", "k", "v", "dO")}
    if kind == "zero_scores":          # Q = 0: every score is 0, every row a uniform average (r_m = 0: the rule does not fire)
        f32["q"][:] = 0.0
    elif kind == "identical_keys":     # one key repeated: all scores of a row equal and non-zero, N-fold ties in every tile
        f32["k"][:] = f32["k"][:, :, :1]
    elif kind == "zero_upstream":      # dO = 0: delta and all three gradients are exactly zero
        f32["dO"][:] = 0.0
    elif kind == "one_dominant_key":   # key 0 outweighs every other by > 100 in the exponent: P is one-hot up to underflow
        f32["q"] = np.abs(f32["q"]) + 1.0
        f32["k"][:] = -np.abs(f32["k"])
        f32["k"][:, :, 0] = 4.0
    return {n: ai.to_bf16_bits(a) for n, a in f32.items()}


@pytest.mark.parametrize("kind", ["zero_scores", "identical_keys", "zero_upstream", "one_dominant_key"])
@pytest.mark.parametrize("d,causal,mode", [(64, True, 0), (64, False, 1), (128, True, 1)])
def test_degenerate_inputs(kind, d, causal, mode):
    B, H, N = 1, 2, 384
    t = _degenerate(kind, B, H, N, d, seed=900 + d)
    m = dict(B=B, H=H, N=N, d=d, causal=causal, alpha=d ** -0.5)
    g = _gpu().run_fwd_bwd(t, m, mode)
    _check_against_oracle(g, _oracle_all(t, m, mode), t, f"{kind} d={d} causal={causal} mode={mode}")
    if kind == "zero_upstream":
        for n in ("dQ", "dK", "dV"):
            assert not np.any(g[n] & 0x7FFF), n                  # +-0 everywhere
        assert not np.any(g["delta"])
    if kind == "zero_scores" and not causal:
        want = as_f64(t["v"]).mean(axis=2, keepdims=True)       # uniform average of V
        assert np.max(np.abs(as_f64(g["O"]) - want)) <= 2e-2
        assert np.allclose(g["L"], np.log(N), atol=L_TOL_FP64)


@pytest.mark.parametrize("N,d,causal", [(32768, 64, True), (16384, 128, False)])
def test_long_sequences_on_sampled_rows(N, d, causal):
    """Hundreds of tiles per head (barrier phases, ring indices and the persistent item list far beyond what the small
    cases reach).  The whole tensors are out of reach of the CPU oracle in test time, so single rows are checked
    against the fp64 definition written out for that row: O and L of sampled queries, dQ of sampled queries, dK and
    dV of sampled keys (each is a sum over one row or one column of P, O(N d) work)."""
    B, H, alpha = 1, 2, d ** -0.5
    t = ai.gaussian(B, H, N, d, seed=1400 + d)
    g = _gpu().run_fwd_bwd(t, dict(B=B, H=H, N=N, d=d, causal=causal, alpha=alpha), 0)
    q, k, v, dO = (as_f64(t[n])[0, 1] for n in ("q", "k", "v", "dO"))
    O, L, dQ, dK, dV = (as_f64(g[n])[0, 1] if g[n].dtype == np.uint16 else g[n][0, 1].astype(np.float64)
                        for n in ("O", "L", "dQ", "dK", "dV"))
    rng = np.random.Generator(np.random.PCG64(7))
    rows = sorted(set([0, 1, 127, 128, N - 1] + [int(x) for x in rng.integers(0, N, 5)]))
    for T in rows:
        nk = T + 1 if causal else N
        s = alpha * (k[:nk] @ q[T])
        Lr = s.max() + np.log(np.exp(s - s.max()).sum())
        p = np.exp(s - Lr)
        assert abs(L[T] - Lr) <= L_TOL_FP64, T
        assert np.max(np.abs(O[T] - p @ v[:nk])) <= MAX_ABS, T
        delta = float(dO[T] @ (p @ v[:nk]))
        ds = p * (v[:nk] @ dO[T] - delta)
        assert np.max(np.abs(dQ[T] - alpha * (ds @ k[:nk]))) <= MAX_ABS, T
    Lf = g["L"][0, 1].astype(np.float64)
    delta_all = (dO * O).sum(-1)                     # the library's own delta convention (BF16 O), as its backward uses
    for tkey in rows:
        T0 = tkey if causal else 0
        p = np.exp(alpha * (q[T0:] @ k[tkey]) - Lf[T0:])
        ds = p * (dO[T0:] @ v[tkey] - delta_all[T0:])
        assert np.max(np.abs(dV[tkey] - p @ dO[T0:])) <= MAX_ABS, tkey
        assert np.max(np.abs(dK[tkey] - alpha * (ds @ q[T0:]))) <= MAX_ABS, tkey
