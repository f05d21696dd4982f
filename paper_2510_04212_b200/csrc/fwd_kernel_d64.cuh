// Forward kernel for head width 64: Algorithm 1 (MODE 0) / Algorithm 3 (MODE 1) on sm_100a.
//
// Persistent: one CTA per SM with two "slots".  A slot owns one 128-row query tile of one (batch, head) at a time and
// walks over 128-row key tiles (B_r = 128, B_c = 128); when the tile is finished it takes the next one of its static list
// (heaviest first, dealt to the slots in snake order).  Per slot:
//   4 softmax warps    thread t owns query row t.  The 128 scores of the row are read from TMEM once, into registers,
//                      and the score columns are released at once: S of the next key tile is computed while this one is
//                      still in its maximum and exponential passes.  Row maximum; tie rule in MODE 1; P-bar =
//                      bf16(exp(S - m)) into its own TMEM columns; l accumulated in FP32 from the rounded values; O-bar
//                      rescaled when a maximum moved; epilogue.
//   1 TMA producer     Q (double-buffered across query tiles), K_j / V_j through two-stage rings.
//   1 MMA issuer       S = Q K_j^T (4 tcgen05.mma, N = 128) and O-bar += P-bar V_j (8, N = 64, P-bar from TMEM, V_j an
//                      MN-major shared-memory operand), FP32 accumulators in TMEM; two commits per key tile.
// TMEM per slot (256 columns): S [0,128) | P-bar [128,192) | O-bar [192,256).
//
// Why this shape (all measured on B200): an SM's tensor front end takes one tcgen05 instruction, MMA or commit, per
// 50-60 clocks whoever issues it, so 64-row key tiles (8 MMAs and 4 commits per tile) spent as long in the front end as
// in the exponentials; a 128-row key tile costs 12 MMAs and 2 commits.  With the scores in registers and P-bar in columns
// of its own the chain softmax(j) -> P-bar V(j) -> S(j+1) -> softmax(j+1) is broken: the softmax warps of a slot go from
// tile to tile without waiting for the tensor pipe, and the two slots keep two warps per scheduler in the exponential
// pass, which is what saturates the 16 exponentials per clock of an SM.
//
// Rounding points (paper Sec. 3.3.2 / Sec. 4): P-bar is rounded to BF16 right after the exponential and that BF16 value
// feeds both l and P-bar V; O-bar accumulates in FP32 over all key tiles and is rounded to BF16 once; O = bf16(O-bar / l).
#pragma once
#include <cuda.h>
#include <type_traits>
#include "ptx.cuh"
#include "fwd_kernel.cuh"

namespace attn {

struct Fwd64Cfg {
    static constexpr int D = 64, BR = 128, BC = 128;
    static constexpr int TILE_BYTES = 128 * 128;                  // 128 rows x 64 BF16 (one 128-byte swizzle panel)
    static constexpr int SLOTS = 2;
    static constexpr int SLOT_BYTES = 6 * TILE_BYTES;             // Q x2 | K x2 | V x2
    static constexpr int TILES_BYTES = SLOTS * SLOT_BYTES;
    static constexpr int SMEM_BYTES = TILES_BYTES + 2048;         // + alignment slack and barriers
    static constexpr int TMEM_COLS = 512, SLOT_COLS = 256;
    static constexpr int S_COL = 0, P_COL = 128, O_COL = 192;
    static constexpr int SOFTMAX_WARPS = 4;                       // per slot
    static constexpr int THREADS = (SLOTS * SOFTMAX_WARPS + 2 * SLOTS) * 32;   // + a producer and an issuer warp per slot
};

// The e-th query tile of slot u (of G2 slots in all): tiles are numbered heaviest first (n = (Tr - 1 - i) * BH + bh: the
// last query tile sees the most keys under the causal mask) and dealt in snake order.  Tiles that hold no query of their
// sequence (per-batch lengths) are skipped; every role of a slot walks the same sequence.
struct Fwd64Item {
    int bh, i, nkv, seqlen;
    int row0, kvrow0;          // first row of the Q / O tile and of the head's K, V in the [rows, d] views
};
__device__ __forceinline__ bool fwd64_item(int& e, int u, int G2, const FwdParams& prm, Fwd64Item& it, bool causal)
{
    while (true) {
        const int n = e * G2 + ((e & 1) ? (G2 - 1 - u) : u);
        if (n >= prm.Tr * prm.BH) return false;
        ++e;
        it.bh = n % prm.BH;
        it.i = prm.Tr - 1 - n / prm.BH;
        it.seqlen = prm.seqlen;
        if (prm.seqlens) {
            it.seqlen = min(max(prm.seqlens[it.bh / prm.H], 0), prm.N);
            if (it.i * 128 >= it.seqlen) continue;                // a query tile of padding
        }
        it.nkv = causal ? it.i + 1 : (it.seqlen + 127) / 128;
        it.row0 = it.bh * prm.N + it.i * 128;
        it.kvrow0 = (it.bh / prm.group) * prm.N;
        return true;
    }
}

// COUNT (compile time): also count, per row, the entries of P-bar that are exactly 1 (Sec. 3.3.2), and round P-bar to
// an 8-bit format when asked to.  PADDED (compile time; full attention only): the sequence may end inside a key tile.
template <int MODE, bool CAUSAL, bool COUNT = false, bool PADDED = false>
__global__ void __launch_bounds__(Fwd64Cfg::THREADS, 1)
attn_fwd64_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                  const FwdParams prm)
{
    using namespace ptx;
    using Cfg = Fwd64Cfg;
    constexpr int D = 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    // Barriers, per slot.  jj = running key-tile count of the slot (over all its query tiles), it = running query-tile count.
    //   Q_FULL [2]   (per it, index it & 1) Q landed
    //   K_FULL [2], V_FULL [2]   (index jj & 1) TMA landed
    //   S_FULL [2]   (index jj & 1) S(jj) done: scores ready, K stage free
    //   S_FREE       (per jj) the softmax warps hold the scores in registers: S(jj + 1) may be written
    //   P_FULL       (per jj) P-bar(jj) in TMEM and O-bar rescaled: P-bar V may be issued
    //   PV_DONE [2]  (index jj & 1) P-bar(jj) V done: V stage and P-bar columns free, O-bar updated
    //   O_FREE       (per it) the epilogue has read O-bar: the next query tile may overwrite it
    //   O_STAGED [2] (index it & 1) the four warps have written their rows of the O tile to the staging buffer, which is the
    //                Q buffer of that query tile; the producer stores it (TMA) and then reuses the buffer for Q
    // A barrier wait costs a shared-memory round trip of 200-300 clocks while MMAs run.  The softmax warps therefore probe
    // the barrier they will need next ahead of time (try_wait before a long stretch of arithmetic, result looked at after
    // it) and fall back to a blocking wait only when the probe said "not yet".
    enum { Q_FULL = 0, K_FULL = 2, V_FULL = 4, S_FULL = 6, PV_DONE = 8, S_FREE = 10, P_FULL = 11, O_FREE = 12,
           O_STAGED = 13, NB = 15 };
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + Cfg::TILES_BYTES);       // [SLOTS][NB]
    uint32_t& tmem_base_s = *reinterpret_cast<uint32_t*>(sm + Cfg::TILES_BYTES + Cfg::SLOTS * NB * 8);
    int& abort_flag = *reinterpret_cast<int*>(sm + Cfg::TILES_BYTES + Cfg::SLOTS * NB * 8 + 4);
    static_assert(Cfg::SLOTS * NB * 8 + 8 <= 1024, "barrier area");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    griddep_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < Cfg::SLOTS; ++s)
            for (int b = 0; b < NB; ++b)
                mbar_init(smem_u32(&bars[s * NB + b]), (b == S_FREE || b == P_FULL || b == O_FREE || b == O_STAGED || b == O_STAGED + 1) ? Cfg::SOFTMAX_WARPS : 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    constexpr int W_PROD = Cfg::SLOTS * Cfg::SOFTMAX_WARPS, W_ISS = W_PROD + Cfg::SLOTS;
    if (warp == W_PROD && lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO); }
    if (warp == W_ISS) { tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    griddep_wait();                                        // everything above ran beside the tail of the previous kernel

    // role and slot of this warp
    const int slot = (warp < W_PROD) ? warp / Cfg::SOFTMAX_WARPS : (warp < W_ISS ? warp - W_PROD : warp - W_ISS);
    const int u = static_cast<int>(blockIdx.x) * Cfg::SLOTS + slot, G2 = static_cast<int>(gridDim.x) * Cfg::SLOTS;
    auto bar = [&](int b) { return smem_u32(&bars[slot * NB + b]); };
    const uint32_t sQ0 = smem_u32(sm) + slot * Cfg::SLOT_BYTES;    // two Q buffers
    const uint32_t sK0 = sQ0 + 2 * Cfg::TILE_BYTES, sV0 = sK0 + 2 * Cfg::TILE_BYTES;
    const uint32_t tmem_slot = tmem_base_s + slot * Cfg::SLOT_COLS;
    Fwd64Item item;

    if (warp >= W_PROD && warp < W_ISS) {
        // ------------------------------------------------------------ TMA producer of the slot
        if (lane == 0) {
            bool ok = true;
            int jj = 0, it = 0;
            int orow[2] = {0, 0};                                 // first row of the O tile staged in each Q buffer
            // the O tile of query tile t, staged by the softmax warps in Q buffer t & 1: store it, wait until the buffer is read
            auto store_o = [&](int t) -> bool {
                if (!mbar_wait(bar(O_STAGED + (t & 1)), (t >> 1) & 1, &abort_flag)) return false;
                tma_store_2d(&tmO, sQ0 + (t & 1) * Cfg::TILE_BYTES, 0, orow[t & 1]);
                tma_store_commit_and_wait();
                return true;
            };
            for (int e = 0; ok && fwd64_item(e, u, G2, prm, item, CAUSAL); ++it) {
                const int qb = it & 1;
                if (it >= 2) ok = store_o(it - 2);                // the buffer holds the O tile of two query tiles ago
                if (!ok) break;
                orow[qb] = item.row0;
                mbar_expect_tx(bar(Q_FULL + qb), Cfg::TILE_BYTES);
                tma_load_2d(sQ0 + qb * Cfg::TILE_BYTES, &tmQ, bar(Q_FULL + qb), 0, item.row0);
                for (int j = 0; j < item.nkv; ++j, ++jj) {
                    const int st = jj & 1, ph = ((jj >> 1) - 1) & 1;          // the stage was used by tile jj - 2
                    if (jj >= 2) ok = mbar_wait(bar(S_FULL + st), ph, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(K_FULL + st), Cfg::TILE_BYTES);
                    tma_load_2d(sK0 + st * Cfg::TILE_BYTES, &tmK, bar(K_FULL + st), 0, item.kvrow0 + j * Cfg::BC);
                    if (jj >= 2) ok = mbar_wait(bar(PV_DONE + st), ph, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(V_FULL + st), Cfg::TILE_BYTES);
                    tma_load_2d(sV0 + st * Cfg::TILE_BYTES, &tmV, bar(V_FULL + st), 0, item.kvrow0 + j * Cfg::BC);
                }
            }
            // the last two O tiles
            if (ok && it >= 2) ok = store_o(it - 2);
            if (ok && it >= 1) ok = store_o(it - 1);
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
        __syncwarp();
    } else if (warp >= W_ISS) {
        // ------------------------------------------------------------ MMA issuer of the slot
        if (lane == 0) {
            constexpr uint32_t idesc_S = make_idesc_bf16(128, Cfg::BC, 0, 0);
            constexpr uint32_t idesc_PV = make_idesc_bf16(128, D, 0, 1);
            const uint64_t dQ0 = make_smem_desc(sQ0, 16, 1024);
            const uint64_t dK0 = make_smem_desc(sK0, 16, 1024);
            const uint64_t dV0 = make_smem_desc(sV0, Cfg::TILE_BYTES, 1024);
            const uint32_t tS = tmem_slot + Cfg::S_COL, tP = tmem_slot + Cfg::P_COL, tO = tmem_slot + Cfg::O_COL;
            // The key tiles of all query tiles of the slot form one sequence jj = 0, 1, ...; step jj issues S(jj + 1), which
            // may belong to the next query tile, as soon as the softmax warps hold S(jj) in registers, and then P-bar V(jj).
            bool ok = true;
            Fwd64Item nxt;
            int en = 0, itn = 0, jn = 0;                  // position of tile jj + 1: query tile count itn, key tile jn of it
            bool have_n = fwd64_item(en, u, G2, prm, nxt, CAUSAL);
            int itc = 0, jc = 0, nkvc = 0;                // position of tile jj
            for (int jj = -1; ok; ++jj) {
                if (have_n) {
                    // ---- S(jj + 1) = Q K^T
                    const int g = jj + 1, st = g & 1;
                    if (jn == 0) ok = mbar_wait(bar(Q_FULL + (itn & 1)), (itn >> 1) & 1, &abort_flag);
                    ok = ok && mbar_wait(bar(K_FULL + st), (g >> 1) & 1, &abort_flag);
                    if (ok && jj >= 0) ok = mbar_wait(bar(S_FREE), jj & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t dQ = dQ0 + static_cast<uint64_t>(((itn & 1) * Cfg::TILE_BYTES) >> 4);
                    const uint64_t dK = dK0 + static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        mma_ss(tS, dQ + ((k * 32) >> 4), dK + ((k * 32) >> 4), idesc_S, k > 0);
                    mma_commit(bar(S_FULL + st));
                }
                if (jj >= 0) {
                    // ---- O-bar += P-bar(jj) V: V as the B operand, N = d contiguous (MN-major), 16 key rows per step
                    const int st = jj & 1;
                    ok = mbar_wait(bar(V_FULL + st), (jj >> 1) & 1, &abort_flag) && mbar_wait(bar(P_FULL), jj & 1, &abort_flag);
                    if (ok && jc == 0 && itc > 0) ok = mbar_wait(bar(O_FREE), (itc - 1) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t dV = dV0 + static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < Cfg::BC / 16; ++k)
                        mma_ts(tO, tP + k * 8, dV + ((k * 2048) >> 4), idesc_PV, (jc > 0 || k > 0) ? 1u : 0u);
                    mma_commit(bar(PV_DONE + st));
                }
                if (!have_n) break;
                itc = itn; jc = jn; nkvc = nxt.nkv;
                if (++jn == nxt.nkv) { jn = 0; ++itn; have_n = fwd64_item(en, u, G2, prm, nxt, CAUSAL); }
            }
            (void)nkvc;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ softmax (thread = query row)
        const int wq = warp % Cfg::SOFTMAX_WARPS;                 // which 32 rows of the tile
        const uint32_t lane_base = static_cast<uint32_t>(wq * 32) << 16;
        const uint32_t tS = tmem_slot + Cfg::S_COL + lane_base, tP = tmem_slot + Cfg::P_COL + lane_base,
                       tO = tmem_slot + Cfg::O_COL + lane_base;
        const int row = wq * 32 + lane;                           // row inside the tile
        const float c_l2 = prm.scale * LOG2E;
        bool ok = true;
        int jj = 0;
        MBAR_PROBE_DECL(p_s_ready);                               // probe of S_FULL for tile jj, taken during the tile before
        MBAR_PROBE_DECL(p_pv_ready);                              // probe of PV_DONE for tile jj - 1, taken at the top of tile jj
        MBAR_PROBE_SET(p_s_ready, 0);

        // (m1, m2) <- two largest of {m1, m2, x, y}
        auto top2 = [](float& m1, float& m2, float x, float y) {
            const float hi = fmaxf(x, y), lo = fminf(x, y);
            m2 = max3(m2, lo, fminf(m1, hi));
            m1 = fmaxf(m1, hi);
        };

        for (int it = 0, e = 0; ok && fwd64_item(e, u, G2, prm, item, CAUSAL); ++it) {
            float m = -INFINITY, l = 0.0f;
            float r_run = -INFINITY;                          // guarded tie rule: largest tile maximum so far
            int n_ones = 0;
            for (int j = 0; j < item.nkv; ++j, ++jj) {
                // The tile is partly masked (DIAG) on the causal diagonal, where key column c is visible to this row iff
                // c <= row, and in the last tile of a sequence that ends inside it (full attention), where c <= seqlen-1-first key.
                const bool diag = (CAUSAL && j == item.i) || (PADDED && (j + 1) * Cfg::BC > item.seqlen);
                const int vis = CAUSAL ? row : item.seqlen - 1 - j * Cfg::BC;
                if (!__all_sync(0xffffffffu, MBAR_PROBE_RESULT(p_s_ready))) {
                    ok = mbar_wait(bar(S_FULL + (jj & 1)), (jj >> 1) & 1, &abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                // probe: has P-bar V of the tile before run?  (looked at after the maximum pass)
                if (jj == 0) MBAR_PROBE_SET(p_pv_ready, 1);
                else MBAR_PROBE(p_pv_ready, bar(PV_DONE + ((jj - 1) & 1)), ((jj - 1) >> 1) & 1);
                tc_fence_after();
                uint32_t s[128];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld32(tS + q * 32, *reinterpret_cast<uint32_t (*)[32]>(&s[q * 32]));
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_FREE));          // the scores are in registers: S of the next tile may be written
                if (diag) {
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c > vis) s[c] = __float_as_uint(-INFINITY);
                }
                // ---- row maximum of the raw accumulators (scale > 0 keeps the order)
                float mx, mx2 = -INFINITY;                          // mx2 (MODE 1): second largest
                if (MODE == 1) {
                    float a1 = -INFINITY, a2 = -INFINITY;
                    mx = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 64; c += 2) {
                        top2(mx, mx2, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
                        top2(a1, a2, __uint_as_float(s[64 + c]), __uint_as_float(s[64 + c + 1]));
                    }
                    mx2 = fmaxf(fminf(mx, a1), fmaxf(mx2, a2));
                    mx = fmaxf(mx, a1);
                } else {
                    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        m0 = max3(m0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
                        m1 = max3(m1, __uint_as_float(s[32 + c]), __uint_as_float(s[32 + c + 1]));
                        m2 = max3(m2, __uint_as_float(s[64 + c]), __uint_as_float(s[64 + c + 1]));
                        m3 = max3(m3, __uint_as_float(s[96 + c]), __uint_as_float(s[96 + c + 1]));
                    }
                    mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
                }
                mx *= prm.scale;
                if (MODE == 1) {
                    // tie rule of Algorithm 3 on the scaled scores of this key tile: r_s is needed only as "r_s > 1", i.e.
                    // whether the second largest score also lies within eps of the maximum
                    const float r_m = mx;
                    const int r_s = (r_m - mx2 * prm.scale <= prm.eps) ? 2 : 1;     // "2": at least two (-inf: false)
                    if (prm.guard_cap > 0.0f) {
                        // guarded variant (an extension, not the paper's rule): the maximum also counts as repeated when
                        // it equals the largest row maximum of the earlier tiles, and m' is the paper's unless that lies
                        // more than guard_cap above r_m (then m' = r_m + guard_cap, so l cannot underflow to 0)
                        const bool rep = (r_s > 1) || (fabsf(r_m - r_run) <= prm.eps);   // -inf operands compare false
                        r_run = fmaxf(r_run, r_m);
                        if (rep && r_m > 0.0f) mx = ((prm.beta - 1.0f) * r_m <= prm.guard_cap) ? prm.beta * r_m : r_m + prm.guard_cap;
                        if (rep && r_m < 0.0f) mx = (-r_m <= prm.guard_cap) ? 0.0f : r_m + prm.guard_cap;
                    } else {
                        if (r_m > 0.0f && r_s > 1) mx = prm.beta * r_m;
                        if (r_m < 0.0f && r_s > 1) mx = 0.0f;
                    }
                }
                const float m_new = fmaxf(m, mx);
                const float a = ex2((m - m_new) * LOG2E);     // m = -inf on the first tile gives a = 0; a = 1 when m stays
                const float negm = -m_new * LOG2E;
                m = m_new;
                // the P-bar columns are free once P-bar V of the tile before has run (issued long ago)
                if (!__all_sync(0xffffffffu, MBAR_PROBE_RESULT(p_pv_ready))) {
                    ok = mbar_wait(bar(PV_DONE + ((jj - 1) & 1)), ((jj - 1) >> 1) & 1, &abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                tc_fence_after();
                // probe: is S of the next tile there?  (looked at when this tile is finished)
                MBAR_PROBE(p_s_ready, bar(S_FULL + ((jj + 1) & 1)), ((jj + 1) >> 1) & 1);
                // ---- P-bar = bf16(exp(S - m)) -> TMEM; l += FP32 sum of the rounded values
                float sum0 = 0.0f, sum1 = 0.0f, sum2 = 0.0f, sum3 = 0.0f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t pk[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        const float s0 = __uint_as_float(s[q * 32 + c]), s1 = __uint_as_float(s[q * 32 + c + 1]);
                        if (MODE == 1) {
                            // the shifted maximum m = beta r_m can lie far above every score of the row: take the difference
                            // first, as Algorithm 3 writes it (one rounding), then bring it to base 2
                            fma2(x0, x1, s0, s1, prm.scale, -m_new);
                            mul2(x0, x1, x0, x1, LOG2E);
                        } else {
                            fma2(x0, x1, s0, s1, c_l2, negm);
                        }
                        float p0 = ex2(x0), p1 = ex2(x1);            // masked entries: ex2(-inf) = 0
                        if (COUNT && prm.pbar_fmt) round_fp8x2(p0, p1, prm.pbar_fmt);   // diagnostic: FP8 P-bar
                        const uint32_t w = pack_bf16(p0, p1);
                        pk[c >> 1] = w;
                        if (COUNT) n_ones += ((w & 0xFFFFu) == 0x3F80u) + ((w >> 16) == 0x3F80u);
                        if ((c & 2) == 0) add_bf16x2_halves(sum0, sum1, w);
                        else              add_bf16x2_halves(sum2, sum3, w);
                    }
                    tmem_st16(tP + q * 16, pk);
                }
                l = a * l + ((sum0 + sum1) + (sum2 + sum3));
                // ---- rescale O-bar when the maximum of any row of this warp moved (P-bar V of the tile before is complete)
                if (j > 0 && __any_sync(0xffffffffu, a != 1.0f)) {
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t o[32];
                        tmem_ld32(tO + c0, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * a);
                        tmem_st32(tO + c0, o);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(P_FULL));
            }
            if (!ok) break;
            // ---- epilogue: O-bar -> BF16, O = bf16(O-bar / l), L = m + log l
            ok = mbar_wait(bar(PV_DONE + ((jj - 1) & 1)), ((jj - 1) >> 1) & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float rl = __frcp_rn(l);
            // the Q tile is no longer needed: stage the O tile there in the same swizzled layout
            uint8_t* stage = sm + slot * Cfg::SLOT_BYTES + (it & 1) * Cfg::TILE_BYTES;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tO + c0, r);
                tmem_wait_ld();
                uint32_t out[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float o0 = __uint_as_float(r[c]), o1 = __uint_as_float(r[c + 1]);
                    if (!prm.single_rounding) {                   // O-bar -> BF16 (the paper's rounding point)
                        const uint32_t ob = pack_bf16(o0, o1);
                        o0 = bf16_lo(ob);
                        o1 = bf16_hi(ob);
                    }
                    out[c >> 1] = pack_bf16(div_rn(o0, l, rl), div_rn(o1, l, rl));
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int cc = (c0 >> 3) + v;
                    *reinterpret_cast<uint4*>(stage + row * 128 + ((cc ^ (row & 7)) << 4)) =
                        make_uint4(out[4 * v], out[4 * v + 1], out[4 * v + 2], out[4 * v + 3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(O_FREE));              // O-bar has been read: the next query tile may start it anew
            prm.lse[static_cast<size_t>(item.row0) + row] = m + lg2(l) * LN2;
            if (COUNT) prm.ones[static_cast<size_t>(item.row0) + row] = n_ones;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(O_STAGED + (it & 1)));  // the producer stores the tile
        }
    }

    // ---------------------------------------------------------------- teardown
    if (abort_flag) {
        // let copies that are still in flight land before shared memory is released
        for (int t = 0; t < 64; ++t) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == W_ISS) tmem_dealloc(tmem_base_s, Cfg::TMEM_COLS);
    if (tid == 0 && abort_flag) atomicExch(prm.status, 1);
}

}  // namespace attn
