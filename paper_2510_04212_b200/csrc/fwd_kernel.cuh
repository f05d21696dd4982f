// Forward kernel: Algorithm 1 (MODE 0) / Algorithm 3 (MODE 1) on sm_100a.
//
// One CTA owns one 128-row query tile of one (batch, head) and walks over 64-row key tiles
// (B_r = 128, B_c = 64).  Roles:
//   softmax warps (4)   thread t owns query row t: row maximum; tie rule in MODE 1; P-bar = bf16(exp(S - m)) written
//                       back to TMEM over S; l accumulated in FP32 from the rounded values; epilogue.
//   TMA producer        Q once, then K_j / V_j tiles through rings.
//   MMA issuer          S = Q K_j^T (operands in shared memory) and O-bar += P-bar V_j (P-bar from TMEM, V_j as an
//                       MN-major shared-memory operand), FP32 accumulators in TMEM.
//   correction warps    (d = 128 only, 4) O-bar *= exp(m_old - m_new) when a maximum of the warp's rows moved.
//
// d = 64: the CTA is deliberately small - 6 warps, 128 TMEM columns (S / P-bar [0,64) | O-bar [64,128)), 49 KB of
// shared memory, 80 registers - so that FOUR CTAs share an SM.  Inside a CTA softmax(j) -> P-bar V(j), S(j+1) ->
// softmax(j+1) is serial (S(j+1) reuses the columns P-bar(j) occupied); the other three CTAs fill the waits.  The 64
// scores of a row are read from TMEM 32 at a time, once per pass (maximum, exponential), which is what fits 80 registers; the softmax warps
// rescale O-bar themselves.
// d = 128: O-bar alone needs 128 columns, so a CTA takes 256 and two share an SM; the spare columns hold a second
// score buffer (S [0,64) and [64,128) | O-bar [128,256)): S(j+1) is computed while the softmax warps work on S(j).
// The scores stay in registers, and the O-bar rescale runs in the correction warps next to the exponential pass.
//
// Rounding points (paper Sec. 3.3.2 / Sec. 4): P-bar is rounded to BF16 right after
// the exponential and that BF16 value feeds both l and P-bar V; O-bar accumulates in
// FP32 over all key tiles and is rounded to BF16 once; O = bf16(O-bar / l).
#pragma once
#include <cuda.h>
#include <type_traits>
#include "ptx.cuh"

namespace attn {

template <int D>
struct FwdCfg {
    static constexpr int BR = 128, BC = 64;
    static constexpr int PANELS = D / 64;                 // 64-element (128-byte) swizzle panels per row
    static constexpr int Q_PANEL_BYTES = BR * 128;        // 128 rows x 128 bytes
    static constexpr int KV_PANEL_BYTES = BC * 128;       // 64 rows x 128 bytes
    static constexpr int Q_BYTES = PANELS * Q_PANEL_BYTES;
    static constexpr int KV_BYTES = PANELS * KV_PANEL_BYTES;
    // d = 128 (256 TMEM columns per CTA, two CTAs per SM either way): two score buffers, so that S(j+1) is computed
    // while the softmax warps work on S(j) and they go from tile to tile without waiting for the tensor pipe.
    // d = 64: one score buffer in 128 columns and four CTAs per SM instead; measured on the same problem, two
    // buffers with two CTAs per SM took 84 us (83 us with the correction warps below) and a variant with each row
    // shared by two threads (eight softmax warps per CTA) 80 us, against 73 us for this one: a warp spends
    // 0.5-0.9 us on the maximum and the 64 exponentials of a tile in every variant (the TMEM loads and stores
    // around them take 0.03-0.06 us each), so what counts is how many tiles the SM has in flight.
    static constexpr int S_BUFS = (D == 128) ? 2 : 1;
    // With two score buffers the O-bar rescale is done by four correction warps (thread = query row, like the softmax
    // warps) next to the softmax warps' exponential pass instead of inside their per-tile chain: the running maximum of
    // some row of a warp moves in most tiles (probability 1 - (j/(j+1))^32 at tile j for random scores), so the TMEM
    // load, multiply and store of the row's d accumulators were paid almost every tile.
    static constexpr bool CORR = (S_BUFS == 2);
    static constexpr int STAGES = 2;                       // K / V ring depth: 49 KB per CTA at d = 64, 97 KB at d = 128
    static constexpr int TILES_BYTES = Q_BYTES + 2 * STAGES * KV_BYTES + 1024;
    static constexpr int TMEM_COLS = (S_BUFS == 2 || D == 128) ? 256 : 128;
    static constexpr int CTAS_PER_SM = (TMEM_COLS == 128) ? 4 : 2;
    // 256 TMEM columns per CTA: only two CTAs fit an SM; ask for enough shared memory that a third one is never made
    // resident just to sit in tcgen05.alloc
    static constexpr int SMEM_BYTES = (CTAS_PER_SM == 2 && TILES_BYTES < 80 * 1024) ? 80 * 1024 : TILES_BYTES;
    static constexpr int S_COL = 0, O_COL = 64 * S_BUFS;  // S buffer b at columns [64 b, 64 b + 64)
    static constexpr int SOFTMAX_WARPS = 4, CORR_WARPS = CORR ? 4 : 0;
    static constexpr int THREADS = (SOFTMAX_WARPS + CORR_WARPS + 2) * 32;
    static constexpr bool CHUNKED = (CTAS_PER_SM == 4);   // softmax passes read the scores 32 at a time (register budget)
    static_assert(STAGES <= 3 && O_COL + D <= TMEM_COLS, "barrier numbering / TMEM budget");
};

struct FwdParams {
    float* lse;
    int* ones;                 // COUNT instantiations only: per-row count of P-bar entries equal to 1 (may be nullptr)
    float* o_f32;              // COUNT instantiations only, may be nullptr: O = O-bar / l with O-bar left in FP32
    int pbar_fmt;              // COUNT instantiations only: 0 = BF16 P-bar, 1 = E4M3, 2 = E5M2 (diagnostic)
    int single_rounding;       // != 0: O-bar is not rounded to BF16 before the division (diagnostic variant)
    int N, BH, Tr;             // N: rows per head in memory; Tr: 128-row query tiles that hold one of the seqlen queries
    int seqlen;                // queries and keys per head that count (<= N); rows beyond are padding
    const int* seqlens;        // != nullptr: one sequence length per batch element (device memory, [B]) instead of seqlen
    int H;                     // query heads (batch element of head bh: bh / H)
    int group;                 // query heads per key/value head (grouped-query attention; 1 = multi-head)
    float scale, beta, eps;
    float guard_cap;           // > 0: guarded variant of the tie rule (mode 1 only)
    float v_descale;           // FP8PV instantiations only: O-bar is multiplied by this before it is rounded
    int* status;
};

// COUNT (compile time): also count, per row, the entries of P-bar that are exactly 1 (Sec. 3.3.2)
// PADDED (compile time; full attention only, the causal mask already hides the padding keys from every sequence row):
// the sequence may end inside a key tile, whose remaining keys are masked
// FP8PV (compile time): P-bar is rounded to E4M3 and multiplied with an E4M3 V on the 8-bit tensor path
// (tcgen05.mma kind::f8f6f4).  tmV then describes V transposed, [B*H*d rows][N keys] of one-byte elements, so that a
// key tile is a K-major operand ([d rows][64 keys], 64-byte rows, 64-byte swizzle).
template <int D, int MODE, bool CAUSAL, bool COUNT = false, bool PADDED = false, bool FP8PV = false>
__global__ void __launch_bounds__(FwdCfg<D>::THREADS, FwdCfg<D>::CTAS_PER_SM)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                const FwdParams prm)
{
    using namespace ptx;
    using Cfg = FwdCfg<D>;
    constexpr bool LEAN = (Cfg::S_BUFS == 1);              // one score buffer: one commit per tile, see the issuer
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sQ = smem_u32(sm);                      // also the staging buffer of the O tile
    const uint32_t sK0 = sQ + Cfg::Q_BYTES;
    const uint32_t sV0 = sK0 + Cfg::STAGES * Cfg::KV_BYTES;

    // S_FULL and P_FULL exist once per score buffer (index = j & 1 with two buffers): with a single barrier the
    // second completion could arrive before the waiter has looked at the first, and a parity wait cannot tell.
    // A_FULL / O_READY (correction warps only, per tile parity): the rows' rescale factors are in shared memory / O-bar
    // has been rescaled for tile j (or needed nothing), P-bar(j) V_j may be issued.
    enum { Q_FULL = 0, K_FULL = 1, K_EMPTY = 4, V_FULL = 7, V_EMPTY = 10, S_FULL = 13, P_FULL = 15, PV_DONE = 17,
           EPI = 19, A_FULL = 20, O_READY = 22, NBARS = 24 };
    // PV_DONE: completion of P-bar(j) V_j.  With two score buffers there are two, used alternately (index j & 1, phase
    // (j >> 1) & 1), because its waiters do not wait every tile (the O-bar rescale only when a maximum moved, the
    // epilogue once) and a warp can be more than one completion ahead of it: having finished tile j, whose S was
    // ready early, it may find P-bar V of tile j-1 not even issued.  A parity wait only tells the current phase from the
    // one before, so on a single barrier "wait for tile j" would then return at once (or, in the other direction,
    // never).  Phase j-2 is always complete for a warp that has seen S(j) (S(j) is issued after P-bar V of j-2 and its
    // commit tracks it), which is exactly the distance the alternating pair covers.
    __shared__ float sA[2][Cfg::CORR ? 128 : 1];            // rescale factor per row, by tile parity
    __shared__ __align__(8) uint64_t bars[NBARS];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x % prm.BH;
    const int i = prm.Tr - 1 - blockIdx.x / prm.BH;        // heaviest (most key tiles) first
    int seqlen = prm.seqlen;
    griddep_launch_dependents();
    if (prm.seqlens) {                                     // per-sequence lengths: a query tile of padding has nothing to do
        griddep_wait();                                    // (the lengths may come from the kernel before this one)
        seqlen = min(max(prm.seqlens[bh / prm.H], 0), prm.N);
        if (i * Cfg::BR >= seqlen) return;
    }
    // 64-row key tiles this query tile sees (full attention: those that hold one of the seqlen keys)
    const int nkv = CAUSAL ? 2 * (i + 1) : (seqlen + Cfg::BC - 1) / Cfg::BC;
    const int row0 = bh * prm.N + i * Cfg::BR;             // first row of this Q tile in the [B*H*N, d] view
    const int kvrow0 = (bh / prm.group) * prm.N;           // K, V are [B][H / group][N][d]

    auto bar = [&](int b) { return smem_u32(&bars[b]); };
    auto pv_done_bar = [&](int j) { return smem_u32(&bars[PV_DONE + ((Cfg::S_BUFS == 2) ? (j & 1) : 0)]); };
    auto pv_done_phase = [&](int j) { return static_cast<uint32_t>(((Cfg::S_BUFS == 2) ? (j >> 1) : j) & 1); };

    if (tid == 0) {
        for (int b = 0; b < NBARS; ++b) mbar_init(bar(b), (b == P_FULL || b == P_FULL + 1 || b == EPI || b >= A_FULL) ? 128 : 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    constexpr int PRODUCER = Cfg::SOFTMAX_WARPS + Cfg::CORR_WARPS, ISSUER = PRODUCER + 1;
    if (warp == PRODUCER && lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO); }
    if (warp == ISSUER) { tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    griddep_wait();                                        // everything above ran beside the tail of the previous kernel
    const uint32_t tmem_S = tmem_base_s + Cfg::S_COL;
    const uint32_t tmem_O = tmem_base_s + Cfg::O_COL;

    if (warp == PRODUCER) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(Q_FULL), Cfg::Q_BYTES);
            for (int p = 0; p < Cfg::PANELS; ++p) tma_load_2d(sQ + p * Cfg::Q_PANEL_BYTES, &tmQ, bar(Q_FULL), p * 64, row0);
            for (int j = 0; j < nkv; ++j) {
                const int s = j % Cfg::STAGES, ph = (j / Cfg::STAGES) & 1;
                if constexpr (LEAN) {                       // K_{j-2} was read by S(j-2), whose commit is S_FULL of that tile
                    if (j >= 2 && !mbar_wait(bar(S_FULL + (j & 1)), ((j - 2) >> 1) & 1, &abort_flag)) break;
                } else {
                    if (!mbar_wait(bar(K_EMPTY + s), ph ^ 1, &abort_flag)) break;
                }
                mbar_expect_tx(bar(K_FULL + s), Cfg::KV_BYTES);
                for (int p = 0; p < Cfg::PANELS; ++p)
                    tma_load_2d(sK0 + s * Cfg::KV_BYTES + p * Cfg::KV_PANEL_BYTES, &tmK, bar(K_FULL + s), p * 64, kvrow0 + j * Cfg::BC);
                if constexpr (LEAN) {                       // V_{j-2} was read by P-bar V of tile j-2, issued before S(j-1): that commit covers it
                    if (j >= 2 && !mbar_wait(bar(S_FULL + ((j - 1) & 1)), ((j - 1) >> 1) & 1, &abort_flag)) break;
                } else {
                    if (!mbar_wait(bar(V_EMPTY + s), ph ^ 1, &abort_flag)) break;
                }
                if constexpr (FP8PV) {                      // one box: 64 keys (bytes) x d rows of the transposed V
                    mbar_expect_tx(bar(V_FULL + s), D * Cfg::BC);
                    tma_load_2d(sV0 + s * Cfg::KV_BYTES, &tmV, bar(V_FULL + s), j * Cfg::BC, (bh / prm.group) * D);
                } else {
                    mbar_expect_tx(bar(V_FULL + s), Cfg::KV_BYTES);
                    for (int p = 0; p < Cfg::PANELS; ++p)
                        tma_load_2d(sV0 + s * Cfg::KV_BYTES + p * Cfg::KV_PANEL_BYTES, &tmV, bar(V_FULL + s), p * 64, kvrow0 + j * Cfg::BC);
                }
            }
        }
        __syncwarp();
    } else if (warp == ISSUER) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_S = make_idesc_bf16(128, Cfg::BC, 0, 0);
            constexpr uint32_t idesc_PV = make_idesc_bf16(128, D, 0, 1);
            // descriptors are built once; inside the loops only the start-address field (low word, in
            // 16-byte units) moves, by compile-time constants per k-step plus the stage
            const uint64_t dQ0 = make_smem_desc(sQ, 16, 1024);
            const uint64_t dK0 = make_smem_desc(sK0, 16, 1024);
            const uint64_t dV0 = FP8PV ? make_smem_desc_sw64(sV0, 16, 512) : make_smem_desc(sV0, Cfg::KV_PANEL_BYTES, 1024);
            constexpr uint32_t idesc_PV8 = make_idesc_e4m3(128, D);
            // One score buffer (LEAN): the issuer's three waits and four commits per tile sit in the chain
            // softmax(j) -> P-bar V(j), S(j+1) -> softmax(j+1).  The two waits on TMA barriers are asked ahead of the wait for
            // P-bar (non-blocking test into a predicate, looked at later; a wait whose answer is used at once costs a
            // shared-memory round trip), and one commit per tile (after S(j+1)) tells the softmax warps and the producer
            // everything: it tracks every MMA issued before it.
            asm volatile(".reg .pred p_kfull, p_vfull;");
            auto issue_S = [&](int j, bool probed) -> bool {           // S(j) = Q K_j^T
                const int s = j % Cfg::STAGES, ph = (j / Cfg::STAGES) & 1;
                uint32_t ready = 0;
                if (LEAN && probed) asm volatile("selp.u32 %0, 1, 0, p_kfull;" : "=r"(ready));
                if (!ready && !mbar_wait(bar(K_FULL + s), ph, &abort_flag)) return false;
                tc_fence_after();
                const uint64_t dK = dK0 + static_cast<uint64_t>((s * Cfg::KV_BYTES) >> 4);
                const int sb = (Cfg::S_BUFS == 2) ? (j & 1) : 0;
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    mma_ss(tmem_S + sb * 64, dQ0 + (((k >> 2) * Cfg::Q_PANEL_BYTES + (k & 3) * 32) >> 4),
                           dK + (((k >> 2) * Cfg::KV_PANEL_BYTES + (k & 3) * 32) >> 4), idesc_S, k > 0);
                mma_commit(bar(S_FULL + (LEAN ? (j & 1) : sb)));
                if (!LEAN) mma_commit(bar(K_EMPTY + s));
                return true;
            };
            bool ok = mbar_wait(bar(Q_FULL), 0, &abort_flag);
            ok = ok && issue_S(0, false);
            if (Cfg::S_BUFS == 2 && nkv > 1) ok = ok && issue_S(1, false);
            for (int j = 0; ok && j < nkv; ++j) {
                const int s = j % Cfg::STAGES, ph = (j / Cfg::STAGES) & 1;
                const int sb = (Cfg::S_BUFS == 2) ? (j & 1) : 0, sph = (Cfg::S_BUFS == 2) ? ((j >> 1) & 1) : (j & 1);
                if constexpr (LEAN) {
                    asm volatile("mbarrier.test_wait.parity.shared::cta.b64 p_vfull, [%0], %1;"
                                 ::"r"(bar(V_FULL + s)), "r"(static_cast<uint32_t>(ph)) : "memory");
                    if (j + 1 < nkv)
                        asm volatile("mbarrier.test_wait.parity.shared::cta.b64 p_kfull, [%0], %1;"
                                     ::"r"(bar(K_FULL + (j + 1) % Cfg::STAGES)), "r"(static_cast<uint32_t>(((j + 1) / Cfg::STAGES) & 1)) : "memory");
                    ok = mbar_wait(bar(P_FULL + sb), sph, &abort_flag);
                    uint32_t v_ready;
                    asm volatile("selp.u32 %0, 1, 0, p_vfull;" : "=r"(v_ready));
                    ok = ok && (v_ready || mbar_wait(bar(V_FULL + s), ph, &abort_flag));
                } else {
                    ok = mbar_wait(bar(P_FULL + sb), sph, &abort_flag) && mbar_wait(bar(V_FULL + s), ph, &abort_flag);
                }
                if (Cfg::CORR) ok = ok && mbar_wait(bar(O_READY + (j & 1)), (j >> 1) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint64_t dV = dV0 + static_cast<uint64_t>((s * Cfg::KV_BYTES) >> 4);
                const uint32_t tP = tmem_S + sb * 64;
                // O-bar += P-bar(j) V_j: V_j as the B operand, N = d contiguous (MN-major), 16 key rows per step
                if constexpr (FP8PV) {
                    // 8-bit operands: 32 keys per step (8 TMEM columns of P-bar, 32 bytes along a row of V^T)
                    mma_ts_f8(tmem_O, tP, dV, idesc_PV8, (j > 0) ? 1u : 0u);
                    mma_ts_f8(tmem_O, tP + 8, dV + (32 >> 4), idesc_PV8, 1u);
                } else {
                    mma_ts(tmem_O, tP, dV, idesc_PV, (j > 0) ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < Cfg::BC / 16; ++k)
                        mma_ts(tmem_O, tP + k * 8, dV + ((k * 2048) >> 4), idesc_PV, 1u);
                }
                if constexpr (LEAN) {
                    if (j == nkv - 1) mma_commit(pv_done_bar(j));      // only the epilogue waits for it
                } else {
                    mma_commit(pv_done_bar(j));
                    mma_commit(bar(V_EMPTY + s));
                }
                // the next S for this buffer overwrites it; the MMAs just issued consume its P-bar(j) first
                if (j + Cfg::S_BUFS < nkv) ok = issue_S(j + Cfg::S_BUFS, true);
            }
        }
        __syncwarp();
    } else if (Cfg::CORR && warp >= Cfg::SOFTMAX_WARPS) {
        // ------------------------------------------------------------ correction (thread = query row): O-bar *= a
        const uint32_t tO = tmem_O + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row = tid & 127;
        for (int j = 0; j < nkv; ++j) {
            bool ok = mbar_wait(bar(A_FULL + (j & 1)), (j >> 1) & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const float a = sA[j & 1][row];
            // exact skip when no row of this warp moved its maximum; tile 0 starts the accumulator
            if (j > 0 && __any_sync(0xffffffffu, a != 1.0f)) {
                ok = __all_sync(0xffffffffu, mbar_wait(pv_done_bar(j - 1), pv_done_phase(j - 1), &abort_flag));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 64) {
                    uint32_t oa[32], ob[32];
                    tmem_ld32(tO + c0, oa);
                    tmem_ld32(tO + c0 + 32, ob);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) oa[c] = __float_as_uint(__uint_as_float(oa[c]) * a);
                    tmem_st32(tO + c0, oa);
#pragma unroll
                    for (int c = 0; c < 32; ++c) ob[c] = __float_as_uint(__uint_as_float(ob[c]) * a);
                    tmem_st32(tO + c0 + 32, ob);
                }
                tmem_wait_st();
                tc_fence_before();
            }
            mbar_arrive(bar(O_READY + (j & 1)));
        }
    } else {
        // ------------------------------------------------------------ softmax (thread = query row)
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        const uint32_t tS0 = tmem_S + lane_base, tO = tmem_O + lane_base;
        const int row = tid;                              // row inside the tile
        const float c_l2 = prm.scale * LOG2E;
        float m = -INFINITY, l = 0.0f;
        float r_run = -INFINITY;                          // guarded tie rule: largest tile maximum so far
        int n_ones = 0;
        bool ok = true;

        // One 64-key tile.  DIAG (compile time): the tile is partly masked; key column c of the tile is visible to
        // this row iff c <= vis.  Causal diagonal: vis = row - (first key of the tile - first query of the CTA).
        // Last tile of a sequence that ends inside it (full attention): vis = seqlen - 1 - first key, for every row.
        // MODE 1: the tie rule needs r_s only through "r_s > 1", i.e. whether the SECOND largest score of the tile also
        // lies within eps of the maximum (the test r_m - s <= eps is monotone in s, and it holds for the maximum itself).
        // So the maximum pass keeps the two largest raw scores (duplicates included) and no counting pass is needed.
        // (m1, m2) <- two largest of {m1, m2, x, y}
        auto top2 = [](float& m1, float& m2, float x, float y) {
            const float hi = fmaxf(x, y), lo = fminf(x, y);
            m2 = max3(m2, lo, fminf(m1, hi));
            m1 = fmaxf(m1, hi);
        };
        auto tile = [&](auto diag_tag, int j, int vis) -> bool {
            constexpr bool DIAG = decltype(diag_tag)::value;
            const int sb = (Cfg::S_BUFS == 2) ? (j & 1) : 0;
            const uint32_t tS = tS0 + sb * 64;
            float a;                                      // rescale factor of this tile, exp(m_old - m_new)
            if constexpr (Cfg::CHUNKED) {
                // The 64 scores of the row are read from TMEM once per pass, 32 at a time, instead of being kept in
                // registers: the kernel then fits the register budget of four CTAs per SM, and a TMEM load is cheap.
                uint32_t r[32];
                // ---- pass 1: row maximum of the raw accumulators (scale > 0 keeps the order)
                float mx = -INFINITY, mx2 = -INFINITY;          // mx2 (MODE 1): second largest
    #pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    tmem_ld32(tS + h * 32, r);
                    tmem_wait_ld();
                    if (MODE == 1) {
                        float a1 = -INFINITY, a2 = -INFINITY;
    #pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            float x[4];
    #pragma unroll
                            for (int e = 0; e < 4; ++e)
                                x[e] = (!DIAG || h * 32 + c + e <= vis) ? __uint_as_float(r[c + e]) : -INFINITY;
                            top2(mx, mx2, x[0], x[1]);
                            top2(a1, a2, x[2], x[3]);
                        }
                        mx2 = fmaxf(fminf(mx, a1), fmaxf(mx2, a2));
                        mx = fmaxf(mx, a1);
                    } else if (DIAG) {
    #pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (h * 32 + c <= vis) mx = fmaxf(mx, __uint_as_float(r[c]));
                    } else {
                        float m0 = mx, m1 = -INFINITY;
    #pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            m0 = max3(m0, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
                            m1 = max3(m1, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
                        }
                        mx = fmaxf(m0, m1);
                    }
                }
                mx *= prm.scale;
                if (MODE == 1) {
                    // tie rule of Algorithm 3 on the scaled scores of this key tile
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
                a = ex2((m - m_new) * LOG2E);     // m = -inf on the first tile gives a = 0; a = 1 when m stays
                const float negm = -m_new * LOG2E;
                // Argument of ex2 for two scores.  Standard mode: one packed FMA, acc * (scale log2 e) - m log2 e.  Stabilised
                // mode: the shifted maximum m = beta r_m can lie far above every score of the row, so the difference is taken
                // first, as Algorithm 3 writes it, t = acc * scale - m (one rounding), and t is then brought to base 2; the
                // error of the argument is then relative to |s - m| instead of |m|.
                auto exp_arg = [&](float& x0, float& x1, float a0, float a1) {
                    if (MODE == 1) {
                        fma2(x0, x1, a0, a1, prm.scale, -m_new);
                        mul2(x0, x1, x0, x1, LOG2E);
                    } else {
                        fma2(x0, x1, a0, a1, c_l2, negm);
                    }
                };
                m = m_new;
                // ---- last pass: P-bar = bf16(exp(S - m)) -> TMEM (over S); l += FP32 sum of the rounded values
                float sum0 = 0.0f, sum1 = 0.0f, sum2 = 0.0f, sum3 = 0.0f;
    #pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    tmem_ld32(tS + h * 32, r);
                    tmem_wait_ld();
                    if constexpr (FP8PV) {
                        uint32_t pk8[8];
    #pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            float x0, x1, x2, x3;
                            exp_arg(x0, x1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
                            exp_arg(x2, x3, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
                            float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                            if (DIAG) {
                                if (h * 32 + c > vis) p0 = 0.0f;
                                if (h * 32 + c + 1 > vis) p1 = 0.0f;
                                if (h * 32 + c + 2 > vis) p2 = 0.0f;
                                if (h * 32 + c + 3 > vis) p3 = 0.0f;
                            }
                            pk8[c >> 2] = pack_e4m3x4(p0, p1, p2, p3);
                            sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
                        }
                        // E4M3 P-bar columns [8h, 8h + 8) overlay score columns read in this or the earlier step
                        tmem_st8(tS + h * 8, pk8);
                    } else {
                    uint32_t pk[16];
    #pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        exp_arg(x0, x1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
                        float p0 = ex2(x0), p1 = ex2(x1);
                        if (DIAG) {
                            if (h * 32 + c > vis) p0 = 0.0f;
                            if (h * 32 + c + 1 > vis) p1 = 0.0f;
                        }
                        if (COUNT && prm.pbar_fmt) round_fp8x2(p0, p1, prm.pbar_fmt);   // diagnostic: FP8 P-bar
                        const uint32_t w = pack_bf16(p0, p1);
                        pk[c >> 1] = w;
                        if (COUNT) n_ones += ((w & 0xFFFFu) == 0x3F80u) + ((w >> 16) == 0x3F80u);
                        if ((c & 2) == 0) add_bf16x2_halves(sum0, sum1, w);
                        else              add_bf16x2_halves(sum2, sum3, w);
                    }
                    // P-bar columns [16h, 16h+16) overlay score columns [16h, 16h+16): for h = 0 those are in registers
                    // already; for h = 1 they are columns [16,32), read in the h = 0 step -- nothing still needed is lost
                    tmem_st16(tS + h * 16, pk);
                    }
                }
                l = a * l + ((sum0 + sum1) + (sum2 + sum3));
            } else {
                // all 64 scores of the row in registers
                uint32_t ra[32], rb[32];
                tmem_ld32(tS + 0, ra);
                tmem_ld32(tS + 32, rb);
                tmem_wait_ld();
                // ---- row maximum of the raw accumulators (scale > 0 keeps the order)
                float mx, mx2 = -INFINITY;                      // mx2 (MODE 1): second largest
                if (MODE == 1) {
                    float a1 = -INFINITY, a2 = -INFINITY;
                    mx = -INFINITY;
    #pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float x0 = (!DIAG || c <= vis) ? __uint_as_float(ra[c]) : -INFINITY;
                        const float x1 = (!DIAG || c + 1 <= vis) ? __uint_as_float(ra[c + 1]) : -INFINITY;
                        const float y0 = (!DIAG || 32 + c <= vis) ? __uint_as_float(rb[c]) : -INFINITY;
                        const float y1 = (!DIAG || 32 + c + 1 <= vis) ? __uint_as_float(rb[c + 1]) : -INFINITY;
                        top2(mx, mx2, x0, x1);
                        top2(a1, a2, y0, y1);
                    }
                    mx2 = fmaxf(fminf(mx, a1), fmaxf(mx2, a2));
                    mx = fmaxf(mx, a1);
                } else if (DIAG) {
                    mx = -INFINITY;
    #pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        if (c <= vis) mx = fmaxf(mx, __uint_as_float(ra[c]));
                        if (32 + c <= vis) mx = fmaxf(mx, __uint_as_float(rb[c]));
                    }
                } else {
                    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
    #pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        m0 = max3(m0, __uint_as_float(ra[c]), __uint_as_float(ra[c + 1]));
                        m1 = max3(m1, __uint_as_float(ra[c + 2]), __uint_as_float(ra[c + 3]));
                        m2 = max3(m2, __uint_as_float(rb[c]), __uint_as_float(rb[c + 1]));
                        m3 = max3(m3, __uint_as_float(rb[c + 2]), __uint_as_float(rb[c + 3]));
                    }
                    mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
                }
                mx *= prm.scale;
                if (MODE == 1) {
                    // tie rule of Algorithm 3 on the scaled scores of this key tile
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
                a = ex2((m - m_new) * LOG2E);     // m = -inf on the first tile gives a = 0; a = 1 when m stays
                const float negm = -m_new * LOG2E;
                // Argument of ex2 for two scores.  Standard mode: one packed FMA, acc * (scale log2 e) - m log2 e.  Stabilised
                // mode: the shifted maximum m = beta r_m can lie far above every score of the row, so the difference is taken
                // first, as Algorithm 3 writes it, t = acc * scale - m (one rounding), and t is then brought to base 2; the
                // error of the argument is then relative to |s - m| instead of |m|.
                auto exp_arg = [&](float& x0, float& x1, float a0, float a1) {
                    if (MODE == 1) {
                        fma2(x0, x1, a0, a1, prm.scale, -m_new);
                        mul2(x0, x1, x0, x1, LOG2E);
                    } else {
                        fma2(x0, x1, a0, a1, c_l2, negm);
                    }
                };
                m = m_new;
                if constexpr (Cfg::CORR) {                // the correction warps rescale O-bar under the exponential pass
                    sA[j & 1][row] = a;
                    mbar_arrive(bar(A_FULL + (j & 1)));
                }
                // ---- P-bar = bf16(exp(S - m)) -> TMEM (over S); l += FP32 sum of the rounded values
                float sum0 = 0.0f, sum1 = 0.0f, sum2 = 0.0f, sum3 = 0.0f;
                auto exp_chunk = [&](const uint32_t (&r)[32], int h) {
                    if constexpr (FP8PV) {
                        uint32_t pk8[8];
    #pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            float x0, x1, x2, x3;
                            exp_arg(x0, x1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
                            exp_arg(x2, x3, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
                            float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                            if (DIAG) {
                                if (h * 32 + c > vis) p0 = 0.0f;
                                if (h * 32 + c + 1 > vis) p1 = 0.0f;
                                if (h * 32 + c + 2 > vis) p2 = 0.0f;
                                if (h * 32 + c + 3 > vis) p3 = 0.0f;
                            }
                            pk8[c >> 2] = pack_e4m3x4(p0, p1, p2, p3);
                            sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
                        }
                        tmem_st8(tS + h * 8, pk8);
                    } else {
                    uint32_t pk[16];
    #pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        exp_arg(x0, x1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
                        float p0 = ex2(x0), p1 = ex2(x1);
                        if (DIAG) {
                            if (h * 32 + c > vis) p0 = 0.0f;
                            if (h * 32 + c + 1 > vis) p1 = 0.0f;
                        }
                        if (COUNT && prm.pbar_fmt) round_fp8x2(p0, p1, prm.pbar_fmt);   // diagnostic: FP8 P-bar
                        const uint32_t w = pack_bf16(p0, p1);
                        pk[c >> 1] = w;
                        if (COUNT) n_ones += ((w & 0xFFFFu) == 0x3F80u) + ((w >> 16) == 0x3F80u);
                        if ((c & 2) == 0) add_bf16x2_halves(sum0, sum1, w);
                        else              add_bf16x2_halves(sum2, sum3, w);
                    }
                    tmem_st16(tS + h * 16, pk);
                    }
                };
                exp_chunk(ra, 0);
                exp_chunk(rb, 1);
                l = a * l + ((sum0 + sum1) + (sum2 + sum3));
            }
            // ---- rescale O-bar when the maximum of any row of this warp moved, once P-bar V of tile j-1 is complete
            //      (one score buffer: S(j), which this thread has seen, was issued after it)
            if (!Cfg::CORR && j > 0 && __any_sync(0xffffffffu, a != 1.0f)) {
                if (Cfg::S_BUFS == 2) {                   // S(j) no longer implies that P-bar(j-1) V(j-1) has finished
                    if (!__all_sync(0xffffffffu, mbar_wait(pv_done_bar(j - 1), pv_done_phase(j - 1), &abort_flag))) return false;
                    tc_fence_after();
                }
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 64) {
                    uint32_t oa[32], ob[32];
                    tmem_ld32(tO + c0, oa);
                    if constexpr (Cfg::CHUNKED) {                 // one array live at a time
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) oa[c] = __float_as_uint(__uint_as_float(oa[c]) * a);
                        tmem_st32(tO + c0, oa);
                        tmem_ld32(tO + c0 + 32, ob);
                        tmem_wait_ld();
                    } else {
                        tmem_ld32(tO + c0 + 32, ob);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) oa[c] = __float_as_uint(__uint_as_float(oa[c]) * a);
                        tmem_st32(tO + c0, oa);
                    }
#pragma unroll
                    for (int c = 0; c < 32; ++c) ob[c] = __float_as_uint(__uint_as_float(ob[c]) * a);
                    tmem_st32(tO + c0 + 32, ob);
                }
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(P_FULL + sb));
            return true;
        };

        for (int j = 0; j < nkv; ++j) {
            ok = (Cfg::S_BUFS == 2 || LEAN) ? mbar_wait(bar(S_FULL + (j & 1)), (j >> 1) & 1, &abort_flag)
                                            : mbar_wait(bar(S_FULL), j & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (CAUSAL && j >= 2 * i)                         ok = tile(std::true_type{}, j, row - (j - 2 * i) * Cfg::BC);
            else if (PADDED && (j + 1) * Cfg::BC > seqlen)      ok = tile(std::true_type{}, j, seqlen - 1 - j * Cfg::BC);
            else                                              ok = tile(std::false_type{}, j, 0);
            if (!ok) break;
        }
        // ---- epilogue: O-bar -> BF16, O = bf16(O-bar / l), L = m + log l
        if (ok) {
            ok = mbar_wait(pv_done_bar(nkv - 1), LEAN ? 0u : pv_done_phase(nkv - 1), &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float rl = __frcp_rn(l);
            // the Q tile is no longer needed: stage the O tile there in the same swizzled panel layout
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tO + c0, r);
                tmem_wait_ld();
                if constexpr (COUNT) {
                    if (prm.o_f32) {                              // the output that skips both BF16 roundings (Sec. 3.2)
                        float4* dst = reinterpret_cast<float4*>(prm.o_f32 + (static_cast<size_t>(row0) + row) * D + c0);
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            dst[c >> 2] = make_float4(__fdiv_rn(__uint_as_float(r[c]), l), __fdiv_rn(__uint_as_float(r[c + 1]), l),
                                                      __fdiv_rn(__uint_as_float(r[c + 2]), l), __fdiv_rn(__uint_as_float(r[c + 3]), l));
                    }
                }
                uint32_t out[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float o0 = __uint_as_float(r[c]), o1 = __uint_as_float(r[c + 1]);
                    if constexpr (FP8PV) { o0 *= prm.v_descale; o1 *= prm.v_descale; }
                    if (!prm.single_rounding) {                   // O-bar -> BF16 (the paper's rounding point)
                        const uint32_t ob = pack_bf16(o0, o1);
                        o0 = bf16_lo(ob);
                        o1 = bf16_hi(ob);
                    }
                    out[c >> 1] = pack_bf16(div_rn(o0, l, rl), div_rn(o1, l, rl));
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int c16 = (c0 >> 3) + v, panel = c16 >> 3, cc = c16 & 7;
                    sts128(sQ + panel * Cfg::Q_PANEL_BYTES + row * 128 + ((cc ^ (row & 7)) << 4),
                           out[4 * v], out[4 * v + 1], out[4 * v + 2], out[4 * v + 3]);
                }
            }
            prm.lse[static_cast<size_t>(row0) + row] = m + lg2(l) * LN2;
            if (COUNT && prm.ones) prm.ones[static_cast<size_t>(row0) + row] = n_ones;
            fence_proxy_async_smem();
            mbar_arrive(bar(EPI));
            if (tid == 0) {
                if (mbar_wait(bar(EPI), 0, &abort_flag)) {
                    for (int p = 0; p < Cfg::PANELS; ++p) tma_store_2d(&tmO, sQ + p * Cfg::Q_PANEL_BYTES, p * 64, row0);
                    tma_store_commit_and_wait();
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    if (abort_flag) {
        // let copies that are still in flight land before shared memory is released
        for (int t = 0; t < 64; ++t) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == ISSUER) tmem_dealloc(tmem_base_s, Cfg::TMEM_COLS);
    if (tid == 0 && abort_flag) atomicExch(prm.status, 1);
}

}  // namespace attn
