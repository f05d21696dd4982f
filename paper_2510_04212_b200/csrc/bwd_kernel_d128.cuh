// Backward main kernel for head width 128: Algorithm 2, one CTA per 128-row key tile j of one (batch, head),
// looping over the query tiles i that see it.
//
// Per (i, j) pair, five tcgen05 MMAs (FP32 accumulators in TMEM), on the transposes so that a thread owns a key row:
//   S^T  = K_j Q_i^T     dP^T = V_j dO_i^T     dV += P^T dO_i     dK += dS^T Q_i     dQ_i = dS K_j
// TMEM has 512 columns and dV, dK take 256 of them at this head width, so the rest is shared:
//   S^T [0,128) (P^T, BF16, is written over parts of it) | dP^T, then dQ [128,256) | dV [256,384) | dK [384,512).
// That aliasing fixes the order of the tensor work.  The compute warps take a pair in two halves, each with its own
// barrier pair, so that the tensor pipe works behind them:
//   first half   wait S^T(i):  P^T = bf16(exp(S^T - L)) over the S^T columns, the unrounded p kept in registers
//                -> issuer: dV(i), then S^T(i+1) (dV is the last reader of P^T; the pipe runs them in order)
//   second half  wait dP^T(i): dS^T = bf16(p (dP^T - delta)) into shared memory
//                -> issuer: dQ(i), dK(i), then, once the drain warps have read dQ(i) out of the shared columns, dP^T(i+1)
// P^T is placed over S^T columns that the writing thread has already loaded: the 16 packed columns of queries
// [32c, 32c+32) go to S^T columns [32c, 32c+16) (c = 0..3), and the dV product addresses its eight
// 16-query steps there.
//
// dQ: the FP32 accumulator in global memory is private to the backward pass and keeps the layout of the staging
// buffer (128-row tile, 32-column panel, row, swizzled 16-byte chunk), so a staged panel goes out as one contiguous
// 16 KB bulk reduce-add.  An SM's reduce-adds drain at 30-50 GB/s whichever instruction issues them (measured), i.e.
// 1.3-2.2 us for the 64 KB of a pair: that stream bounds the kernel, so the two staging panels alternate and the next
// one is written while the previous one is being read.  `dq_convert_tiled128_kernel` undoes the layout.
//
// Warps: 0-7 compute (thread = key row x 64 query columns: warps 0-3 take query columns [0,64), warps 4-7
// [64,128)); 8-11 drain (dQ tile: TMEM -> staging panels, 32 columns at a time; three of the four panels of a pair
// wait in registers, so that the shared columns are released after one staging step); 12 TMA producer (K, V once; Q_i through a
// two-stage ring so that S^T of the next pair can be queued early; dO_i single-buffered, reloaded as soon as dV has
// run); 13 MMA issuer; 14 staging consumer (bulk reduce-add of the staged panels into the FP32 accumulator: scattered
// red.global instructions from the drain warps cost 0.95 ms of 2.46 ms on B=2,H=16,N=8192).  dV and scale * dK are
// written by the compute warps at the end.
//
// Rounding: P = bf16(exp(S - L)) feeds dV; dS = bf16(p32 (dP - delta)) feeds dQ and dK; all three
// gradients accumulate in FP32 and are rounded to BF16 once; scale is applied in FP32.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "ptx.cuh"
#include "bwd_kernel.cuh"

namespace attn {

struct Bwd128Cfg {
    static constexpr int D = 128;
    static constexpr int PANEL_BYTES = 128 * 128;                 // 128 rows x 64 BF16
    static constexpr int TILE_BYTES = 2 * PANEL_BYTES;            // 128 rows x 128 BF16: two 64-column panels
    static constexpr int QS = 2;                                  // Q ring depth (dO: one buffer)
    static constexpr int X_BYTES = 2 * PANEL_BYTES;               // dS^T [128 keys][128 queries] BF16
    static constexpr int STG_BYTES = 2 * PANEL_BYTES;             // dQ staging: two [128][32] FP32 panels, used in turn
    // K | V | Q x2 | dO | X | staging | barriers, per-query vectors, flags: all dynamic, 227 KB in total
    static constexpr int TILES_BYTES = (3 + QS) * TILE_BYTES + X_BYTES + STG_BYTES;
    static constexpr int MISC_BYTES = 2432;
    static constexpr int SMEM_BYTES = 232448;
    static_assert(TILES_BYTES + MISC_BYTES <= SMEM_BYTES, "shared memory budget");
    static constexpr int TMEM_COLS = 512;
    static constexpr int ST_COL = 0, DP_COL = 128, DQ_COL = 128, DV_COL = 256, DK_COL = 384;
    static constexpr int THREADS = 480;
};

// GENERAL (compile time): the instantiation for grouped query heads and / or a sequence that ends inside a tile
template <bool CAUSAL, bool GENERAL>
__global__ void __launch_bounds__(480, 1)
attn_bwd_kernel_d128(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                     const __grid_constant__ CUtensorMap tmdK, const __grid_constant__ CUtensorMap tmdV,
                     const BwdParams prm)
{
    using namespace ptx;
    using Cfg = Bwd128Cfg;
    constexpr int D = 128;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    if (sm + Cfg::TILES_BYTES + Cfg::MISC_BYTES > smem_raw + Cfg::SMEM_BYTES) {   // never expected: the base is aligned
        if (threadIdx.x == 0) atomicExch(prm.status, 2);
        return;
    }
    const uint32_t sK = smem_u32(sm);
    const uint32_t sV = sK + Cfg::TILE_BYTES;
    const uint32_t sQ0 = sV + Cfg::TILE_BYTES;                    // QS stages
    const uint32_t sdO = sQ0 + Cfg::QS * Cfg::TILE_BYTES;
    const uint32_t sX = sdO + Cfg::TILE_BYTES;
    const uint32_t sStg = sX + Cfg::X_BYTES;

    enum { KV_FULL = 0, Q_FULL = 1, Q_EMPTY = 3, DO_FULL = 5, DO_EMPTY = 6, S_FULL = 7, P_FULL = 8, DQ_FULL = 9,
           DQ_EMPTY = 10, DKV_DONE = 11, VEC_FULL = 12, STG_FULL = 14, STG_FREE = 16, DP_FULL = 18, DS_FULL = 19,
           NBARS = 20 };
    uint8_t* misc = sm + Cfg::TILES_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(misc);                           // NBARS x 8 bytes (256 reserved)
    float (*sNegL)[128] = reinterpret_cast<float (*)[128]>(misc + 256);           // [2][128]: -L * log2(e) per query of the tile
    float (*sDelta)[128] = reinterpret_cast<float (*)[128]>(misc + 256 + 1024);   // [2][128]: -delta
    // (both written by bulk copies from the vectors the preprocess kernel left in the tile's part of the dQ buffer)
    uint32_t& tmem_base_s = *reinterpret_cast<uint32_t*>(misc + 2304);
    int& abort_flag = *reinterpret_cast<int*>(misc + 2308);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Causal: key tile 0 sees the most query tiles, so the tile 0 of several heads first (longest jobs first) -- of
    // as many heads as keep their tensors and FP32 dQ accumulators in L2 together (the host chooses the group;
    // B=2,H=16,N=8192: all 32 heads at once 1.43 ms, groups of 4 to 8 heads 1.35-1.37 ms).  Full attention: every job
    // is the same size; walk head by head.
    int bh, j;
    if (CAUSAL) {
        // groups of prm.head_group heads, inside a group key tile 0 of all its heads first, ...
        const int hg = prm.head_group;
        const int grp = blockIdx.x / (hg * prm.Tr), rem = blockIdx.x % (hg * prm.Tr);
        const int gsz = min(hg, prm.BH - grp * hg);              // the last group may be smaller
        bh = grp * hg + rem % gsz;
        j = rem / gsz;
    } else {
        bh = blockIdx.x / prm.Tr;
        j = blockIdx.x % prm.Tr;
    }
    const int i0 = CAUSAL ? j : 0;
    int seqlen = prm.seqlen, Tr = prm.Tr;
    griddep_launch_dependents();
    if (GENERAL && prm.seqlens) {                // per-sequence lengths: a key tile of padding has nothing to do
        griddep_wait();                          // (the lengths may come from the kernel before this one)
        seqlen = min(max(prm.seqlens[bh / prm.Hkv], 0), prm.N);
        Tr = (seqlen + 127) / 128;
        if (j >= Tr) return;
    }
    const int nqh = Tr - i0;                     // query tiles per query head
    const int nq = nqh * prm.group;              // pairs of this key tile: the group's query heads one after the other
    const int kvrow0 = bh * prm.N + j * 128;
    // first row of a pair's Q / dO / dQ tile in the [B*H*N, d] view; (qh, ii) = query head inside the group, query tile
    // offset inside the head, stepped along with `it` (no division in the loops)
    auto pair_row = [&](int qh, int ii) { return (bh * prm.group + qh) * prm.N + (i0 + ii) * 128; };

    auto bar = [&](int b) { return smem_u32(&bars[b]); };

    if (tid == 0) {
        for (int b = 0; b < NBARS; ++b) {
            uint32_t cnt = 1;
            if (b == P_FULL || b == DS_FULL) cnt = 256;
            if (b == DQ_EMPTY || b == STG_FULL || b == STG_FULL + 1) cnt = 128;
            mbar_init(bar(b), cnt);
        }
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 12 && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmdO);
        tma_prefetch_desc(&tmdK); tma_prefetch_desc(&tmdV);
    }
    if (warp == 13) { tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    griddep_wait();                              // everything above ran beside the tail of the previous kernel
    const uint32_t tmem = tmem_base_s;

    if (warp == 12) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(KV_FULL), 2 * Cfg::TILE_BYTES);
            for (int p = 0; p < 2; ++p) {
                tma_load_2d(sK + p * Cfg::PANEL_BYTES, &tmK, bar(KV_FULL), p * 64, kvrow0);
                tma_load_2d(sV + p * Cfg::PANEL_BYTES, &tmV, bar(KV_FULL), p * 64, kvrow0);
            }
            for (int it = 0, qh = 0, ii = 0; it < nq; ++it, qh += (ii + 1 == nqh), ii = (ii + 1 == nqh) ? 0 : ii + 1) {
                const int st = it % Cfg::QS, ph = (it / Cfg::QS) & 1;
                const int qrow = pair_row(qh, ii);
                if (!mbar_wait_relaxed(bar(Q_EMPTY + st), ph ^ 1, &abort_flag)) break;
                mbar_expect_tx(bar(Q_FULL + st), Cfg::TILE_BYTES);
                for (int p = 0; p < 2; ++p)
                    tma_load_2d(sQ0 + st * Cfg::TILE_BYTES + p * Cfg::PANEL_BYTES, &tmQ, bar(Q_FULL + st), p * 64, qrow);
                {   // per-query vectors of this pair, into the buffer the compute warps used two pairs ago: free, because the
                    // Q stage just waited for was released behind dK of that pair, which followed the compute warps' work on it
                    const int vb = it & 1;
                    const uint8_t* vec = reinterpret_cast<const uint8_t*>(prm.dq) + static_cast<size_t>(qrow >> 7) * (128 * D * 2);
                    mbar_expect_tx(bar(VEC_FULL + vb), 1024);
                    bulk_load_1d(smem_u32(&sNegL[vb][0]), vec + VEC_NEGL_OFFSET, 512, bar(VEC_FULL + vb));
                    bulk_load_1d(smem_u32(&sDelta[vb][0]), vec + VEC_NDELTA_OFFSET, 512, bar(VEC_FULL + vb));
                }
                if (!mbar_wait(bar(DO_EMPTY), (it & 1) ^ 1, &abort_flag)) break;       // dV of the previous pair has run
                mbar_expect_tx(bar(DO_FULL), Cfg::TILE_BYTES);
                for (int p = 0; p < 2; ++p)
                    tma_load_2d(sdO + p * Cfg::PANEL_BYTES, &tmdO, bar(DO_FULL), p * 64, qrow);
            }
        }
        __syncwarp();
    } else if (warp == 13) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_T = make_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T: both operands K-major
            constexpr uint32_t idesc_KN = make_idesc_bf16(128, D, 0, 1);    // dV, dK: A K-major (or TMEM), B MN-major
            constexpr uint32_t idesc_NN = make_idesc_bf16(128, D, 1, 1);    // dQ: A MN-major, B MN-major
            // descriptors: only the start-address field (low word, 16-byte units) changes in the loops
            const uint64_t dK_k = make_smem_desc(sK, 16, 1024), dV_k = make_smem_desc(sV, 16, 1024);
            const uint64_t dK_mn = make_smem_desc(sK, Cfg::PANEL_BYTES, 1024);
            const uint64_t dQ_k0 = make_smem_desc(sQ0, 16, 1024), dQ_mn0 = make_smem_desc(sQ0, Cfg::PANEL_BYTES, 1024);
            const uint64_t ddO_k = make_smem_desc(sdO, 16, 1024), ddO_mn = make_smem_desc(sdO, Cfg::PANEL_BYTES, 1024);
            const uint64_t dX_k = make_smem_desc(sX, 16, 1024), dX_mn = make_smem_desc(sX, Cfg::PANEL_BYTES, 1024);
            // K-major operand with 128 columns: k-step k lies in panel k / 4 at byte (k % 4) * 32 of the row
            auto koff = [](int k) { return static_cast<uint64_t>(((k >> 2) * Cfg::PANEL_BYTES + (k & 3) * 32) >> 4); };
            auto issue_S = [&](uint64_t so) {
#pragma unroll
                for (int k = 0; k < 8; ++k) mma_ss(tmem + Cfg::ST_COL, dK_k + koff(k), dQ_k0 + so + koff(k), idesc_T, k > 0);
            };
            auto issue_dP = [&]() {
#pragma unroll
                for (int k = 0; k < 8; ++k) mma_ss(tmem + Cfg::DP_COL, dV_k + koff(k), ddO_k + koff(k), idesc_T, k > 0);
            };
            bool ok = mbar_wait(bar(KV_FULL), 0, &abort_flag) && mbar_wait(bar(Q_FULL), 0, &abort_flag) &&
                      mbar_wait(bar(DO_FULL), 0, &abort_flag);
            if (ok) {
                tc_fence_after();
                issue_S(0);
                mma_commit(bar(S_FULL));
                issue_dP();
                mma_commit(bar(DP_FULL));
            }
            for (int it = 0; ok && it < nq; ++it) {
                const int st = it % Cfg::QS;
                const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
                ok = mbar_wait(bar(P_FULL), it & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                // dV += P^T dO_i : A = P^T in TMEM (queries [32c, 32c+32) at S^T columns [32c, 32c+16)), B = dO_i MN-major.
                // It is the last reader of dO_i, whose buffer is reloaded for the next pair behind it.
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    mma_ts(tmem + Cfg::DV_COL, tmem + Cfg::ST_COL + (k >> 1) * 32 + (k & 1) * 8,
                           ddO_mn + ((k * 2048) >> 4), idesc_KN, (it > 0 || k > 0) ? 1u : 0u);
                mma_commit(bar(DO_EMPTY));
                const bool more = it + 1 < nq;
                const int st1 = (it + 1) % Cfg::QS, ph1 = ((it + 1) / Cfg::QS) & 1;
                if (more) {
                    // S^T of the next pair: behind dV in the pipe, which was the last reader of P^T
                    ok = mbar_wait(bar(Q_FULL + st1), ph1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_S(static_cast<uint64_t>((st1 * Cfg::TILE_BYTES) >> 4));
                    mma_commit(bar(S_FULL));
                }
                ok = mbar_wait(bar(DS_FULL), it & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                // dQ_i = dS K_j : A = dS^T read as (M = query, K = key), MN-major; B = K_j MN-major.  Into the dP^T columns,
                // which the compute warps have consumed.
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    mma_ss(tmem + Cfg::DQ_COL, dX_mn + ((k * 2048) >> 4), dK_mn + ((k * 2048) >> 4), idesc_NN, k > 0);
                mma_commit(bar(DQ_FULL));
                // dK += dS^T Q_i : A = dS^T rows (queries contiguous, K-major), B = Q_i MN-major
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    mma_ss(tmem + Cfg::DK_COL, dX_k + koff(k), dQ_mn0 + so + ((k * 2048) >> 4), idesc_KN, (it > 0 || k > 0) ? 1u : 0u);
                mma_commit(bar(Q_EMPTY + st));                    // Q_i and dS^T are free after everything queued so far
                if (more) {
                    // dP^T of the next pair: dQ(i) must have left the shared columns, dO_{i+1} must have landed.  It completes
                    // behind dK(i), so the compute warps may overwrite dS^T once they see it.
                    ok = mbar_wait(bar(DQ_EMPTY), it & 1, &abort_flag) && mbar_wait(bar(DO_FULL), (it + 1) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_dP();
                    mma_commit(bar(DP_FULL));
                }
            }
            if (ok) mma_commit(bar(DKV_DONE));
        }
        __syncwarp();
    } else if (warp == 14) {
        // ------------------------------------------------------------ staging consumer: staged dQ panels -> FP32 accumulator
        // The accumulator keeps the staging layout (tile, 32-column panel, row, swizzled 16-byte chunk), so a panel is one
        // contiguous 16 KB reduce-add.  An SM's reduce-adds drain at about 30-50 GB/s: this loop is what bounds the kernel,
        // so the two panels alternate and the next one is staged while the previous one is being read.
        if (lane == 0) {
            int n = 0;
            bool ok = true;
            for (int it = 0, qh = 0, ii = 0; ok && it < nq; ++it, qh += (ii + 1 == nqh), ii = (ii + 1 == nqh) ? 0 : ii + 1) {
                float* tile = prm.dq_acc + static_cast<size_t>(pair_row(qh, ii)) * D;
                for (int pnl = 0; pnl < 4; ++pnl, ++n) {
                    const int b = n & 1;
                    ok = mbar_wait_relaxed(bar(STG_FULL + b), (n >> 1) & 1, &abort_flag);
                    if (!ok) break;
                    bulk_reduce_add_f32(tile + pnl * (Cfg::PANEL_BYTES / 4), sStg + b * Cfg::PANEL_BYTES, Cfg::PANEL_BYTES);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    if (n > 0) {                                  // the previous panel has been read: its buffer is free
                        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        mbar_arrive(bar(STG_FREE + (b ^ 1)));
                    }
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all reduce-adds performed before exit
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ------------------------------------------------------------ drain (thread = query row of the dQ tile)
        const int r = tid - 256;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        int n = 0;                                                // panels staged so far; panel n uses buffer n & 1
        // one [128 rows][32 floats = 128 bytes] panel, 128-byte swizzle
        auto stage = [&](const uint32_t (&x)[32]) -> bool {
            const int b = n & 1;
            if (n >= 2) {                                         // the reduce-add of panel n - 2 must have read this buffer
                bool ok = mbar_wait_relaxed(bar(STG_FREE + b), ((n >> 1) - 1) & 1, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return false;
            }
#pragma unroll
            for (int c = 0; c < 8; ++c)
                sts128(sStg + b * Cfg::PANEL_BYTES + r * 128 + ((c ^ (r & 7)) << 4), x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]);
            fence_proxy_async_smem();
            mbar_arrive(bar(STG_FULL + b));
            ++n;
            return true;
        };
        for (int it = 0; it < nq; ++it) {
            bool ok = mbar_wait_relaxed(bar(DQ_FULL), it & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t a[32], b[32], c[32];
            tmem_ld32(tmem + Cfg::DQ_COL + lane_base, a);
            tmem_ld32(tmem + Cfg::DQ_COL + lane_base + 32, b);
            tmem_ld32(tmem + Cfg::DQ_COL + lane_base + 64, c);
            tmem_wait_ld();
            if (!stage(a)) break;
            tmem_ld32(tmem + Cfg::DQ_COL + lane_base + 96, a);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(DQ_EMPTY));                           // everything is in registers: dP^T of the next pair may be written
            if (!stage(b)) break;
            if (!stage(c)) break;
            if (!stage(a)) break;
        }
    } else {
        // ------------------------------------------------------------ compute (thread = key row x 64 query columns)
        const int half = warp >> 2;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const float c_l2 = prm.scale * LOG2E;
        bool ok = true;
        for (int it = 0, ii = 0; it < nq; ++it, ii = (ii + 1 == nqh) ? 0 : ii + 1) {
            const int buf = it & 1;
            ok = mbar_wait(bar(VEC_FULL + buf), (it >> 1) & 1, &abort_flag) && mbar_wait(bar(S_FULL), it & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            // DIAG (compile time): a partly masked pair: the causal diagonal (first query tile of a query head: key row r
            // sees query column q only if r <= q), key rows or query columns beyond the sequence length.  Key row r sees the
            // query columns q with qlo <= q < qlo + span.
            const bool diag = CAUSAL && ii == 0;
            const int kvalid = GENERAL ? seqlen - j * 128 : 128;
            const int qvalid = GENERAL ? seqlen - (i0 + ii) * 128 : 128;
            const bool edge = diag || (GENERAL && (kvalid < 128 || qvalid < 128));
            const int qlo = (GENERAL && r >= kvalid) ? 128 : (diag ? r : 0);
            const unsigned span = (qvalid > qlo) ? static_cast<unsigned>(qvalid - qlo) : 0u;
            const int qb = half * 64;                             // first query column of this thread
            float p[64];                                          // unrounded probabilities: kept for dS
            // ---- first half of the pair: P^T = exp(S^T - L), rounded to BF16 over the S^T columns just read
            auto exp_phase = [&](auto diag_tag) {
                constexpr bool DIAG = decltype(diag_tag)::value;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int q0 = qb + h * 32;
                    uint32_t sacc[32];
                    tmem_ld32(tmem + Cfg::ST_COL + lane_base + q0, sacc);
                    tmem_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 nl = lds128f(smem_u32(&sNegL[buf][0]) + (q0 + c) * 4);
                        const float nlv[4] = {nl.x, nl.y, nl.z, nl.w};
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {          // packed FP32 pairs: half the issue slots
                            float x0, x1;
                            fma2v(x0, x1, __uint_as_float(sacc[c + e]), __uint_as_float(sacc[c + e + 1]), c_l2, nlv[e], nlv[e + 1]);
                            float p0 = ex2(x0), p1 = ex2(x1);
                            if (DIAG) {                                                // masked entries: P = 0
                                p0 = (static_cast<unsigned>(q0 + c + e - qlo) < span) ? p0 : 0.0f;
                                p1 = (static_cast<unsigned>(q0 + c + e + 1 - qlo) < span) ? p1 : 0.0f;
                            }
                            p[h * 32 + c + e] = p0;
                            p[h * 32 + c + e + 1] = p1;
                        }
                        pk[(c >> 1)] = pack_bf16(p[h * 32 + c], p[h * 32 + c + 1]);
                        pk[(c >> 1) + 1] = pack_bf16(p[h * 32 + c + 2], p[h * 32 + c + 3]);
                    }
                    // P^T of these 32 queries over the first 16 of the S^T columns just read
                    tmem_st16(tmem + Cfg::ST_COL + lane_base + q0, pk);
                }
            };
            if (edge) exp_phase(std::true_type{});
            else      exp_phase(std::false_type{});
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(P_FULL));                             // dV(i) and S^T(i+1) run behind the second half
            // ---- second half: dS^T = P o (dP^T - delta), rounded to BF16, into shared memory for dQ and dK
            ok = mbar_wait(bar(DP_FULL), it & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            auto ds_phase = [&](auto diag_tag) {
                constexpr bool DIAG = decltype(diag_tag)::value;
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const int q0 = qb + h * 16;
                    uint32_t dpacc[16];
                    tmem_ld16(tmem + Cfg::DP_COL + lane_base + q0, dpacc);
                    tmem_wait_ld();
                    uint32_t dsk[8];
#pragma unroll
                    for (int c = 0; c < 16; c += 4) {
                        const float4 dl = lds128f(smem_u32(&sDelta[buf][0]) + (q0 + c) * 4);
                        const float dlv[4] = {dl.x, dl.y, dl.z, dl.w};
                        float ds[4];
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            mul_sum2(ds[e], ds[e + 1], p[h * 16 + c + e], p[h * 16 + c + e + 1], __uint_as_float(dpacc[c + e]),
                                     __uint_as_float(dpacc[c + e + 1]), dlv[e], dlv[e + 1]);   // dlv holds -delta
                            if (GENERAL && DIAG) {                                     // dS = 0 whatever the padding holds
                                ds[e] = (static_cast<unsigned>(q0 + c + e - qlo) < span) ? ds[e] : 0.0f;
                                ds[e + 1] = (static_cast<unsigned>(q0 + c + e + 1 - qlo) < span) ? ds[e + 1] : 0.0f;
                            }
                        }
                        dsk[(c >> 1)] = pack_bf16(ds[0], ds[1]);
                        dsk[(c >> 1) + 1] = pack_bf16(ds[2], ds[3]);
                    }
                    // dS^T row r, queries [q0, q0+16): two 16-byte chunks of panel `half`, 128-byte swizzle
#pragma unroll
                    for (int q2 = 0; q2 < 2; ++q2) {
                        const int cc = h * 2 + q2;
                        sts128(sX + half * Cfg::PANEL_BYTES + r * 128 + ((cc ^ (r & 7)) << 4), dsk[4 * q2], dsk[4 * q2 + 1], dsk[4 * q2 + 2], dsk[4 * q2 + 3]);
                    }
                }
            };
            if (edge) ds_phase(std::true_type{});
            else      ds_phase(std::false_type{});
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(DS_FULL));
        }
        // ---- dV (warps 0-3) and scale * dK (warps 4-7) -> BF16 -> the two Q stages (free now: every MMA has completed
        // and nothing more is loaded), in the layout of a loaded tile -> TMA stores
        if (ok) {
            ok = mbar_wait(bar(DKV_DONE), 0, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float mul = half ? prm.scale : 1.0f;
            uint8_t* out = sm + (2 + half) * Cfg::TILE_BYTES;                 // Q stage `half`
            const uint32_t src = tmem + (half ? Cfg::DK_COL : Cfg::DV_COL) + lane_base;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t a[32];
                tmem_ld32(src + c0, a);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(a[8 * v + 0]) * mul, __uint_as_float(a[8 * v + 1]) * mul);
                    o.y = pack_bf16(__uint_as_float(a[8 * v + 2]) * mul, __uint_as_float(a[8 * v + 3]) * mul);
                    o.z = pack_bf16(__uint_as_float(a[8 * v + 4]) * mul, __uint_as_float(a[8 * v + 5]) * mul);
                    o.w = pack_bf16(__uint_as_float(a[8 * v + 6]) * mul, __uint_as_float(a[8 * v + 7]) * mul);
                    const int chunk = ((c0 & 63) >> 3) + v;                   // 16-byte chunk inside the 128-byte panel row
                    sts128(smem_u32(out) + (c0 >> 6) * Cfg::PANEL_BYTES + r * 128 + ((chunk ^ (r & 7)) << 4), o.x, o.y, o.z, o.w);
                }
            }
            fence_proxy_async_smem();
        }
        // the four warps of this half meet here whatever happened before (every path of the loop above ends here); a
        // wait that gave up has set abort_flag, and then nothing is stored
        if (half) asm volatile("bar.sync 2, 128;" ::: "memory");
        else      asm volatile("bar.sync 1, 128;" ::: "memory");
        if ((warp & 3) == 0 && lane == 0 && !abort_flag) {
            const uint32_t s_out = sQ0 + half * Cfg::TILE_BYTES;
            const CUtensorMap* tm = half ? &tmdK : &tmdV;
            tma_store_2d(tm, s_out, 0, kvrow0);
            tma_store_2d(tm, s_out + Cfg::PANEL_BYTES, 64, kvrow0);
            tma_store_commit_and_wait();                                      // shared memory read before the CTA exits
        }
    }

    // ---------------------------------------------------------------- teardown
    if (abort_flag) {
        for (int t = 0; t < 64; ++t) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 13) tmem_dealloc(tmem_base_s, Cfg::TMEM_COLS);
    if (tid == 0 && abort_flag) atomicExch(prm.status, 1);
}

}  // namespace attn
