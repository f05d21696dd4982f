// Backward main kernel for head width 64: Algorithm 2 as a persistent, warp-specialised kernel.
//
// Work item = one 128-row key tile j of one (batch, head) together with the query tiles i that see it.
// One CTA per SM walks a static list of items (heaviest first, dealt out in snake order); all roles keep
// running across item boundaries, so the loads, the first MMAs and the output stores of neighbouring
// items overlap instead of adding a prologue and a tail per item.
//
// Per (i, j) pair, five tcgen05 MMAs (FP32 accumulators in TMEM):
//   group A   S^T  = K_j Q_i^T     dP^T = V_j dO_i^T
//   group B   dV  += P^T dO_i      dK  += dS^T Q_i      dQ_i = dS K_j
// TMEM (512 columns): S^T [0,128) | dP^T [128,256) | P^T (BF16) [256,320) | dV [320,384) |
// dK [384,448) | dQ [448,512).  The compute warps release S^T / dP^T as soon as they have loaded them
// into registers (half way through their work on the pair), so A of the next pair runs under the second
// half; P^T has its own columns and dS^T is double-buffered in shared memory.
//
// Warps: 0-7 compute (thread = key row x 64 query columns: warps 0-3 take query columns [0,64), warps 4-7
// [64,128)); 8-11 drain (dQ tiles and, once per item, dV / dK: TMEM -> shared-memory staging; also the
// final dQ conversion described below); 12 TMA producer; 13 and 14 MMA issuers (13: group A and dV,
// 14: dK and dQ; one thread issues about one MMA per 100 clocks, the tensor pipe retires one in 50-70);
// 15 staging consumer (TMA reduce-add of dQ tiles into the FP32 accumulator in global memory, TMA stores
// of dV / dK, arrival counting).
//
// dQ leaves the kernel finished: the first 32-bit word of every 128-row dQ output tile serves as an
// arrival counter (cleared by the preprocess kernel) until the tile is written.  After its reduce-adds
// for query tile i are complete, a CTA increments that counter; the CTA that brings it to the number of
// key tiles that see tile i reads the FP32 accumulator tile back from L2, scales it, rounds to BF16 and
// writes the output tile (counter word included).  No CTA waits for another one.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "ptx.cuh"
#include "bwd_kernel.cuh"

namespace attn {

struct Bwd64Cfg {
    static constexpr int D = 64;
    static constexpr int TILE_BYTES = 128 * 128;                  // 128 rows x 64 BF16
    static constexpr int X_BYTES = 2 * TILE_BYTES;                // dS^T [128 keys][128 queries] BF16, two panels
    static constexpr int QS = 3;                                  // Q / dO ring depth
    static constexpr int STG_BYTES = 2 * TILE_BYTES;              // staging: dQ as two [128][32] FP32 panels, or dV | dK
    // K | V | Q x3 | dO x3 | X x2 | staging | barriers, per-query vectors, flags
    static constexpr int TILES_BYTES = (2 + 2 * QS) * TILE_BYTES + 2 * X_BYTES + STG_BYTES;
    static constexpr int MISC_BYTES = 2432;
    // Everything lives in dynamic shared memory (the kernel has no static shared memory), so that the tiles start
    // on a 1024-byte boundary with little or no padding: the total is the 227 KB a CTA can have.
    static constexpr int SMEM_BYTES = 232448;
    static_assert(TILES_BYTES + MISC_BYTES <= SMEM_BYTES, "shared memory budget");
    static constexpr int TMEM_COLS = 512;
    static constexpr int ST_COL = 0, DP_COL = 128, PT_COL = 256, DV_COL = 320, DK_COL = 384, DQ_COL = 448;
    static constexpr int THREADS = 512;
};

// The w-th work item of this CTA.  Items are numbered heaviest first (n = j * BH + bh: key tile 0 sees the most
// query tiles under the causal mask) and dealt to the CTAs in snake order, which evens out the totals.
struct BwdItem {
    int bh, j, i0, nq, nqh;   // nqh: query tiles per query head; nq = nqh * group: all (query head, query tile) pairs
    int seqlen, Tr;           // sequence length of the item's batch element and its tile count
};
// The pairs of an item: the query heads of the group one after the other, each with its nqh query tiles.  Position
// kept incrementally (no division in the loops).
// GENERAL (compile time): the instantiation for grouped query heads (more than one query head per key/value head)
// and / or a sequence that ends inside a tile; without it the position is just the pair count and only the causal
// diagonal is masked.
template <bool GENERAL>
struct BwdPairPos {
    int ii = 0, qh = 0;                                   // query tile offset inside the head, query head inside the group
    __device__ __forceinline__ void next(const BwdItem& item) {
        ++ii;
        if (GENERAL && ii == item.nqh) { ii = 0; ++qh; }
    }
    // first row of the pair's Q / dO / dQ tile in the [B*H*N, d] view
    __device__ __forceinline__ int row(const BwdItem& item, const BwdParams& prm) const {
        return (GENERAL ? item.bh * prm.group + qh : item.bh) * prm.N + (item.i0 + ii) * 128;
    }
};
// The next work item of this CTA.  `e` is the CTA's cursor into the static enumeration (start at 0; advanced here).
// With per-sequence lengths (GENERAL and prm.seqlens) the key tiles that hold only padding are skipped, so the cursor
// can advance by more than one; every role walks the same sequence.
template <bool CAUSAL, bool GENERAL>
__device__ __forceinline__ bool bwd_item(int& e, const BwdParams& prm, BwdItem& item)
{
    const int G = static_cast<int>(gridDim.x), c = static_cast<int>(blockIdx.x);
    while (true) {
        const int n = e * G + ((e & 1) ? (G - 1 - c) : c);
        if (n >= prm.Tr * prm.BH) return false;
        ++e;
        // causal: heaviest key tiles first; full attention: head by head (the head's FP32 dQ accumulator stays in L2)
        item.bh = CAUSAL ? n % prm.BH : n / prm.Tr;
        item.j = CAUSAL ? n / prm.BH : n % prm.Tr;
        item.i0 = CAUSAL ? item.j : 0;
        item.seqlen = prm.seqlen;
        item.Tr = prm.Tr;
        if (GENERAL && prm.seqlens) {
            item.seqlen = min(max(prm.seqlens[item.bh / prm.Hkv], 0), prm.N);
            item.Tr = (item.seqlen + 127) / 128;
            if (item.j >= item.Tr) continue;              // a key tile of padding
        }
        item.nqh = item.Tr - item.i0;
        item.nq = item.nqh * prm.group;
        return true;
    }
}

// dQ tile t = bf16(scale * accumulator tile): 32 KB read from L2, 16 KB written, by the 128 drain threads (r = 0..127).
// Out of line: it runs about once per work item and is called from three places.
__device__ __noinline__ void bwd64_finish_tile(const float* dq_acc, uint16_t* dq, float sc, int t, int r)
{
    constexpr int D = 64;
    const float4* src = reinterpret_cast<const float4*>(dq_acc + static_cast<size_t>(t) * 128 * D);
    uint4* dst = reinterpret_cast<uint4*>(dq + static_cast<size_t>(t) * 128 * D);
#pragma unroll
    for (int k0 = 0; k0 < 8; k0 += 4) {
        float4 a[4], b[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int idx = (k0 + k) * 128 + r;
            a[k] = __ldcg(src + 2 * idx);
            b[k] = __ldcg(src + 2 * idx + 1);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint4 o;
            o.x = ptx::pack_bf16(a[k].x * sc, a[k].y * sc);
            o.y = ptx::pack_bf16(a[k].z * sc, a[k].w * sc);
            o.z = ptx::pack_bf16(b[k].x * sc, b[k].y * sc);
            o.w = ptx::pack_bf16(b[k].z * sc, b[k].w * sc);
            dst[(k0 + k) * 128 + r] = o;
        }
    }
}

template <bool CAUSAL, bool GENERAL>
__global__ void __launch_bounds__(512, 1)
attn_bwd_kernel_d64(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                    const __grid_constant__ CUtensorMap tmdK, const __grid_constant__ CUtensorMap tmdV,
                    const __grid_constant__ CUtensorMap tmAcc, const BwdParams prm)
{
    using namespace ptx;
    using Cfg = Bwd64Cfg;
    constexpr int D = 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    if (sm + Cfg::TILES_BYTES + Cfg::MISC_BYTES > smem_raw + Cfg::SMEM_BYTES) {   // never expected: the base is aligned
        if (threadIdx.x == 0) atomicExch(prm.status, 2);
        return;
    }
    const uint32_t sK = smem_u32(sm);
    const uint32_t sV = sK + Cfg::TILE_BYTES;
    const uint32_t sQ0 = sV + Cfg::TILE_BYTES;                    // QS stages
    const uint32_t sdO0 = sQ0 + Cfg::QS * Cfg::TILE_BYTES;        // QS stages
    const uint32_t sX0 = sdO0 + Cfg::QS * Cfg::TILE_BYTES;        // two buffers
    const uint32_t sStg = sX0 + 2 * Cfg::X_BYTES;
    uint8_t* sX_ptr = sm + (2 + 2 * Cfg::QS) * Cfg::TILE_BYTES;
    uint8_t* sStg_ptr = sX_ptr + 2 * Cfg::X_BYTES;

    // Barriers.  g = running pair count of this CTA (over all its items), w = running item count, n = running
    // staging step count (one per pair plus one per item).  Unless noted, a barrier completes one phase per g.
    //   K_FULL, V_FULL (per w)      TMA landed                          K_FREE (per w, 2 commits), V_FREE (per w): MMAs done reading
    //   QDO_FULL / QDO_EMPTY [QS]   Q_i, dO_i ring (EMPTY: both issuers' commits)
    //   SDP_FULL                    A(g) done                           SDP_FREE: compute warps hold S^T, dP^T of g in registers
    //   PDS_FULL [2]                P^T in TMEM, dS^T in X[g & 1]       PT_FREE: dV(g) done; X_FREE [2]: dK(g), dQ(g) done
    //   DQ_FULL / DQ_EMPTY          dQ tile in TMEM / read by the drain
    //   DKV_DONE (per w, 2 commits) dV, dK of the item complete         DKV_FREE (per w): read by the drain
    //   STG_FULL / STG_FREE (per n) staging written / read by TMA       VEC_FULL [2]: per-query vectors of g landed (bulk copies)
    //   FIN                         last arrival verdicts written
    // PDS_FULL and X_FREE exist once per dS^T buffer (index = g & 1): issuer 14 may run up to two pairs behind the
    // compute warps (it also waits for the drain), which a single barrier's phase parity could not tell apart.
    enum { K_FULL = 0, V_FULL = 1, K_FREE = 2, V_FREE = 3, QDO_FULL = 4, QDO_EMPTY = 7, SDP_FULL = 10, SDP_FREE = 11,
           PDS_FULL = 12, PT_FREE = 14, X_FREE = 15, DQ_FULL = 17, DQ_EMPTY = 18, DKV_DONE = 19, DKV_FREE = 20,
           STG_FULL = 21, STG_FREE = 22, VEC_FULL = 23, FIN = 25, NBARS = 26 };
    uint8_t* misc = sm + Cfg::TILES_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(misc);                           // NBARS x 8 bytes (256 reserved)
    float (*sNegL)[128] = reinterpret_cast<float (*)[128]>(misc + 256);           // [2][128]: -L * log2(e) per query of the tile
    float (*sDelta)[128] = reinterpret_cast<float (*)[128]>(misc + 256 + 1024);   // [2][128]: -delta
    // (both written by bulk copies from the vectors the preprocess kernel left in the tile's part of the dQ buffer)
    uint32_t& tmem_base_s = *reinterpret_cast<uint32_t*>(misc + 2304);
    int& abort_flag = *reinterpret_cast<int*>(misc + 2308);
    int* s_final = reinterpret_cast<int*>(misc + 2312);           // [8]: dQ tile to finish (global tile index, -1: none), by n & 7
    static_assert(NBARS * 8 <= 256 && 2312 + 32 <= Cfg::MISC_BYTES, "misc layout");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    griddep_launch_dependents();
    auto bar = [&](int b) { return smem_u32(&bars[b]); };

    if (tid == 0) {
        for (int b = 0; b < NBARS; ++b) {
            uint32_t cnt = 1;
            if (b == SDP_FREE || b == PDS_FULL || b == PDS_FULL + 1) cnt = 256;
            if (b == DQ_EMPTY || b == STG_FULL || b == DKV_FREE) cnt = 128;
            if ((b >= QDO_EMPTY && b < QDO_EMPTY + Cfg::QS) || b == DKV_DONE || b == K_FREE) cnt = 2;   // both MMA issuers
            mbar_init(bar(b), cnt);
        }
        abort_flag = 0;
        for (int k = 0; k < 8; ++k) s_final[k] = -1;
        fence_mbar_init();
    }
    if (warp == 12 && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmdO);
        tma_prefetch_desc(&tmdK); tma_prefetch_desc(&tmdV); tma_prefetch_desc(&tmAcc);
    }
    if (warp == 13) { tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    griddep_wait();                                        // everything above ran beside the tail of the previous kernel
    const uint32_t tmem = tmem_base_s;
    BwdItem item;

    if (warp == 12) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            int g = 0;
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                const int kvrow0 = item.bh * prm.N + item.j * 128;
                // V is free once the last A of the previous item has run, K only after its last dQ: V, the first
                // Q / dO pair, then K
                if (w > 0) ok = mbar_wait_relaxed_ool(bar(V_FREE), (w - 1) & 1, &abort_flag);
                if (!ok) break;
                mbar_expect_tx(bar(V_FULL), Cfg::TILE_BYTES);
                tma_load_2d(sV, &tmV, bar(V_FULL), 0, kvrow0);
                BwdPairPos<GENERAL> pos;
                for (int it = 0; it < item.nq; ++it, ++g, pos.next(item)) {
                    const int st = g % Cfg::QS, ph = (g / Cfg::QS) & 1;
                    ok = mbar_wait_relaxed_ool(bar(QDO_EMPTY + st), ph ^ 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(QDO_FULL + st), 2 * Cfg::TILE_BYTES);
                    const int qrow = pos.row(item, prm);
                    tma_load_2d(sQ0 + st * Cfg::TILE_BYTES, &tmQ, bar(QDO_FULL + st), 0, qrow);
                    tma_load_2d(sdO0 + st * Cfg::TILE_BYTES, &tmdO, bar(QDO_FULL + st), 0, qrow);
                    {   // per-query vectors of this pair, into the buffer the compute warps used two pairs ago
                        const int vb = g & 1;
                        if (g >= 2) ok = mbar_wait_relaxed_ool(bar(PDS_FULL + vb), ((g - 2) >> 1) & 1, &abort_flag);
                        if (!ok) break;
                        const uint8_t* vec = reinterpret_cast<const uint8_t*>(prm.dq) + static_cast<size_t>(qrow >> 7) * (128 * D * 2);
                        mbar_expect_tx(bar(VEC_FULL + vb), 1024);
                        bulk_load_1d(smem_u32(&sNegL[vb][0]), vec + VEC_NEGL_OFFSET, 512, bar(VEC_FULL + vb));
                        bulk_load_1d(smem_u32(&sDelta[vb][0]), vec + VEC_NDELTA_OFFSET, 512, bar(VEC_FULL + vb));
                    }
                    if (it == 0) {
                        if (w > 0) ok = mbar_wait_relaxed_ool(bar(K_FREE), (w - 1) & 1, &abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(bar(K_FULL), Cfg::TILE_BYTES);
                        tma_load_2d(sK, &tmK, bar(K_FULL), 0, kvrow0);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 13) {
        // ------------------------------------------------------------ MMA issuer 1: group A and dV
        if (lane == 0) {
            constexpr uint32_t idesc_T = make_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T: both operands K-major
            constexpr uint32_t idesc_KN = make_idesc_bf16(128, D, 0, 1);    // dV: A from TMEM, B MN-major
            // descriptors: only the start-address field (low word, 16-byte units) changes in the loops
            const uint64_t dK_k = make_smem_desc(sK, 16, 1024);             // K_j, K-major (rows of d)
            const uint64_t dV_k = make_smem_desc(sV, 16, 1024);
            const uint64_t dQ_k0 = make_smem_desc(sQ0, 16, 1024);
            const uint64_t ddO_k0 = make_smem_desc(sdO0, 16, 1024);
            const uint64_t ddO_mn0 = make_smem_desc(sdO0, Cfg::TILE_BYTES, 1024);

            // group A of pair gn; `last`: it is the last pair of its item (V and, for this issuer, K are free after it)
            auto issue_A = [&](int gn, bool last) -> bool {
                const int st = gn % Cfg::QS, ph = (gn / Cfg::QS) & 1;
                if (!mbar_wait_ool(bar(QDO_FULL + st), ph, &abort_flag)) return false;
                tc_fence_after();
                const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    mma_ss(tmem + Cfg::DP_COL, dV_k + ((k * 32) >> 4), ddO_k0 + so + ((k * 32) >> 4), idesc_T, k > 0);
                if (last) mma_commit(bar(V_FREE));
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    mma_ss(tmem + Cfg::ST_COL, dK_k + ((k * 32) >> 4), dQ_k0 + so + ((k * 32) >> 4), idesc_T, k > 0);
                mma_commit(bar(SDP_FULL));
                if (last) mma_commit(bar(K_FREE));
                return true;
            };

            // One code copy of group A and one of dV (instruction-cache footprint): the loop walks the pairs with a
            // one-pair lookahead; step g issues A(g + 1) and dV(g).  Within an item A(g + 1) goes first (as soon as
            // the compute warps hold S^T, dP^T of pair g in registers); across an item boundary dV(g) goes first,
            // because the next item's K arrives only after this item's last dQ.
            bool ok = true;
            BwdItem nxt;
            int wn = 0, itn = 0;                          // position of pair g + 1
            int en = 0;                                   // enumeration cursor of the lookahead
            bool have_n = bwd_item<CAUSAL, GENERAL>(en, prm, nxt);
            int wc = 0, itc = 0, nqc = 0;                 // position of pair g
            for (int g = -1; ok; ++g) {
                const int a_phase = (have_n && itn != 0) ? 0 : 1;
#pragma unroll 1
                for (int phase = 0; ok && phase < 2; ++phase) {
                    if (phase == a_phase) {
                        if (!have_n) continue;
                        if (g >= 0) ok = mbar_wait_ool(bar(SDP_FREE), g & 1, &abort_flag);
                        if (ok && itn == 0)
                            ok = mbar_wait_ool(bar(V_FULL), wn & 1, &abort_flag) &&
                                 mbar_wait_ool(bar(K_FULL), wn & 1, &abort_flag);
                        ok = ok && issue_A(g + 1, itn == nxt.nq - 1);
                    } else {
                        if (g < 0) continue;
                        ok = mbar_wait_ool(bar(PDS_FULL + (g & 1)), (g >> 1) & 1, &abort_flag);
                        if (ok && itc == 0 && wc > 0) ok = mbar_wait_ool(bar(DKV_FREE), (wc - 1) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const int st = g % Cfg::QS;
                        const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
                        // dV += P^T dO_i : A = P^T in TMEM, B = dO_i with d contiguous (MN-major), 16 queries per step
                        mma_ts(tmem + Cfg::DV_COL, tmem + Cfg::PT_COL, ddO_mn0 + so, idesc_KN, (itc > 0) ? 1u : 0u);
#pragma unroll
                        for (int k = 1; k < 8; ++k)
                            mma_ts(tmem + Cfg::DV_COL, tmem + Cfg::PT_COL + k * 8, ddO_mn0 + so + ((k * 2048) >> 4), idesc_KN, 1u);
                        mma_commit(bar(PT_FREE));
                        mma_commit(bar(QDO_EMPTY + st));
                        if (itc == nqc - 1) mma_commit(bar(DKV_DONE));
                    }
                }
                if (!have_n) break;
                wc = wn; itc = itn; nqc = nxt.nq;
                if (++itn == nxt.nq) { itn = 0; ++wn; have_n = bwd_item<CAUSAL, GENERAL>(en, prm, nxt); }
            }
        }
        __syncwarp();
    } else if (warp == 14) {
        // ------------------------------------------------------------ MMA issuer 2: dK and dQ
        if (lane == 0) {
            constexpr uint32_t idesc_KN = make_idesc_bf16(128, D, 0, 1);    // dK: A K-major, B MN-major
            constexpr uint32_t idesc_NN = make_idesc_bf16(128, D, 1, 1);    // dQ: A MN-major, B MN-major
            const uint64_t dK_mn = make_smem_desc(sK, Cfg::TILE_BYTES, 1024);    // K_j as [key][d], MN-major B
            const uint64_t dQ_mn0 = make_smem_desc(sQ0, Cfg::TILE_BYTES, 1024);
            const uint64_t dX_k0 = make_smem_desc(sX0, 16, 1024);           // dS^T rows (queries contiguous): K-major A
            const uint64_t dX_mn0 = make_smem_desc(sX0, Cfg::TILE_BYTES, 1024);  // same bytes as (M = query, K = key): MN-major A
            bool ok = true;
            int g = 0;
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                const int nq = item.nq;
                ok = mbar_wait_ool(bar(K_FULL), w & 1, &abort_flag);
                for (int it = 0; ok && it < nq; ++it, ++g) {
                    const int st = g % Cfg::QS, ph = (g / Cfg::QS) & 1;
                    ok = mbar_wait_ool(bar(PDS_FULL + (g & 1)), (g >> 1) & 1, &abort_flag) &&
                         mbar_wait_ool(bar(QDO_FULL + st), ph, &abort_flag);
                    if (ok && it == 0 && w > 0) ok = mbar_wait_ool(bar(DKV_FREE), (w - 1) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
                    const uint64_t xo = static_cast<uint64_t>(((g & 1) * Cfg::X_BYTES) >> 4);
                    // dK += dS^T Q_i : A = dS^T rows (K-major: 4 steps per 64-query panel), B = Q_i MN-major
                    mma_ss(tmem + Cfg::DK_COL, dX_k0 + xo, dQ_mn0 + so, idesc_KN, (it > 0) ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < 8; ++k)
                        mma_ss(tmem + Cfg::DK_COL, dX_k0 + xo + (((k >> 2) * Cfg::TILE_BYTES + (k & 3) * 32) >> 4),
                               dQ_mn0 + so + ((k * 2048) >> 4), idesc_KN, 1u);
                    if (g > 0) {
                        ok = mbar_wait_ool(bar(DQ_EMPTY), (g - 1) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    // dQ_i = dS K_j : A = the same dS^T buffer read as (M = query, K = key), B = K_j MN-major
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tmem + Cfg::DQ_COL, dX_mn0 + xo + ((k * 2048) >> 4), dK_mn + ((k * 2048) >> 4), idesc_NN, k > 0);
                    mma_commit(bar(DQ_FULL));
                    mma_commit(bar(X_FREE + (g & 1)));                    // this dS^T buffer has been read
                    mma_commit(bar(QDO_EMPTY + st));
                    if (it == nq - 1) {
                        mma_commit(bar(DKV_DONE));
                        mma_commit(bar(K_FREE));
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 15) {
        // ------------------------------------------------------------ staging consumer: TMA out of the staging buffer, arrival counts
        if (lane == 0) {
            // Arrival counting, two steps behind the TMA issue so that neither the completion of the reduce-adds nor
            // the atomic's round trip holds up the next staging step:
            //   step n, after its STG_FREE arrival:  (1) the atomic issued in step n-1 (for step n-2) has returned by now:
            //   turn it into the verdict on step n-2;  (2) the bulk group of step n-1 is the only older one: wait for it,
            //   then issue the atomic for step n-1 without touching its result.
            // The atomic releases this CTA's completed reduce-adds; the CTA that brings a tile's counter to the number
            // of key tiles that see the tile acquires the others' and finishes the tile.
            bool ok = true;
            int n = 0;
            int prev_t = -1, prev_i = 0, prev_Tr = 0;             // dQ tile of step n-1 (-1: it was a dV / dK step)
            int pend_t = -1;                                      // dQ tile of step n-2 whose atomic is in flight (-1: none)
            unsigned pend_old = 0, pend_expected = 0;
            auto settle = [&]() {
                if (n >= 2) {
                    int verdict = -1;
                    if (pend_t >= 0 && pend_old + 1 == pend_expected) { fence_acq_rel_gpu(); verdict = pend_t; }
                    s_final[(n - 2) & 7] = verdict;
                }
                if (n >= 1) {
                    asm volatile("cp.async.bulk.wait_group 1;" ::: "memory");
                    pend_t = prev_t;
                    if (prev_t >= 0) {
                        pend_expected = CAUSAL ? static_cast<unsigned>(prev_i + 1) : static_cast<unsigned>(prev_Tr);
                        pend_old = atom_add_release_gpu(
                            reinterpret_cast<unsigned*>(prm.dq + static_cast<size_t>(prev_t) * 128 * D), 1u);
                    }
                }
            };
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                BwdPairPos<GENERAL> pos;
                for (int it = 0; it < item.nq; ++it, pos.next(item)) {
                    ok = mbar_wait_relaxed_ool(bar(STG_FULL), n & 1, &abort_flag);
                    if (!ok) break;
                    const int i = item.i0 + pos.ii;
                    const int qrow = pos.row(item, prm);
                    tma_reduce_add_2d(&tmAcc, sStg, 0, qrow);                         // columns [0,32)
                    tma_reduce_add_2d(&tmAcc, sStg + Cfg::TILE_BYTES, 32, qrow);      // columns [32,64)
                    tma_store_commit_and_wait();                  // staging read; the adds complete asynchronously
                    mbar_arrive(bar(STG_FREE));
                    settle();
                    prev_t = qrow >> 7;
                    prev_i = i;
                    prev_Tr = item.Tr;
                    ++n;
                }
                if (!ok) break;
                ok = mbar_wait_relaxed_ool(bar(STG_FULL), n & 1, &abort_flag);
                if (!ok) break;
                const int kvrow0 = item.bh * prm.N + item.j * 128;
                tma_store_2d(&tmdV, sStg, 0, kvrow0);
                tma_store_2d(&tmdK, sStg + Cfg::TILE_BYTES, 0, kvrow0);
                tma_store_commit_and_wait();
                mbar_arrive(bar(STG_FREE));
                settle();
                prev_t = -1;
                ++n;
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // everything written before exit
            if (ok) {                                             // verdicts on the last two steps
                settle();
                ++n;
                prev_t = -1;
                settle();
            }
            mbar_arrive(bar(FIN));
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ------------------------------------------------------------ drain (thread = row of the dQ / dV / dK tile)
        const int r = tid - 256;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        auto finish_tile = [&](int t) { bwd64_finish_tile(prm.dq_acc, prm.dq, prm.scale, t, r); };
        bool ok = true;
        int g = 0, n = 0;
        // Before writing the staging buffer in step n: the previous TMA must have read it.  The staging consumer
        // wrote the verdict on step n-4 before that STG_FREE arrival and rewrites the slot only after the STG_FULL
        // arrivals of later steps: read it here, use it after the stores.
        auto staging_ready = [&](int& fi) -> bool {
            bool o = true;
            if (n > 0) o = mbar_wait_relaxed_ool(bar(STG_FREE), (n - 1) & 1, &abort_flag);
            o = __all_sync(0xffffffffu, o);
            fi = (o && n >= 4) ? s_final[(n - 4) & 7] : -1;
            return o;
        };
        for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
            for (int it = 0; it < item.nq; ++it, ++g, ++n) {
                ok = mbar_wait_relaxed_ool(bar(DQ_FULL), g & 1, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t a[32], b[32];
                tmem_ld32(tmem + Cfg::DQ_COL + lane_base, a);
                tmem_ld32(tmem + Cfg::DQ_COL + lane_base + 32, b);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(DQ_EMPTY));                       // the dQ columns may be overwritten
                int fi;
                ok = staging_ready(fi);
                if (!ok) break;
                // two [128 rows][32 floats = 128 bytes] panels, 128-byte swizzle
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    *reinterpret_cast<uint4*>(sStg_ptr + r * 128 + ((c ^ (r & 7)) << 4)) =
                        make_uint4(a[4 * c], a[4 * c + 1], a[4 * c + 2], a[4 * c + 3]);
                    *reinterpret_cast<uint4*>(sStg_ptr + Cfg::TILE_BYTES + r * 128 + ((c ^ (r & 7)) << 4)) =
                        make_uint4(b[4 * c], b[4 * c + 1], b[4 * c + 2], b[4 * c + 3]);
                }
                fence_proxy_async_smem();
                mbar_arrive(bar(STG_FULL));
                if (fi >= 0) finish_tile(fi);
            }
            if (!ok) break;
            // ---- dV and scale * dK of the item -> BF16 -> staging (dV | dK, [128 rows][64 BF16], 128-byte swizzle)
            ok = mbar_wait_relaxed_ool(bar(DKV_DONE), w & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            int fi;
            ok = staging_ready(fi);
            if (!ok) break;
#pragma unroll
            for (int t = 0; t < 2; ++t) {                         // t = 0: dV, t = 1: scale * dK
                const float mul = t ? prm.scale : 1.0f;
                uint8_t* stage = sStg_ptr + t * Cfg::TILE_BYTES + r * 128;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t a[32];
                    tmem_ld32(tmem + (t ? Cfg::DK_COL : Cfg::DV_COL) + lane_base + c0, a);
                    tmem_wait_ld();
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(a[8 * v + 0]) * mul, __uint_as_float(a[8 * v + 1]) * mul);
                        o.y = pack_bf16(__uint_as_float(a[8 * v + 2]) * mul, __uint_as_float(a[8 * v + 3]) * mul);
                        o.z = pack_bf16(__uint_as_float(a[8 * v + 4]) * mul, __uint_as_float(a[8 * v + 5]) * mul);
                        o.w = pack_bf16(__uint_as_float(a[8 * v + 6]) * mul, __uint_as_float(a[8 * v + 7]) * mul);
                        const int cc = (c0 >> 3) + v;
                        *reinterpret_cast<uint4*>(stage + ((cc ^ (r & 7)) << 4)) = o;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(DKV_FREE));                           // the next item may start new dV, dK accumulators
            fence_proxy_async_smem();
            mbar_arrive(bar(STG_FULL));
            if (fi >= 0) finish_tile(fi);
            ++n;
        }
        // the verdicts of the last four staging steps
        if (ok) {
            ok = mbar_wait_relaxed_ool(bar(FIN), 0, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
#pragma unroll 1
            for (int s = (n > 4 ? n - 4 : 0); s < n; ++s) {
                const int fi = s_final[s & 7];
                if (fi >= 0) finish_tile(fi);
            }
        }
    } else {
        // ------------------------------------------------------------ compute (thread = key row x 64 query columns)
        const int half = warp >> 2;                               // which 64 query columns
        const int r = (warp & 3) * 32 + lane;                     // key row of the tile
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const float c_l2 = prm.scale * LOG2E;
        bool ok = true;
        int g = 0;
        for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
            int ii = 0;                                           // query tile offset inside the current query head
            for (int it = 0; it < item.nq; ++it, ++g, ii = (GENERAL && ii + 1 == item.nqh) ? 0 : ii + 1) {
                const int buf = g & 1;
                ok = mbar_wait_ool(bar(VEC_FULL + buf), (g >> 1) & 1, &abort_flag) && mbar_wait_ool(bar(SDP_FULL), g & 1, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint8_t* xrow = sX_ptr + buf * Cfg::X_BYTES + half * Cfg::TILE_BYTES + r * 128;
                // the pair on the causal diagonal: key row r sees query column q only if r <= q.  One copy of the arithmetic
                // for both kinds of pair (instruction-cache footprint); the mask sits behind a CTA-uniform branch.
                // Partly masked pairs: the causal diagonal (key row r sees query column q only if r <= q), key rows and query
                // columns beyond the sequence length.  Key row r of the tile sees the query columns q with qlo <= q < qlo + span.
                const bool diag = CAUSAL && ii == 0;             // first query tile of a query head
                const int kvalid = GENERAL ? item.seqlen - item.j * 128 : 128;
                const int qvalid = GENERAL ? item.seqlen - (item.i0 + ii) * 128 : 128;
                const bool edge = diag || (GENERAL && (kvalid < 128 || qvalid < 128));
                const int qlo = (GENERAL && r >= kvalid) ? 128 : (diag ? r : 0);
                const unsigned span = (qvalid > qlo) ? static_cast<unsigned>(qvalid - qlo) : 0u;
                {
// not unrolled: the two chunks share one copy of the arithmetic (the unrolled loop body no longer fitted the
                    // instruction cache next to the other roles' code: 6 % slower)
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        const int q0 = half * 64 + h * 32;            // first query column of this chunk
                        uint32_t sacc[32], dpacc[32];
                        tmem_ld32(tmem + Cfg::ST_COL + lane_base + q0, sacc);
                        tmem_ld32(tmem + Cfg::DP_COL + lane_base + q0, dpacc);
                        tmem_wait_ld();
                        if (h == 1) {                                 // S^T, dP^T of this pair are in registers: A of the next pair may run
                            tc_fence_before();
                            mbar_arrive(bar(SDP_FREE));
                        }
                        uint32_t pk[16], dsk[16];
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 nl = *reinterpret_cast<const float4*>(&sNegL[buf][q0 + c]);
                            const float4 dl = *reinterpret_cast<const float4*>(&sDelta[buf][q0 + c]);
                            const float nlv[4] = {nl.x, nl.y, nl.z, nl.w}, dlv[4] = {dl.x, dl.y, dl.z, dl.w};
                            float p[4], ds[4];
#pragma unroll
                            for (int e = 0; e < 4; e += 2) {          // packed FP32 pairs: half the issue slots
                                float x0, x1;
                                fma2v(x0, x1, __uint_as_float(sacc[c + e]), __uint_as_float(sacc[c + e + 1]), c_l2, nlv[e], nlv[e + 1]);
                                p[e] = ex2(x0);
                                p[e + 1] = ex2(x1);
                                if (edge) {                                                    // masked entries: P = 0
                                    p[e] = (static_cast<unsigned>(q0 + c + e - qlo) < span) ? p[e] : 0.0f;
                                    p[e + 1] = (static_cast<unsigned>(q0 + c + e + 1 - qlo) < span) ? p[e + 1] : 0.0f;
                                }
                                mul_sum2(ds[e], ds[e + 1], p[e], p[e + 1], __uint_as_float(dpacc[c + e]),
                                         __uint_as_float(dpacc[c + e + 1]), dlv[e], dlv[e + 1]);   // dlv holds -delta
                                if (GENERAL && edge) {                                         // ... and dS = 0 whatever the padding holds
                                    ds[e] = (static_cast<unsigned>(q0 + c + e - qlo) < span) ? ds[e] : 0.0f;
                                    ds[e + 1] = (static_cast<unsigned>(q0 + c + e + 1 - qlo) < span) ? ds[e + 1] : 0.0f;
                                }
                            }
                            pk[(c >> 1)] = pack_bf16(p[0], p[1]);
                            pk[(c >> 1) + 1] = pack_bf16(p[2], p[3]);
                            dsk[(c >> 1)] = pack_bf16(ds[0], ds[1]);
                            dsk[(c >> 1) + 1] = pack_bf16(ds[2], ds[3]);
                        }
                        if (h == 0) {
                            // first write of this pair into P^T and dS^T: dV of pair g-1 and dK, dQ of pair g-2 must have
                            // read them (they ran under the arithmetic above)
                            if (g > 0) ok = mbar_wait_ool(bar(PT_FREE), (g - 1) & 1, &abort_flag);
                            if (ok && g > 1) ok = mbar_wait_ool(bar(X_FREE + buf), ((g >> 1) - 1) & 1, &abort_flag);
                        }
                        tmem_st16(tmem + Cfg::PT_COL + lane_base + (q0 >> 1), pk);
                        // dS^T row r, 32 queries: four 16-byte chunks of this half's panel, 128-byte swizzle
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const int cc = h * 4 + q4;
                            *reinterpret_cast<uint4*>(xrow + ((cc ^ (r & 7)) << 4)) =
                                make_uint4(dsk[4 * q4], dsk[4 * q4 + 1], dsk[4 * q4 + 2], dsk[4 * q4 + 3]);
                        }
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;                                   // a wait gave up: the abort flag is set, every role unwinds
                tmem_wait_st();
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(bar(PDS_FULL + buf));
            }
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
