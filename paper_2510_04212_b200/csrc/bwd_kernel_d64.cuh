// Backward main kernel for head width 64: Algorithm 2 as a persistent, warp-specialised kernel.
//
// Work item = one 128-row key tile j of one (batch, head) together with the query tiles i that see it.
// One CTA per SM walks a static list of items (heaviest first, dealt out in snake order); all roles keep
// running across item boundaries, so the loads, the first MMAs and the output stores of neighbouring
// items overlap instead of adding a prologue and a tail per item.
//
// Per (i, j) pair, five products on the tensor cores (FP32 accumulators in TMEM), 32 tcgen05.mma in all:
//   group A   S^T  = K_j Q_i^T     dP^T = V_j dO_i^T                         (8 instructions, N = 128)
//   group B   dQ_i = dS K_j        dV  += P^T dO_i      dK  += dS^T Q_i      (24 instructions, N = 64)
// TMEM (512 columns): S^T [0,128) | dP^T [128,256) | P^T (BF16) [256,320) | dV [320,384) |
// dK [384,448) | dQ [448,512).
//
// What bounds this kernel is the rate at which an SM's tensor front end takes tcgen05 instructions: one
// tcgen05.mma OR tcgen05.commit per 50-60 clocks, whichever thread issues it (measured: a stream of N = 64
// MMAs retires one per 46-49 clocks, N = 128 one per 63; eight N = 64 MMAs issued into an idle pipe take 514
// clocks, and every commit after them another 45-54).  So the kernel is built to issue as few of them as
// possible: 32 MMAs and 3 commits per pair (S^T/dP^T ready; dV and dQ
// done; dK done), plus two commits per work item (V free, K free).  A pair then costs about 1.8 k
// clocks of front-end time, which the element-wise work of the compute warps (also about 1.8 k clocks per
// pair) runs beside.
//
// Warps: 0-7 compute (thread = key row x 64 query columns: warps 0-3 take query columns [0,64), warps 4-7
// [64,128)); 8-11 drain (dQ tiles and, once per item, dV / dK: TMEM -> shared-memory staging; also the
// final dQ conversion described below); 12 TMA producer; 13 MMA issuer for group A; 14 MMA issuer for group B;
// 15 staging consumer
// (TMA reduce-add of dQ tiles into the FP32 accumulator in global memory, TMA stores of dV / dK, arrival
// counting).  Barriers that whole warps arrive on count one arrival per warp (lane 0, after __syncwarp).
//
// Order of the issuer's stream inside a work item: A(g+1) as soon as the compute warps hold S^T, dP^T of
// pair g in registers (half way through their work on it), then, when they have finished pair g, dV(g)
// and dQ(g) under one commit (the compute warps' next P^T, the drain and, on the last pair of an item,
// the reload of K wait for it), then dK(g).
// The staging buffer is two 16 KB panels with a full / free barrier each, so that the drain writes one
// panel while the TMA engine still reads the other (an SM's FP32 reduce-adds leave at 30-50 GB/s: the
// 32 KB of a pair take about as long as the pair itself).
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
    // The tile was written by bulk reduce-adds (async proxy) of this and other CTAs, each complete (bulk-group wait)
    // before its CTA's releasing increment of the arrival counter, which this CTA's counting thread has acquired.
    // The reads below go through the generic proxy: order them after the other proxy's writes explicitly.
    asm volatile("fence.proxy.async.global;" ::: "memory");
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
    const uint32_t sStg = sX0 + 2 * Cfg::X_BYTES;                 // two panels of TILE_BYTES

    // Barriers.  g = running pair count of this CTA (over all its items), w = running item count, n = running
    // staging step count (one per pair plus one per item).  Unless noted, a barrier completes one phase per g.
    // A wait on a barrier costs a shared-memory round trip of some 200 clocks while MMAs run (their operand fetch has
    // the shared-memory pipe), so each MMA issuer waits on ONE barrier per pair, which collects every arrival it needs:
    //   A_READY [QS] (per stage)    Q_i, dO_i of pair g landed (TMA) AND the compute warps hold S^T, dP^T of pair g - 1 in
    //                               registers (8 warp arrivals; before the first pair they arrive once unconditionally)
    //   B_READY                     P^T in TMEM and dS^T in X[g & 1] (8 compute-warp arrivals) AND the drain has read dQ of
    //                               pair g - 1 (4 drain-warp arrivals; once unconditionally before the first pair)
    //   K_FULL, V_FULL (per w)      TMA landed                          K_FREE, V_FREE (per w): last dQ / last A of the item done
    //   SDP_FULL                    A(g) done                           VEC_FULL [2]: per-query vectors of g landed (bulk copies)
    //   PDS_FULL [2]                the compute warps have finished pair g (index g & 1, phase (g >> 1) & 1): only the
    //                               producer waits here, for pair g - 2, before it reuses that pair's vector buffer
    //   DQ_FULL                     dV(g) and dQ(g) done: the dQ tile is in TMEM and P^T may be overwritten (with everything
    //                               issued before them: the dS^T buffer of pair g - 1 is free too)
    //   B_DONE [2]                  dK(g) and everything issued before it complete: the Q / dO stage of g is free; on the
    //                               last pair of an item dV, dK are final (index g & 1, phase (g >> 1) & 1: the producer
    //                               looks three pairs back and may be late by a pair after waiting for K)
    //   DKV_FREE (per w)            dV, dK read by the drain
    //   STG_FULL / STG_FREE [2]     (per n, one pair per staging panel) panel written / read by TMA
    //   FIN                         last arrival verdicts written
    enum { K_FULL = 0, V_FULL = 1, K_FREE = 2, V_FREE = 3, A_READY = 4, SDP_FULL = 7, B_READY = 8,
           PDS_FULL = 9, B_DONE = 11, DQ_FULL = 13, DKV_FREE = 14,
           STG_FULL = 15, STG_FREE = 17, VEC_FULL = 19, FIN = 21, NBARS = 22 };
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
            if (b == PDS_FULL || b == PDS_FULL + 1) cnt = 8;                                    // one arrival per compute warp
            if (b >= A_READY && b < A_READY + Cfg::QS) cnt = 9;                                 // ... plus the producer's (with the TMA bytes)
            if (b == B_READY) cnt = 12;                                                         // compute warps and drain warps
            if (b == DKV_FREE || b == STG_FULL || b == STG_FULL + 1) cnt = 4;                   // one per drain warp
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
                if (w > 0) ok = mbar_wait_ool(bar(V_FREE), (w - 1) & 1, &abort_flag);
                if (!ok) break;
                mbar_expect_tx(bar(V_FULL), Cfg::TILE_BYTES);
                tma_load_2d(sV, &tmV, bar(V_FULL), 0, kvrow0);
                BwdPairPos<GENERAL> pos;
                for (int it = 0; it < item.nq; ++it, ++g, pos.next(item)) {
                    const int st = g % Cfg::QS;
                    // the stage was last used by pair g - QS: free when that pair's dV, dK have run
                    if (g >= Cfg::QS) ok = mbar_wait_relaxed_ool(bar(B_DONE + ((g - Cfg::QS) & 1)), ((g - Cfg::QS) >> 1) & 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(A_READY + st), 2 * Cfg::TILE_BYTES);
                    const int qrow = pos.row(item, prm);
                    tma_load_2d(sQ0 + st * Cfg::TILE_BYTES, &tmQ, bar(A_READY + st), 0, qrow);
                    tma_load_2d(sdO0 + st * Cfg::TILE_BYTES, &tmdO, bar(A_READY + st), 0, qrow);
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
                        if (w > 0) ok = mbar_wait_ool(bar(K_FREE), (w - 1) & 1, &abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(bar(K_FULL), Cfg::TILE_BYTES);
                        tma_load_2d(sK, &tmK, bar(K_FULL), 0, kvrow0);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 13) {
        // ------------------------------------------------------------ MMA issuer 1: group A (S^T, dP^T), one pair ahead
        if (lane == 0) {
            constexpr uint32_t idesc_T = make_idesc_bf16(128, 128, 0, 0);   // both operands K-major
            // descriptors: only the start-address field (low word, 16-byte units) changes in the loops
            const uint64_t dK_k = make_smem_desc(sK, 16, 1024);             // K_j, K-major (rows of d)
            const uint64_t dV_k = make_smem_desc(sV, 16, 1024);
            const uint64_t dQ_k0 = make_smem_desc(sQ0, 16, 1024);
            const uint64_t ddO_k0 = make_smem_desc(sdO0, 16, 1024);
            bool ok = true;
            int g = 0;
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                const int nq = item.nq;
                ok = mbar_wait_ool(bar(V_FULL), w & 1, &abort_flag) && mbar_wait_ool(bar(K_FULL), w & 1, &abort_flag);
                for (int it = 0; ok && it < nq; ++it, ++g) {
                    const int st = g % Cfg::QS, ph = (g / Cfg::QS) & 1;
                    ok = mbar_wait_ool(bar(A_READY + st), ph, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        mma_ss(tmem + Cfg::DP_COL, dV_k + ((k * 32) >> 4), ddO_k0 + so + ((k * 32) >> 4), idesc_T, k > 0);
                    if (it == nq - 1) mma_commit(bar(V_FREE));                // last pair of the item: V may be reloaded
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        mma_ss(tmem + Cfg::ST_COL, dK_k + ((k * 32) >> 4), dQ_k0 + so + ((k * 32) >> 4), idesc_T, k > 0);
                    mma_commit(bar(SDP_FULL));
                }
            }
        }
        __syncwarp();
    } else if (warp == 14) {
        // ------------------------------------------------------------ MMA issuer 2: group B (dV, dQ, dK)
        if (lane == 0) {
            constexpr uint32_t idesc_KN = make_idesc_bf16(128, D, 0, 1);    // dV (A from TMEM), dK (A K-major): B MN-major
            constexpr uint32_t idesc_NN = make_idesc_bf16(128, D, 1, 1);    // dQ: A MN-major, B MN-major
            const uint64_t ddO_mn0 = make_smem_desc(sdO0, Cfg::TILE_BYTES, 1024);
            const uint64_t dK_mn = make_smem_desc(sK, Cfg::TILE_BYTES, 1024);    // K_j as [key][d], MN-major B
            const uint64_t dQ_mn0 = make_smem_desc(sQ0, Cfg::TILE_BYTES, 1024);
            const uint64_t dX_k0 = make_smem_desc(sX0, 16, 1024);           // dS^T rows (queries contiguous): K-major A
            const uint64_t dX_mn0 = make_smem_desc(sX0, Cfg::TILE_BYTES, 1024);  // same bytes as (M = query, K = key): MN-major A
            bool ok = true;
            int g = 0;
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                const int nq = item.nq;
                // the accumulators of a new item overwrite dV, dK: the drain must have read the previous item's
                if (w > 0) ok = mbar_wait_ool(bar(DKV_FREE), (w - 1) & 1, &abort_flag);
                for (int it = 0; ok && it < nq; ++it, ++g) {
                    const int st = g % Cfg::QS;
                    ok = mbar_wait_ool(bar(B_READY), g & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = static_cast<uint64_t>((st * Cfg::TILE_BYTES) >> 4);
                    const uint64_t xo = static_cast<uint64_t>(((g & 1) * Cfg::X_BYTES) >> 4);
                    // dQ_i = dS K_j : A = the dS^T buffer read as (M = query, K = key), B = K_j MN-major
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tmem + Cfg::DQ_COL, dX_mn0 + xo + ((k * 2048) >> 4), dK_mn + ((k * 2048) >> 4), idesc_NN, k > 0);
                    if (it == nq - 1) mma_commit(bar(K_FREE));                 // last pair of the item: K may be reloaded
                    // dV += P^T dO_i : A = P^T in TMEM, B = dO_i with d contiguous (MN-major), 16 queries per step
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_ts(tmem + Cfg::DV_COL, tmem + Cfg::PT_COL + k * 8, ddO_mn0 + so + ((k * 2048) >> 4), idesc_KN,
                               (it > 0 || k > 0) ? 1u : 0u);
                    mma_commit(bar(DQ_FULL));                                  // dQ(g) and dV(g): dQ tile ready, P^T free
                    // dK += dS^T Q_i : A = dS^T rows (K-major: 4 steps per 64-query panel), B = Q_i MN-major
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tmem + Cfg::DK_COL, dX_k0 + xo + (((k >> 2) * Cfg::TILE_BYTES + (k & 3) * 32) >> 4),
                               dQ_mn0 + so + ((k * 2048) >> 4), idesc_KN, (it > 0 || k > 0) ? 1u : 0u);
                    mma_commit(bar(B_DONE + (g & 1)));
                }
            }
        }
        __syncwarp();
    } else if (warp == 15) {
        // ------------------------------------------------------------ staging consumer: TMA out of the staging panels, arrival counts
        if (lane == 0) {
            // Arrival counting, two steps behind the TMA issue so that neither the completion of the reduce-adds nor
            // the atomic's round trip holds up the next staging step:
            //   step n, after its two bulk groups are issued:  (1) the atomic issued in step n-1 (for step n-2) has returned by
            //   now: turn it into the verdict on step n-2;  (2) the two groups of step n are the only ones that may still be
            //   incomplete: wait for everything older (step n-1), then issue the atomic for step n-1 without touching its result.
            // The atomic releases this CTA's completed reduce-adds; the CTA that brings a tile's counter to the number
            // of key tiles that see the tile acquires the others' and finishes the tile.
            bool ok = true;
            int n = 0;
            int prev_t = -1, prev_i = 0, prev_Tr = 0;             // dQ tile of step n-1 (-1: it was a dV / dK step)
            int pend_t = -1;                                      // dQ tile of step n-2 whose atomic is in flight (-1: none)
            unsigned pend_old = 0, pend_expected = 0;
            auto settle = [&](int pending_groups) {
                if (n >= 2) {
                    int verdict = -1;
                    if (pend_t >= 0 && pend_old + 1 == pend_expected) { fence_acq_rel_gpu(); verdict = pend_t; }
                    s_final[(n - 2) & 7] = verdict;
                }
                if (n >= 1) {
                    if (pending_groups == 2) asm volatile("cp.async.bulk.wait_group 2;" ::: "memory");
                    else                     asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                    pend_t = prev_t;
                    if (prev_t >= 0) {
                        pend_expected = CAUSAL ? static_cast<unsigned>(prev_i + 1) : static_cast<unsigned>(prev_Tr);
                        pend_old = atom_add_release_gpu(
                            reinterpret_cast<unsigned*>(prm.dq + static_cast<size_t>(prev_t) * 128 * D), 1u);
                    }
                }
            };
            // One staging step: panel 0 then panel 1, each handed over by the drain on its own barrier and given back as
            // soon as the TMA engine has read it, so that the drain writes one panel while the other is being read.
            auto step = [&](auto issue_panel) -> bool {
                if (!mbar_wait_relaxed_ool(bar(STG_FULL + 0), n & 1, &abort_flag)) return false;
                issue_panel(0);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (!mbar_wait_relaxed_ool(bar(STG_FULL + 1), n & 1, &abort_flag)) return false;
                issue_panel(1);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");      // panel 0 has been read
                mbar_arrive(bar(STG_FREE + 0));
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");      // panel 1 has been read
                mbar_arrive(bar(STG_FREE + 1));
                return true;
            };
            for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
                BwdPairPos<GENERAL> pos;
                for (int it = 0; it < item.nq; ++it, pos.next(item)) {
                    const int i = item.i0 + pos.ii;
                    const int qrow = pos.row(item, prm);
                    ok = step([&](int p) { tma_reduce_add_2d(&tmAcc, sStg + p * Cfg::TILE_BYTES, 32 * p, qrow); });   // columns [32 p, 32 p + 32)
                    if (!ok) break;
                    settle(2);
                    prev_t = qrow >> 7;
                    prev_i = i;
                    prev_Tr = item.Tr;
                    ++n;
                }
                if (!ok) break;
                const int kvrow0 = item.bh * prm.N + item.j * 128;
                ok = step([&](int p) { tma_store_2d(p ? &tmdK : &tmdV, sStg + p * Cfg::TILE_BYTES, 0, kvrow0); });
                if (!ok) break;
                settle(2);
                prev_t = -1;
                ++n;
            }
            if (ok) {                                             // everything written before exit; verdicts on the last two steps
                settle(0);
                ++n;
                prev_t = -1;
                settle(0);
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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
        if (lane == 0) mbar_arrive(bar(B_READY));                 // "dQ of the pair before the first one has been read"
        // Before writing staging panel p in step n: the TMA transfer of step n-1 must have read it.
        auto panel_ready = [&](int p) -> bool {
            bool o = true;
            if (n > 0) o = mbar_wait_relaxed_ool(bar(STG_FREE + p), (n - 1) & 1, &abort_flag);
            return __all_sync(0xffffffffu, o);
        };
        auto panel_written = [&](int p) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(STG_FULL + p));
        };
        // The staging consumer wrote the verdict on step n-4 before it gave panel 0 of step n-1 back and rewrites the
        // slot only many steps later: read it once panel 0 is ours.
        auto verdict = [&]() { return (n >= 4) ? s_final[(n - 4) & 7] : -1; };
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
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_READY));         // the dQ columns may be overwritten
                // two [128 rows][32 floats = 128 bytes] panels, 128-byte swizzle
                ok = panel_ready(0);
                if (!ok) break;
                const int fi = verdict();
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    sts128(sStg + r * 128 + ((c ^ (r & 7)) << 4), a[4 * c], a[4 * c + 1], a[4 * c + 2], a[4 * c + 3]);
                panel_written(0);
                ok = panel_ready(1);
                if (!ok) break;
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    sts128(sStg + Cfg::TILE_BYTES + r * 128 + ((c ^ (r & 7)) << 4), b[4 * c], b[4 * c + 1], b[4 * c + 2], b[4 * c + 3]);
                panel_written(1);
                if (fi >= 0) finish_tile(fi);
            }
            if (!ok) break;
            // ---- dV and scale * dK of the item -> BF16 -> staging (dV | dK, [128 rows][64 BF16], 128-byte swizzle)
            ok = mbar_wait_relaxed_ool(bar(B_DONE + ((g - 1) & 1)), ((g - 1) >> 1) & 1, &abort_flag);     // the item's last pair: dV, dK are final
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            int fi = -1;
#pragma unroll
            for (int t = 0; t < 2; ++t) {                         // t = 0: dV, t = 1: scale * dK
                ok = panel_ready(t);
                if (!ok) break;
                if (t == 0) fi = verdict();
                const float mul = t ? prm.scale : 1.0f;
                const uint32_t stage = sStg + t * Cfg::TILE_BYTES + r * 128;
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
                        sts128(stage + ((cc ^ (r & 7)) << 4), o.x, o.y, o.z, o.w);
                    }
                }
                if (t == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(DKV_FREE));    // the next item may start new dV, dK accumulators
                }
                panel_written(t);
            }
            if (!ok) break;
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
        if (lane == 0) mbar_arrive(bar(A_READY));                 // "S^T, dP^T of the pair before the first one are free"
        for (int w = 0, e = 0; ok && bwd_item<CAUSAL, GENERAL>(e, prm, item); ++w) {
            int ii = 0;                                           // query tile offset inside the current query head
            for (int it = 0; it < item.nq; ++it, ++g, ii = (GENERAL && ii + 1 == item.nqh) ? 0 : ii + 1) {
                const int buf = g & 1;
                ok = mbar_wait_ool(bar(VEC_FULL + buf), (g >> 1) & 1, &abort_flag) && mbar_wait_ool(bar(SDP_FULL), g & 1, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t xrow = sX0 + buf * Cfg::X_BYTES + half * Cfg::TILE_BYTES + r * 128;
                const uint32_t vecL = smem_u32(&sNegL[buf][0]), vecD = smem_u32(&sDelta[buf][0]);
                // Partly masked pairs: the causal diagonal (key row r sees query column q only if r <= q), key rows and query
                // columns beyond the sequence length.  Key row r of the tile sees the query columns q with qlo <= q < qlo + span.
                // One copy of the arithmetic for both kinds of pair (instruction-cache footprint); the mask sits behind a
                // CTA-uniform branch.
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
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar(A_READY + (g + 1) % Cfg::QS));
                        }
                        uint32_t pk[16], dsk[16];
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 nl = lds128f(vecL + (q0 + c) * 4);
                            const float4 dl = lds128f(vecD + (q0 + c) * 4);
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
                        if (h == 0 && g > 0) {
                            // first write of this pair into P^T and dS^T: dV of pair g-1 (and with it dK, dQ of pair g-2) must
                            // have read them (they ran under the arithmetic above)
                            ok = mbar_wait_ool(bar(DQ_FULL), (g - 1) & 1, &abort_flag);
                        }
                        tmem_st16(tmem + Cfg::PT_COL + lane_base + (q0 >> 1), pk);
                        // dS^T row r, 32 queries: four 16-byte chunks of this half's panel, 128-byte swizzle
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const int cc = h * 4 + q4;
                            sts128(xrow + ((cc ^ (r & 7)) << 4), dsk[4 * q4], dsk[4 * q4 + 1], dsk[4 * q4 + 2], dsk[4 * q4 + 3]);
                        }
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;                                   // a wait gave up: the abort flag is set, every role unwinds
                tmem_wait_st();
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(bar(B_READY)); mbar_arrive(bar(PDS_FULL + buf)); }
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
