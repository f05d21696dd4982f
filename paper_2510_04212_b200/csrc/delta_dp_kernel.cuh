// delta = rowsum(dP o P) with dP = dO V^T and P = exp(scale Q K^T - L): the alternative formulation of
// Sec. 3.2, which never reads O.  A diagnostic (the paper uses it to show that the error of O is what breaks
// training), not a step of the hot path: written for clarity on the ordinary FP32 pipes, no tensor cores.
//
// One CTA per (64 query rows, head); key tiles of 64 rows pass through shared memory.  Thread = (query row,
// quarter): it takes every fourth key of a tile, forms the two dot products of length d in FP32 (BF16 products
// are exact in FP32), p = exp2(scale * log2(e) * s - L * log2(e)) unrounded, and accumulates p * dP in FP32;
// the four partial sums of a row are added at the end.
#pragma once
#include "ptx.cuh"

namespace attn {

template <int D>
struct DeltaDpCfg {
    static constexpr int ROWS = 64, KEYS = 64;
    static constexpr int C16 = D / 8;                // 16-byte chunks per row
    static constexpr int PAD = C16 + 1;              // key rows padded by one chunk: the four quarters hit distinct banks
    static constexpr int SMEM_BYTES = (2 * ROWS * C16 + 2 * KEYS * PAD) * 16;   // 34 KB at d = 64, 67 KB at d = 128
};

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(256)
delta_dp_kernel(const uint4* __restrict__ q, const uint4* __restrict__ k, const uint4* __restrict__ v,
                const uint4* __restrict__ dO, const float* __restrict__ lse, float* __restrict__ delta,
                int N, float scale)
{
    constexpr int ROWS = DeltaDpCfg<D>::ROWS, KEYS = DeltaDpCfg<D>::KEYS;
    constexpr int C16 = DeltaDpCfg<D>::C16, PAD = DeltaDpCfg<D>::PAD;
    extern __shared__ uint4 delta_dp_smem[];
    uint4 (*sQ)[C16] = reinterpret_cast<uint4 (*)[C16]>(delta_dp_smem);
    uint4 (*sG)[C16] = sQ + ROWS;
    uint4 (*sK)[PAD] = reinterpret_cast<uint4 (*)[PAD]>(sG + ROWS);
    uint4 (*sV)[PAD] = sK + KEYS;
    const int tid = threadIdx.x;
    const int nrb = N / ROWS;                        // 64-row blocks per head
    const int bh = blockIdx.x / nrb, r0 = (blockIdx.x % nrb) * ROWS;
    const size_t head = static_cast<size_t>(bh) * N;
    for (int idx = tid; idx < ROWS * C16; idx += 256) {
        const int r = idx / C16, c = idx % C16;
        sQ[r][c] = q[(head + r0 + r) * C16 + c];
        sG[r][c] = dO[(head + r0 + r) * C16 + c];
    }
    const int r = tid >> 2, quarter = tid & 3;
    const int T = r0 + r;                            // query index inside the head
    const float c_l2 = scale * LOG2E;
    const float negl = -lse[head + T] * LOG2E;
    float acc = 0.0f;
    const int ntiles = CAUSAL ? (r0 + ROWS + KEYS - 1) / KEYS : N / KEYS;
    for (int j = 0; j < ntiles; ++j) {
        __syncthreads();                             // the previous tile has been read (first pass: sQ, sG written)
        for (int idx = tid; idx < KEYS * C16; idx += 256) {
            const int kr = idx / C16, c = idx % C16;
            sK[kr][c] = k[(head + j * KEYS + kr) * C16 + c];
            sV[kr][c] = v[(head + j * KEYS + kr) * C16 + c];
        }
        __syncthreads();
#pragma unroll 1
        for (int kk = quarter; kk < KEYS; kk += 4) {
            const int t = j * KEYS + kk;             // key index inside the head
            float s = 0.0f, dp = 0.0f;
#pragma unroll
            for (int c = 0; c < C16; ++c) {
                const uint4 a = sQ[r][c], b = sK[kk][c], g = sG[r][c], w = sV[kk][c];
                const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
                const uint32_t gv[4] = {g.x, g.y, g.z, g.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    s = fmaf(ptx::bf16_lo(av[e]), ptx::bf16_lo(bv[e]), s);
                    s = fmaf(ptx::bf16_hi(av[e]), ptx::bf16_hi(bv[e]), s);
                    dp = fmaf(ptx::bf16_lo(gv[e]), ptx::bf16_lo(wv[e]), dp);
                    dp = fmaf(ptx::bf16_hi(gv[e]), ptx::bf16_hi(wv[e]), dp);
                }
            }
            const float p = ptx::ex2(fmaf(s, c_l2, negl));
            if (!CAUSAL || t <= T) acc = fmaf(p, dp, acc);
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    if (quarter == 0) delta[head + T] = acc;
}

}  // namespace attn
