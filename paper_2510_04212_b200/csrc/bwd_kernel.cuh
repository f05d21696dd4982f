// Backward kernels: Algorithm 2 on sm_100a.
//
//   bwd_preprocess_kernel  delta = rowsum(dO o O) (streaming, HBM bound); for the main kernels it also clears the
//                          FP32 dQ accumulator and lays out the per-query vectors and arrival counters.
//   (the main kernels live in bwd_kernel_d64.cuh and bwd_kernel_d128.cuh)
//   dq_convert_tiled128_kernel   dQ = bf16(scale * FP32 accumulator) for d = 128.
//
// Rounding: P = bf16(exp(S - L)) feeds dV; dS = bf16(p32 (dP - delta)) feeds dQ and dK; all three
// gradients accumulate in FP32 and are rounded to BF16 once; scale is applied in FP32.
#pragma once
#include <cuda.h>
#include "ptx.cuh"

namespace attn {

// ------------------------------------------------------------------ delta = rowsum(dO o O)
// One thread per 8 contiguous elements (16 bytes) of a row; D/8 threads cooperate on a row.
//
// For the main backward kernels the same pass prepares, per 128-row query tile, in the bytes of that tile of
// the dQ OUTPUT buffer (free until the tile's dQ is written at the very end):
//   bytes [0,4)          arrival counter of the tile, cleared (used at d = 64)
//   bytes [16,528)       -L * log2(e) of the 128 rows, FP32
//   bytes [528,1040)     -delta of the 128 rows, FP32
// so that the main kernel fetches the two per-query vectors of a pair with two bulk copies next to Q_i and dO_i.
// A tile is overwritten with its dQ only after every key tile that sees it has added its part, i.e. after the
// last reader of these vectors.
constexpr int VEC_NEGL_OFFSET = 16, VEC_NDELTA_OFFSET = 16 + 512;

template <int D>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const uint4* __restrict__ o, const uint4* __restrict__ dO, float* __restrict__ delta,
                      const float* __restrict__ delta_given, const float* __restrict__ lse,
                      float4* __restrict__ dq_acc, uint8_t* __restrict__ dq_tiles, long long n_chunks)
{
    constexpr int TPR = D / 8;                       // threads per row
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    float acc = 0.0f;
    ptx::griddep_launch_dependents();
    ptx::griddep_wait();
    if (idx < n_chunks) {
        const uint4 a = __ldg(o + idx);
        const uint4 b = __ldg(dO + idx);
        const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            acc = fmaf(ptx::bf16_lo(av[t]), ptx::bf16_lo(bv[t]), acc);
            acc = fmaf(ptx::bf16_hi(av[t]), ptx::bf16_hi(bv[t]), acc);
        }
        if (dq_acc) {
            dq_acc[2 * idx] = make_float4(0.f, 0.f, 0.f, 0.f);
            dq_acc[2 * idx + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
#pragma unroll
    for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (idx < n_chunks && (threadIdx.x % TPR) == 0) {
        const long long row = idx / TPR;
        if (delta_given) acc = delta_given[row];      // the caller supplies delta (diagnostic variant)
        else if (delta) delta[row] = acc;
        if (dq_tiles) {
            uint8_t* tile = dq_tiles + (row >> 7) * (128ll * D * 2);
            const int rr = static_cast<int>(row & 127);
            if (rr == 0) *reinterpret_cast<unsigned*>(tile) = 0u;
            reinterpret_cast<float*>(tile + VEC_NEGL_OFFSET)[rr] = -lse[row] * LOG2E;
            reinterpret_cast<float*>(tile + VEC_NDELTA_OFFSET)[rr] = -acc;
        }
    }
}

// ------------------------------------------------------------------ delta = rowsum(dO o O) with O in FP32
// The "O kept in FP32" variant of Sec. 3.2: same pass, O read as FP32 (the forward's o_f32 output).
template <int D>
__global__ void __launch_bounds__(256)
delta_f32_kernel(const float4* __restrict__ o, const uint4* __restrict__ dO, float* __restrict__ delta, long long n_chunks)
{
    constexpr int TPR = D / 8;
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    float acc = 0.0f;
    if (idx < n_chunks) {
        const float4 a0 = o[2 * idx], a1 = o[2 * idx + 1];
        const uint4 b = __ldg(dO + idx);
        acc = fmaf(a0.x, ptx::bf16_lo(b.x), acc);
        acc = fmaf(a0.y, ptx::bf16_hi(b.x), acc);
        acc = fmaf(a0.z, ptx::bf16_lo(b.y), acc);
        acc = fmaf(a0.w, ptx::bf16_hi(b.y), acc);
        acc = fmaf(a1.x, ptx::bf16_lo(b.z), acc);
        acc = fmaf(a1.y, ptx::bf16_hi(b.z), acc);
        acc = fmaf(a1.z, ptx::bf16_lo(b.w), acc);
        acc = fmaf(a1.w, ptx::bf16_hi(b.w), acc);
    }
#pragma unroll
    for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (idx < n_chunks && (threadIdx.x % TPR) == 0) delta[idx / TPR] = acc;
}

// ------------------------------------------------------------------ dQ = bf16(scale * acc), d = 128
// (at d = 64 the main kernel converts a dQ tile itself when its last contribution has arrived)
// The d = 128 main kernel's accumulator keeps the layout of that kernel's staging buffer so that a staged panel is
// one contiguous reduce-add: per 128-row tile four panels of 32 columns, a panel = 128 rows x 128
// bytes, the 16-byte chunk c of row r stored at chunk position c ^ (r & 7).  One thread per 8 output columns.
__global__ void __launch_bounds__(256)
dq_convert_tiled128_kernel(const float4* __restrict__ acc, uint4* __restrict__ dq, float scale, long long n_chunks)
{
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    ptx::griddep_launch_dependents();
    ptx::griddep_wait();
    if (idx >= n_chunks) return;
    const long long row = idx >> 4;                       // 16 chunks of 8 columns per row
    const int c8 = static_cast<int>(idx & 15), r = static_cast<int>(row & 127);
    const long long base = (row >> 7) * 4096 + (c8 >> 2) * 1024 + r * 8;        // in float4 units
    const int c0 = (c8 & 3) * 2;
    const float4 a = acc[base + (c0 ^ (r & 7))], b = acc[base + ((c0 + 1) ^ (r & 7))];
    uint4 out;
    out.x = ptx::pack_bf16(a.x * scale, a.y * scale);
    out.y = ptx::pack_bf16(a.z * scale, a.w * scale);
    out.z = ptx::pack_bf16(b.x * scale, b.y * scale);
    out.w = ptx::pack_bf16(b.z * scale, b.w * scale);
    dq[idx] = out;
}

// ------------------------------------------------------------------ arguments of the main backward kernels
struct BwdParams {
    const float* lse;
    const float* delta;
    float* dq_acc;
    uint16_t* dq;
    uint16_t* dk;
    uint16_t* dv;
    int N, BH, Tr;             // N: rows per head in memory; BH: number of key/value heads, B * H_kv;
                               // Tr: 128-row tiles per head that hold one of the seqlen rows
    int seqlen;                // queries and keys per head that count (<= N); rows beyond are padding
    const int* seqlens;        // != nullptr: one sequence length per batch element (device memory, [B]) instead of seqlen
    int Hkv;                   // key/value heads (batch element of key/value head bh: bh / Hkv)
    int group;                 // query heads per key/value head (grouped-query attention; 1 = multi-head): query
                               // head g of key/value head bh is head bh * group + g of the [B][H] tensors
    int head_group;            // d = 128, causal: key/value heads whose key tiles are launched together (>= 1)
    float scale;
    int* status;
};

}  // namespace attn
