// V (BF16, [B][H][N][d]) -> E4M3, transposed to [B][H][d][N]: the operand layout of the 8-bit P-bar V product
// (a key tile of V^T is K-major: d rows of 64 contiguous keys).  One thread per (d column, group of 16 keys):
// lanes read neighbouring columns of one key (coalesced), each thread writes 16 contiguous bytes of its row.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace attn {

__device__ __forceinline__ uint32_t quant_e4m3x4(float a, float b, float c, float d) {
    uint32_t w;
    asm("{ .reg .b16 h0, h1;\n"
        "cvt.rn.satfinite.e4m3x2.f32 h0, %2, %1;\n"
        "cvt.rn.satfinite.e4m3x2.f32 h1, %4, %3;\n"
        "mov.b32 %0, {h0, h1}; }" : "=r"(w) : "f"(a), "f"(b), "f"(c), "f"(d));
    return w;
}

template <int D>
__global__ void __launch_bounds__(256)
quantize_v_e4m3_kernel(const uint16_t* __restrict__ v, uint8_t* __restrict__ vt, int N, float v_scale)
{
    constexpr int KEYS_PER_BLOCK = 16 * (256 / D);                // 64 at d = 64, 32 at d = 128
    const int bh = blockIdx.y;
    const int c = threadIdx.x % D, kg = threadIdx.x / D;
    const int n0 = blockIdx.x * KEYS_PER_BLOCK + kg * 16;
    const uint16_t* src = v + (static_cast<size_t>(bh) * N + n0) * D + c;
    float x[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = __uint_as_float(static_cast<uint32_t>(src[static_cast<size_t>(i) * D]) << 16) * v_scale;
    uint4 out;
    out.x = quant_e4m3x4(x[0], x[1], x[2], x[3]);
    out.y = quant_e4m3x4(x[4], x[5], x[6], x[7]);
    out.z = quant_e4m3x4(x[8], x[9], x[10], x[11]);
    out.w = quant_e4m3x4(x[12], x[13], x[14], x[15]);
    *reinterpret_cast<uint4*>(vt + (static_cast<size_t>(bh) * D + c) * N + n0) = out;
}

}  // namespace attn
