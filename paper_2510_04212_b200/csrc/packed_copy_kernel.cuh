// Copies between the packed variable-length layout (token-major, no padding rows, cumulative offsets) and the
// padded per-batch layout [B][Hx][N][d] that the attention kernels work on.  Plain streaming kernels: one thread per
// 16 bytes of a padded row (or per row of a per-row FP32 vector); threads of padding rows write zeros where the kernels
// will read (inside the tiles that hold part of the sequence) and nothing elsewhere.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace attn {

// seqlens[b] = min(cu[b + 1] - cu[b], N), never negative
__global__ void packed_seqlens_kernel(const int* __restrict__ cu, int* __restrict__ seqlens, int B, int N)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) seqlens[b] = max(0, min(cu[b + 1] - cu[b], N));
}

// TO_PADDED:  padded[b][h][n][:] = packed[cu[b] + n][h][:] for n < len_b, zeros for the other rows of the tiles in use
// !TO_PADDED: packed[cu[b] + n][h][:] = padded[b][h][n][:] for n < len_b
// rows: [.., d] of 2-byte elements, d / 8 chunks of 16 bytes per row.  n_chunks = B * Hx * N * (d / 8).
template <bool TO_PADDED>
__global__ void __launch_bounds__(256)
packed_rows_kernel(uint4* __restrict__ padded, uint4* __restrict__ packed, const int* __restrict__ cu,
                   int Hx, int N, int cpr /* chunks per row */, long long n_chunks)
{
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= n_chunks) return;
    const int c = static_cast<int>(idx % cpr);
    const long long row = idx / cpr;
    const int n = static_cast<int>(row % N);
    const long long bh = row / N;
    const int h = static_cast<int>(bh % Hx), b = static_cast<int>(bh / Hx);
    const int start = cu[b], len = max(0, min(cu[b + 1] - start, N));
    if (n < len) {
        uint4* p = packed + (static_cast<long long>(start + n) * Hx + h) * cpr + c;
        if (TO_PADDED) padded[idx] = *p;
        else           *p = padded[idx];
    } else if (TO_PADDED && n < ((len + 127) & ~127)) {
        padded[idx] = make_uint4(0u, 0u, 0u, 0u);
    }
}

// per-row FP32 vectors: padded [B][H][N], packed [H][T]
template <bool TO_PADDED>
__global__ void __launch_bounds__(256)
packed_vec_kernel(float* __restrict__ padded, float* __restrict__ packed, const int* __restrict__ cu,
                  int H, int N, int T, long long n_rows)
{
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= n_rows) return;
    const int n = static_cast<int>(idx % N);
    const long long bh = idx / N;
    const int h = static_cast<int>(bh % H), b = static_cast<int>(bh / H);
    const int start = cu[b], len = max(0, min(cu[b + 1] - start, N));
    if (n < len) {
        float* p = packed + static_cast<long long>(h) * T + start + n;
        if (TO_PADDED) padded[idx] = *p;
        else           *p = padded[idx];
    } else if (TO_PADDED && n < ((len + 127) & ~127)) {
        padded[idx] = 0.0f;
    }
}

}  // namespace attn
