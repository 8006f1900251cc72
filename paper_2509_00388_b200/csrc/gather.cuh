// Step (IV), second half: copy the kept prefix rows and the window rows of K and V into the
// compact cache, 16 bytes per thread, bit for bit.
#pragma once

#include "common.cuh"

namespace graphkv {

constexpr int kGatherThreads = 256;

// out[unit][t] = X[b][h][idx[unit][t]] for t < B, X[b][h][N + (t - B)] for B <= t < B + W.
// vec_per_row = D * sizeof(element) / 16.  One thread moves one 16-byte piece of K and of V.
__global__ void __launch_bounds__(kGatherThreads) gather_rows_kernel(
    Dims d, int elem_bytes, const unsigned char *__restrict__ K, const unsigned char *__restrict__ V,
    const int *__restrict__ idx, unsigned char *__restrict__ K_out, unsigned char *__restrict__ V_out)
{
    const int vec_per_row = d.D * elem_bytes / 16;
    const long long rows_out = d.B + d.W;
    const long long total = (long long)d.units * rows_out * vec_per_row;
    const long long row_bytes = (long long)d.D * elem_bytes;
    for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < total;
         p += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(p % vec_per_row);
        const long long rt = p / vec_per_row;
        const int t = (int)(rt % rows_out);
        const int unit = (int)(rt / rows_out);
        const int b = unit / d.hkv, h = unit % d.hkv;
        const int src_row = t < d.B ? idx[(long long)unit * d.B + t] : d.N + (t - d.B);
        const long long dst = (rt * row_bytes) + c * 16;
        if (K) {
            const long long off = (b * d.ks[0] + h * d.ks[1] + src_row * d.ks[2]) * elem_bytes;
            *reinterpret_cast<uint4 *>(K_out + dst) =
                *reinterpret_cast<const uint4 *>(K + off + c * 16);
        }
        if (V) {
            const long long off = (b * d.vs[0] + h * d.vs[1] + src_row * d.vs[2]) * elem_bytes;
            *reinterpret_cast<uint4 *>(V_out + dst) =
                *reinterpret_cast<const uint4 *>(V + off + c * 16);
        }
    }
}

}  // namespace graphkv
