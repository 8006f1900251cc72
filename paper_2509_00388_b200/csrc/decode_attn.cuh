// Decode-side use of a cache: the attention of one new token's queries over `rows` cached keys
// and values per KV head (the full cache, or the compact cache this library builds), as a
// micro-benchmark of what the compression buys at decoding time (Efficiency Analysis: the paper's
// only latency table is decoding latency).
//
//   out[b][hq][:] = sum_j softmax_j(q[b][hq] . K[b][h][j] / sqrt(D)) * V[b][h][j],  h = hq / G
//
// The cache is read once: a CTA takes a range of rows of one KV head for all G query heads that
// share it, in tiles of 32 rows (logits by four threads per row, a running maximum and sum per
// query head, values accumulated by threads that own two output dimensions each), and leaves a
// partial (max, sum, accumulator); a second kernel merges the partials of a head.  fp32 arithmetic
// on bf16 or fp32 inputs.
#pragma once

#include "common.cuh"

namespace graphkv {

constexpr int kDecThreads = 128;
constexpr int kDecTile = 32;           // rows per tile
constexpr int kDecMaxG = 8;            // query heads per KV head this kernel serves

struct DecodeArgs {
    int batch, hq, hkv, G, rows, splits;
    long long qs[2];                   // element strides of q: batch, head
    long long ks[3], vs[3];            // element strides of K and V: batch, head, row
    float *part;                       // [units][splits][G][2 + D] partial (max, sum, accumulator)
    float *out;                        // [batch][hq][D]
};

template <typename T>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(DecodeArgs a, const T *__restrict__ q,
                                                                     const T *__restrict__ K,
                                                                     const T *__restrict__ V)
{
    __shared__ float s_q[kDecMaxG * kHeadDim];        // queries, pre-scaled by log2(e) / sqrt(D)
    __shared__ float s_p[kDecMaxG * kDecTile];        // logits, then probabilities of the tile
    __shared__ float s_scale[kDecMaxG];               // rescale of the accumulators after a tile
    __shared__ float s_ml[kDecMaxG * 2];              // final (max, sum) per query head
    const int unit = blockIdx.y, b = unit / a.hkv, h = unit % a.hkv, split = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, G = a.G;
    const int per = (a.rows + a.splits - 1) / a.splits;
    const int r0 = split * per, r1 = min(r0 + per, a.rows);
    const T *Kh = K + b * a.ks[0] + (long long)h * a.ks[1];
    const T *Vh = V + b * a.vs[0] + (long long)h * a.vs[1];
    const float scale = rsqrtf((float)kHeadDim) * kLog2e;
    for (int i = tid; i < G * kHeadDim; i += kDecThreads) {
        const int g = i / kHeadDim, d = i % kHeadDim;
        s_q[i] = (float)q[b * a.qs[0] + (long long)(h * G + g) * a.qs[1] + d] * scale;
    }
    __syncthreads();
    // this thread's slice of a row for the logits, and its output dimensions for the values
    const int row_in_tile = tid >> 2, part = tid & 3;          // 32 dims [part * 32, part * 32 + 32)
    const int dpair = tid & 63, gpar = tid >> 6;               // dims 2 * dpair, +1; heads gpar, gpar + 2, ...
    float acc[kDecMaxG / 2][2];
#pragma unroll
    for (int u = 0; u < kDecMaxG / 2; ++u) acc[u][0] = acc[u][1] = 0.f;
    // running (max, sum) of the softmax: warp w keeps those of query heads w and w + 4
    float m_run = kNegBig, l_run = 0.f, m2 = kNegBig, l2 = 0.f;
    for (int t0 = r0; t0 < r1; t0 += kDecTile) {
        // ---- logits of the tile ----
        const int row = t0 + row_in_tile;
        float dot[kDecMaxG];
#pragma unroll
        for (int g = 0; g < kDecMaxG; ++g) dot[g] = 0.f;
        if (row < r1) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float kv[8];
                load8(Kh + (long long)row * a.ks[2] + part * 32 + c * 8, kv);
#pragma unroll
                for (int g = 0; g < kDecMaxG; ++g) {
                    if (g < G) {
                        const float *qg = s_q + g * kHeadDim + part * 32 + c * 8;
#pragma unroll
                        for (int e = 0; e < 8; ++e) dot[g] = fmaf(kv[e], qg[e], dot[g]);
                    }
                }
            }
        }
#pragma unroll
        for (int g = 0; g < kDecMaxG; ++g) {
            if (g < G) {
                dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], 1);
                dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], 2);
                if (part == 0) s_p[g * kDecTile + row_in_tile] = row < r1 ? dot[g] : -INFINITY;
            }
        }
        __syncthreads();
        // ---- running softmax statistics: warp w updates heads w and w + 4 (lane = row of the tile) ----
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int g = warp + 4 * k;
            if (g < G) {
                float &m_old = k == 0 ? m_run : m2, &l_old = k == 0 ? l_run : l2;
                const float l = s_p[g * kDecTile + lane];
                float mx = l;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_new = fmaxf(m_old, mx);
                const float p = exp2f(l - m_new);
                const float ps = warp_sum(p);
                const float sc = exp2f(m_old - m_new);
                s_p[g * kDecTile + lane] = p;
                if (lane == 0) s_scale[g] = sc;
                l_old = l_old * sc + ps;
                m_old = m_new;
            }
        }
        __syncthreads();
        // ---- values: acc[g] = acc[g] * scale[g] + sum_rows p[g][row] * V[row][dims] ----
#pragma unroll
        for (int u = 0; u < kDecMaxG / 2; ++u) {
            const int g = gpar + 2 * u;
            if (g < G) {
                acc[u][0] *= s_scale[g];
                acc[u][1] *= s_scale[g];
            }
        }
        const int n_rows = min(kDecTile, r1 - t0);
#pragma unroll 8
        for (int r = 0; r < n_rows; ++r) {
            float v0, v1;
            if constexpr (sizeof(T) == 2) {
                const uint32_t raw = *reinterpret_cast<const uint32_t *>(Vh + (long long)(t0 + r) * a.vs[2] + 2 * dpair);
                v0 = __uint_as_float(raw << 16);
                v1 = __uint_as_float(raw & 0xffff0000u);
            } else {
                const float2 raw = *reinterpret_cast<const float2 *>(Vh + (long long)(t0 + r) * a.vs[2] + 2 * dpair);
                v0 = raw.x;
                v1 = raw.y;
            }
#pragma unroll
            for (int u = 0; u < kDecMaxG / 2; ++u) {
                const int g = gpar + 2 * u;
                if (g < G) {
                    const float p = s_p[g * kDecTile + r];
                    acc[u][0] = fmaf(p, v0, acc[u][0]);
                    acc[u][1] = fmaf(p, v1, acc[u][1]);
                }
            }
        }
        __syncthreads();
    }
    // ---- the CTA's partial result ----
    if (lane == 0) {
        if (warp < G) { s_ml[2 * warp] = m_run; s_ml[2 * warp + 1] = l_run; }
        if (warp + 4 < G) { s_ml[2 * (warp + 4)] = m2; s_ml[2 * (warp + 4) + 1] = l2; }
    }
    __syncthreads();
    float *po = a.part + ((long long)unit * a.splits + split) * G * (2 + kHeadDim);
#pragma unroll
    for (int u = 0; u < kDecMaxG / 2; ++u) {
        const int g = gpar + 2 * u;
        if (g < G) {
            float *pg = po + g * (2 + kHeadDim);
            if (dpair == 0) { pg[0] = s_ml[2 * g]; pg[1] = s_ml[2 * g + 1]; }
            pg[2 + 2 * dpair] = acc[u][0];
            pg[2 + 2 * dpair + 1] = acc[u][1];
        }
    }
}

// out[b][hq][d] from the partials of the head's row ranges.  grid (units * G), block 128 (thread = d).
__global__ void __launch_bounds__(kHeadDim) decode_merge_kernel(DecodeArgs a)
{
    const int unit = blockIdx.x / a.G, g = blockIdx.x % a.G, d = threadIdx.x;
    const int b = unit / a.hkv, h = unit % a.hkv;
    const float *p0 = a.part + (long long)unit * a.splits * a.G * (2 + kHeadDim) + g * (2 + kHeadDim);
    const long long stride = (long long)a.G * (2 + kHeadDim);
    float m = kNegBig;
    for (int s = 0; s < a.splits; ++s) m = fmaxf(m, p0[s * stride]);
    float l = 0.f, acc = 0.f;
    for (int s = 0; s < a.splits; ++s) {
        const float w = exp2f(p0[s * stride] - m);
        l = fmaf(p0[s * stride + 1], w, l);
        acc = fmaf(p0[s * stride + 2 + d], w, acc);
    }
    a.out[((long long)b * a.hq + h * a.G + g) * kHeadDim + d] = acc / l;
}

}  // namespace graphkv
