// Steps (II)+(III): edges of the source nodes (Eq. 1, Algorithm 1) and the decay rounds
// (Eq. 3-5, Algorithm 2).  SIMT fp32 similarity path for any input dtype.
#pragma once

#include "common.cuh"

namespace graphkv {

constexpr int kSimThreads = 128;
constexpr int kSimChunk = 512;     // keys per CTA
constexpr int kMaxSrcSmem = 64;    // source rows staged per pass over the key registers

// e[a][j] = <k_src[a], k_j> / (max(|k_src[a]|, eps) * max(|k_j|, eps)), clipped to [-1, 1],
// for all sources a of the head and every prefix key j.  Entry j = src[a] is written too; the
// neighbour selection excludes it by index.
// grid (ceil(N / kSimChunk), units), block kSimThreads.  sims [units][K_src][N].
// The sources' vectors come from tensor S (strides ss), the swept vectors from tensor K (strides
// ks): the same tensor for Eq. 1, keys and values for the other edge kinds.
struct Strides3 {
    long long v[3];
};

template <typename T, int kD>
__global__ void __launch_bounds__(kSimThreads) similarity_simt(Dims d, const T *__restrict__ S, Strides3 ss,
                                                             const T *__restrict__ K, Strides3 ks,
                                                             const int *__restrict__ src,
                                                             float *__restrict__ sims)
{
    __shared__ __align__(16) float srows[kMaxSrcSmem * kD];   // unit-norm source keys
    const int unit = blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const T *Kh = K + b * ks.v[0] + (long long)h * ks.v[1];
    const T *Sh = S + b * ss.v[0] + (long long)h * ss.v[1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j0 = blockIdx.x * kSimChunk;
    const int j1 = min(j0 + kSimChunk, d.N);

    for (int a0 = 0; a0 < d.K_src; a0 += kMaxSrcSmem) {
        const int na = min(kMaxSrcSmem, d.K_src - a0);
        __syncthreads();
        // one warp per source row: load, normalise, store
        for (int a = warp; a < na; a += kSimThreads / 32) {
            const int i = src[(long long)unit * d.K_src + a0 + a];
            const T *kp = Sh + (long long)i * ss.v[2] + lane * 4;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (lane * 4 >= kD) {
                // a row of 64 elements takes the first 16 lanes
            } else if constexpr (sizeof(T) == 2) {
                const uint2 raw = *reinterpret_cast<const uint2 *>(kp);
                v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xffff0000u);
                v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xffff0000u);
            } else {
                const float4 raw = *reinterpret_cast<const float4 *>(kp);
                v[0] = raw.x; v[1] = raw.y; v[2] = raw.z; v[3] = raw.w;
            }
            const float n2 = warp_sum(v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3]);
            const float inv = 1.0f / fmaxf(sqrtf(n2), kNormEps);
            if (lane * 4 < kD)
                *reinterpret_cast<float4 *>(srows + a * kD + lane * 4) =
                    make_float4(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv);
        }
        __syncthreads();
        for (int j = j0 + threadIdx.x; j < j1; j += kSimThreads) {
            float k[kD];
            float n2 = 0.f;
#pragma unroll
            for (int c = 0; c < kD / 8; ++c) {
                float v[8];
                load8(Kh + (long long)j * ks.v[2] + c * 8, v);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    k[c * 8 + e] = v[e];
                    n2 = fmaf(v[e], v[e], n2);
                }
            }
            const float inv = 1.0f / fmaxf(sqrtf(n2), kNormEps);
            for (int a = 0; a < na; ++a) {
                const float4 *sv = reinterpret_cast<const float4 *>(srows + a * kD);
                float a0f = 0.f, a1f = 0.f, a2f = 0.f, a3f = 0.f;
#pragma unroll
                for (int c = 0; c < kD / 4; ++c) {
                    const float4 x = sv[c];
                    a0f = fmaf(x.x, k[4 * c], a0f);
                    a1f = fmaf(x.y, k[4 * c + 1], a1f);
                    a2f = fmaf(x.z, k[4 * c + 2], a2f);
                    a3f = fmaf(x.w, k[4 * c + 3], a3f);
                }
                float e = ((a0f + a1f) + (a2f + a3f)) * inv;
                e = fminf(fmaxf(e, -1.0f), 1.0f);
                sims[((long long)unit * d.K_src + a0 + a) * d.N + j] = e;
            }
        }
    }
}

// T rounds of s_j <- s_j * (1 - lambda * max(e_ij, 0)) over the fixed neighbour lists.
// Sources are applied one after another (threads span one source's m distinct neighbours), so
// overlapping neighbourhoods multiply deterministically.  grid units, block 256.
// nbr_idx / nbr_e [units][K_src][m].
__global__ void decay_rounds_kernel(Dims d, const int *__restrict__ nbr_idx,
                                    const float *__restrict__ nbr_e, float *__restrict__ scores)
{
    const int unit = blockIdx.x;
    float *s = scores + (long long)unit * d.N;
    const int *ni = nbr_idx + (long long)unit * d.K_src * d.m;
    const float *ne = nbr_e + (long long)unit * d.K_src * d.m;
    for (int t = 0; t < d.T; ++t) {
        for (int a = 0; a < d.K_src; ++a) {
            for (int u = threadIdx.x; u < d.m; u += blockDim.x) {
                const int j = ni[a * d.m + u];
                s[j] = d.signal == GRAPHKV_SIGNAL_EVICT ? -INFINITY
                                                        : s[j] * signal_factor(ne[a * d.m + u], d.lambda, 1, d.signal);
            }
            __syncthreads();
        }
    }
}

}  // namespace graphkv
