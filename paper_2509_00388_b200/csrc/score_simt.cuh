// Step (I), SIMT fp32 path: SnapKV-style window-attention scores for any input dtype.
// Used for fp32 inputs and for a head dimension of 64 (the tensor-core path takes bf16 and 128
// only); kD = 64 or 128.  Two sweeps over the keys of a
// head: (1) per-row softmax statistics, (2) the column sums of the normalised probabilities.
#pragma once

#include "common.cuh"

namespace graphkv {

constexpr int kStatsChunk = 1024;   // keys per CTA in the statistics sweep
constexpr int kStatsTile = 32;      // keys staged in shared memory at a time
constexpr int kEmitThreads = 128;   // one key per thread in the emit sweep
constexpr int kEmitChunk = 512;     // keys per CTA in the emit sweep

// Row statistics of the softmax, in the log2 domain: for query row r and the keys of one chunk,
// mx = max_j l2[r][j], z = sum_j 2^(l2[r][j] - mx), l2 = (q.k / sqrt(D)) * log2(e), over the keys
// row r may see (prefix keys and window keys N + r' with r' <= r).
// grid (n_chunks, units), block = GW rounded up to a warp multiple.
// part [units][n_chunks][GW][2].
template <typename T, int kD>
__global__ void __launch_bounds__(kMaxRows) score_stats_simt(Dims d, const T *__restrict__ Q,
                                                            const T *__restrict__ K,
                                                            float *__restrict__ part,
                                                            int n_chunks, int *status_word)
{
    __shared__ __align__(16) float tile[kStatsTile * kD];
    const int unit = blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    const int r = threadIdx.x;
    const bool active = r < d.GW;
    const int g = active ? r / d.W : 0, rw = active ? r % d.W : 0;
    if (status_word && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *status_word = 0;

    float q[kD];
    {
        const T *qp = Q + b * d.qs[0] + (long long)(h * d.G + g) * d.qs[1] + rw * d.qs[2];
        const float scale = rsqrtf((float)kD) * kLog2e;
#pragma unroll
        for (int c = 0; c < kD / 8; ++c) {
            float v[8];
            load8(qp + c * 8, v);
#pragma unroll
            for (int e = 0; e < 8; ++e) q[c * 8 + e] = v[e] * scale;
        }
    }
    const T *Kh = K + b * d.ks[0] + (long long)h * d.ks[1];
    const int j0 = chunk * kStatsChunk;
    const int j1 = min(j0 + kStatsChunk, d.L);
    const int last_visible = d.N + rw;          // row r sees keys 0 .. N + rw
    float mx = kNegBig, z = 0.f;
    for (int t0 = j0; t0 < j1; t0 += kStatsTile) {
        const int nt = min(kStatsTile, j1 - t0);
        __syncthreads();
        for (int i = threadIdx.x; i < nt * (kD / 8); i += blockDim.x) {
            const int kk = i / (kD / 8), c = i % (kD / 8);
            float v[8];
            load8(Kh + (long long)(t0 + kk) * d.ks[2] + c * 8, v);
            float4 *dst = reinterpret_cast<float4 *>(tile + kk * kD + c * 8);
            dst[0] = make_float4(v[0], v[1], v[2], v[3]);
            dst[1] = make_float4(v[4], v[5], v[6], v[7]);
        }
        __syncthreads();
        if (!active) continue;
        for (int kk = 0; kk < nt; ++kk) {
            if (t0 + kk > last_visible) break;
            const float4 *kv = reinterpret_cast<const float4 *>(tile + kk * kD);
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
#pragma unroll
            for (int c = 0; c < kD / 4; ++c) {
                const float4 x = kv[c];
                acc0 = fmaf(q[4 * c], x.x, acc0);
                acc1 = fmaf(q[4 * c + 1], x.y, acc1);
                acc2 = fmaf(q[4 * c + 2], x.z, acc2);
                acc3 = fmaf(q[4 * c + 3], x.w, acc3);
            }
            const float l2 = (acc0 + acc1) + (acc2 + acc3);
            const float mn = fmaxf(mx, l2);
            z = z * exp2f(mx - mn) + exp2f(l2 - mn);
            mx = mn;
        }
    }
    if (active) {
        float *o = part + (((long long)unit * n_chunks + chunk) * d.GW + r) * 2;
        o[0] = mx;
        o[1] = z;
    }
}

// Second sweep: a[j] = sum_r 2^(l2[r][j] - mx_r) / Z_r for the prefix keys j of one head.
// grid (ceil(N / kEmitChunk), units), block kEmitThreads; dynamic shared memory holds the
// scaled queries [GW][D] fp32 and the merged row statistics.
template <typename T, int kD>
__global__ void __launch_bounds__(kEmitThreads) score_emit_simt(Dims d, const T *__restrict__ Q,
                                                              const T *__restrict__ K,
                                                              const float *__restrict__ part,
                                                              int n_chunks,
                                                              float *__restrict__ a_out)
{
    extern __shared__ __align__(16) float sm[];
    float *qs = sm;                         // [GW][D]
    float *row_mx = sm + d.GW * kD;   // [GW]
    float *row_w = row_mx + d.GW;           // [GW] = 1 / Z_r
    const int unit = blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;

    const float scale = rsqrtf((float)kD) * kLog2e;
    for (int i = threadIdx.x; i < d.GW * (kD / 8); i += blockDim.x) {
        const int r = i / (kD / 8), c = i % (kD / 8);
        const int g = r / d.W, rw = r % d.W;
        const T *qp = Q + b * d.qs[0] + (long long)(h * d.G + g) * d.qs[1] + rw * d.qs[2];
        float v[8];
        load8(qp + c * 8, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) qs[r * kD + c * 8 + e] = v[e] * scale;
    }
    for (int r = threadIdx.x; r < d.GW; r += blockDim.x) {
        const float *p = part + ((long long)unit * n_chunks * d.GW + r) * 2;
        float mx = kNegBig;
        for (int c = 0; c < n_chunks; ++c) mx = fmaxf(mx, p[(long long)c * d.GW * 2]);
        float z = 0.f;
        for (int c = 0; c < n_chunks; ++c)
            z += p[(long long)c * d.GW * 2 + 1] * exp2f(p[(long long)c * d.GW * 2] - mx);
        row_mx[r] = mx;
        row_w[r] = 1.0f / z;
    }
    __syncthreads();

    const T *Kh = K + b * d.ks[0] + (long long)h * d.ks[1];
    const int j0 = blockIdx.x * kEmitChunk;
    const int j1 = min(j0 + kEmitChunk, d.N);
    for (int j = j0 + threadIdx.x; j < j1; j += kEmitThreads) {
        float k[kD];
#pragma unroll
        for (int c = 0; c < kD / 8; ++c) {
            float v[8];
            load8(Kh + (long long)j * d.ks[2] + c * 8, v);
#pragma unroll
            for (int e = 0; e < 8; ++e) k[c * 8 + e] = v[e];
        }
        float acc = 0.f;
        for (int r = 0; r < d.GW; ++r) {
            const float4 *qv = reinterpret_cast<const float4 *>(qs + r * kD);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int c = 0; c < kD / 4; ++c) {
                const float4 x = qv[c];
                a0 = fmaf(x.x, k[4 * c], a0);
                a1 = fmaf(x.y, k[4 * c + 1], a1);
                a2 = fmaf(x.z, k[4 * c + 2], a2);
                a3 = fmaf(x.w, k[4 * c + 3], a3);
            }
            const float l2 = (a0 + a1) + (a2 + a3);
            acc = fmaf(exp2f(l2 - row_mx[r]), row_w[r], acc);
        }
        a_out[(long long)unit * d.N + j] = acc;
    }
}

// 1-D pooling, stride 1, same length: the maximum over the positions inside [0,N), or (avg) the
// sum over them divided by kp (zeros outside the row).  grid (ceil(N/256), units), block 256.
__global__ void pool_max_kernel(int N, int kp, int avg, const float *__restrict__ a,
                                float *__restrict__ s)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= N) return;
    const float *row = a + (long long)blockIdx.y * N;
    const int half = (kp - 1) / 2;
    const int lo = max(j - half, 0), hi = min(j + half, N - 1);
    float best = row[lo];
    if (avg) {
        for (int t = lo + 1; t <= hi; ++t) best += row[t];
        best /= (float)kp;
    } else {
        for (int t = lo + 1; t <= hi; ++t) best = fmaxf(best, row[t]);
    }
    s[(long long)blockIdx.y * N + j] = best;
}

}  // namespace graphkv
