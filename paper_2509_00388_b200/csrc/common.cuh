// Shared device/host helpers of the GraphKV CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "graphkv.h"

namespace graphkv {

constexpr int kHeadDim = 128;          // D of the tensor-core kernels (the SIMT kernels also take 64)
constexpr int kMaxRows = 256;          // G*W limit (one TMEM accumulator tile of query rows)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegBig = -1.0e30f;    // finite stand-in for -inf in running maxima
constexpr float kNormEps = 1e-12f;     // floor of a key norm in Eq. 1

// Shape of one call, resolved once on the host and passed by value to kernels.
struct Dims {
    int batch, hq, hkv, G, W, N, L, GW;
    int D;                     // head dimension: 128, or 64 (SIMT kernels only)
    int B, kp, K_src, m, T;
    float lambda;
    int units;                 // batch * hkv independent (sequence, KV head) problems
    int bf16;                  // inputs are bf16 (else fp32)
    int pool_avg;              // mean pooling (zeros outside the row) instead of max pooling
    int signal;                // graphkv_signal
    int reselect;              // sources re-picked every round
    long long qs[3], ks[3], vs[3];
};

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---- element access: 8 consecutive elements of a row as fp32 --------------------------------
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8])
{
    const uint4 raw = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ void load8(const float *p, float (&v)[8])
{
    const float4 a = *reinterpret_cast<const float4 *>(p);
    const float4 b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Order-preserving map fp32 -> uint32 (larger float <=> larger key); -0 and +0 map to one key.
__device__ __forceinline__ uint32_t float_to_key(float x)
{
    uint32_t u = __float_as_uint(x);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// A listed edge: cosine and the position of the key it leads to.
struct Cand {
    float e;
    int j;
};
constexpr int kCandCap = 64;            // candidate slots per (source, key chunk)
constexpr int kCandBins = 256;          // cosine bins of the per-source candidate histogram
constexpr float kCandEmpty = -2.0f;     // cosine stored in an unused slot (valid cosines are >= -1)

// Bin of a cosine: floor(e * kCandBins) clamped to [0, kCandBins); e >= b / kCandBins exactly when
// its bin is >= b (the scaling is exact in binary floating point).
__device__ __forceinline__ int cand_bin(float e)
{
    return min(max(static_cast<int>(floorf(e * kCandBins)), 0), kCandBins - 1);
}

// Order-preserving 64-bit image of an edge: larger cosine first, then lower position.
__device__ __forceinline__ unsigned long long edge_key(float e, int j)
{
    return (static_cast<unsigned long long>(float_to_key(e)) << 32) |
           static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(j));
}

// Programmatic dependent launch: let the next kernel of the stream start its prologue, and wait
// (in that next kernel) until the kernels before it have completed and their writes are visible.
__device__ __forceinline__ void pdl_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- optional phase timing (build with -DGRAPHKV_PHASE_TIMING) --------------------------------
// One thread per CTA stamps %globaltimer at phase boundaries; at the end of the kernel the
// differences are added into per-kernel tables that graphkv_phase_timing_read copies out.  In the
// normal build the marks compile to nothing.
constexpr int kPhaseKernels = 8, kPhaseSlots = 24;
#ifdef GRAPHKV_PHASE_TIMING
__device__ unsigned long long g_phase_sum[kPhaseKernels][kPhaseSlots];
__device__ unsigned long long g_phase_max[kPhaseKernels][kPhaseSlots];
__device__ unsigned long long g_phase_cnt[kPhaseKernels];
struct PhaseClock {
    unsigned long long t[kPhaseSlots];
    int n;
    bool on;
    __device__ explicit PhaseClock(bool o) : n(0), on(o) {}
    __device__ __forceinline__ void mark()
    {
        if (on && n < kPhaseSlots) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t[n++]));
    }
    // slot 0: first to last mark; slot i: mark i-1 to mark i
    __device__ void flush(int k)
    {
        if (!on || n < 2) return;
        for (int i = 1; i < n; ++i) {
            atomicAdd(&g_phase_sum[k][i], t[i] - t[i - 1]);
            atomicMax(&g_phase_max[k][i], t[i] - t[i - 1]);
        }
        atomicAdd(&g_phase_sum[k][0], t[n - 1] - t[0]);
        atomicMax(&g_phase_max[k][0], t[n - 1] - t[0]);
        atomicAdd(&g_phase_cnt[k], 1ull);
    }
};
#else
struct PhaseClock {
    __device__ explicit PhaseClock(bool) {}
    __device__ __forceinline__ void mark() {}
    __device__ __forceinline__ void flush(int) {}
};
#endif

// What a listed edge of cosine e does to its neighbour's score over T rounds of a fixed graph, as
// a factor: (1 - lambda*max(e,0))^T for the decay signal, (1 + lambda*max(e,0))^T for the enhanced
// one.  (The evicted signal is no factor: the score becomes -inf.)
__device__ __forceinline__ float signal_factor(float e, float lambda, int T, int signal)
{
    const float x = lambda * fmaxf(e, 0.f);
    const float f = signal == GRAPHKV_SIGNAL_ENHANCE ? 1.0f + x : 1.0f - x;
    float pw = f;
    for (int t = 1; t < T; ++t) pw *= f;
    return pw;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace graphkv
