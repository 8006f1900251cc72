// Exact top-k of fp32 rows with lower-index-first tie-breaking (Eq. 2 sources, Eq. 3
// neighbourhoods, the final k_l selection).  One CTA per row: a 4 x 8-bit most-significant-digit
// radix search finds the k-th largest value, then an ordered compaction emits exactly k indices
// in ascending position.
#pragma once

#include "common.cuh"

namespace graphkv {

constexpr int kSelectThreads = 1024;

struct SelectArgs {
    const float *x;          // rows of candidates
    long long row_stride;    // elements between rows
    int n;                   // candidates per row
    int k;                   // items to keep, 1 <= k <= n (k <= n-1 when a skip index is given)
    const int *skip;         // optional: one excluded index per row (Eq. 3's j != i)
    int *idx_out;            // [rows][k] ascending indices
    float *val_out;          // optional [rows][k]: x at those indices
};

// Inclusive scan of one 32-bit value per thread over the CTA (kSelectThreads threads).
// Returns the inclusive prefix; *total receives the CTA-wide sum.  `warp_tot` is 33 words.
__device__ __forceinline__ uint32_t block_scan_inclusive(uint32_t v, uint32_t *warp_tot,
                                                         uint32_t *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_tot[lane] = w;      // inclusive totals of warps 0..lane
    }
    __syncthreads();
    const uint32_t before = warp == 0 ? 0u : warp_tot[warp - 1];
    *total = warp_tot[31];
    const uint32_t out = v + before;
    __syncthreads();             // warp_tot may be reused by the next call
    return out;
}

__global__ void __launch_bounds__(kSelectThreads) topk_select_kernel(SelectArgs a)
{
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[33];
    __shared__ uint32_t s_bin, s_remaining;
    const int row = blockIdx.x;
    const float *x = a.x + (long long)row * a.row_stride;
    const int skip = a.skip ? a.skip[row] : -1;
    const int tid = threadIdx.x, lane = tid & 31;
    const int n_iter = ceil_div(a.n, kSelectThreads);

    // ---- radix search for the key of the k-th largest candidate ----
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)a.k;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int it = 0; it < n_iter; ++it) {
            const int i = it * kSelectThreads + tid;
            bool valid = i < a.n && i != skip;
            uint32_t bin = 0;
            if (valid) {
                const uint32_t u = float_to_key(x[i]);
                valid = (u & mask) == prefix;
                bin = (u >> shift) & 255u;
            }
            // lanes sharing the first valid lane's digit are counted with one atomic; the others
            // add for themselves
            const unsigned vm = __ballot_sync(0xffffffffu, valid);
            if (vm) {
                const int leader = __ffs(vm) - 1;
                const uint32_t lbin = __shfl_sync(0xffffffffu, bin, leader);
                const bool same = valid && bin == lbin;
                const unsigned sm = __ballot_sync(0xffffffffu, same);
                if (lane == leader) atomicAdd(&hist[lbin], (uint32_t)__popc(sm));
                else if (valid && !same) atomicAdd(&hist[bin], 1u);
            }
        }
        __syncthreads();
        // bins in descending order: position p holds bin 255 - p
        uint32_t c = tid < 256 ? hist[255 - tid] : 0u, total;
        const uint32_t incl = block_scan_inclusive(c, warp_tot, &total);
        if (tid < 256 && incl >= remaining && incl - c < remaining) {
            s_bin = 255u - tid;
            s_remaining = remaining - (incl - c);
        }
        __syncthreads();
        prefix |= s_bin << shift;
        mask |= 255u << shift;
        remaining = s_remaining;
        __syncthreads();
    }
    const uint32_t thr = prefix;          // key of the k-th largest; `remaining` ties are taken

    // ---- ordered compaction: greater-than always, equal only the `remaining` lowest indices ----
    uint32_t run_gt = 0, run_eq = 0;
    int *out = a.idx_out + (long long)row * a.k;
    float *vout = a.val_out ? a.val_out + (long long)row * a.k : nullptr;
    for (int it = 0; it < n_iter; ++it) {
        const int i = it * kSelectThreads + tid;
        uint32_t gt = 0, eq = 0;
        float xv = 0.f;
        if (i < a.n && i != skip) {
            xv = x[i];
            const uint32_t u = float_to_key(xv);
            gt = u > thr;
            eq = u == thr;
        }
        uint32_t total;
        const uint32_t incl = block_scan_inclusive(gt | (eq << 16), warp_tot, &total);
        const uint32_t gt_before = run_gt + (incl & 0xffffu) - gt;
        const uint32_t eq_before = run_eq + (incl >> 16) - eq;
        if (gt || (eq && eq_before < remaining)) {
            const uint32_t pos = gt_before + min(eq_before, remaining);
            out[pos] = i;
            if (vout) vout[pos] = xv;
        }
        run_gt += total & 0xffffu;
        run_eq += total >> 16;
        if (run_gt + min(run_eq, remaining) >= (uint32_t)a.k) break;
    }
}

}  // namespace graphkv
