// Row-wise stages on thread-block clusters: one cluster of C CTAs owns the N scores of one
// (sequence, KV head) unit, each CTA keeping a contiguous chunk of the row in shared memory.
//
//   pool_select_kernel   max pooling of the attention mass (step (I), last part) and the
//                        source nodes of Eq. 2: top-k of the pooled scores.
//   finish_kernel        the neighbourhoods of Eq. 3 merged from the per-chunk candidate lists of
//                        the similarity sweep, the decay rounds of Eq. 5 / Algorithm 2 over them,
//                        the final k_l selection and the gather of the compact cache.
//
// Every exact top-k here is a most-significant-digit radix search over the order-preserving
// uint32 image of the fp32 scores (digits of 11, 11 and 10 bits).  Per digit each CTA
// histograms its chunk, the cluster reduces the histograms through distributed shared memory,
// and every CTA locates the digit of the k-th largest value.  The kept indices come out in
// ascending position; among equal values the lowest indices are kept.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace graphkv {
namespace cs {

namespace cg = cooperative_groups;

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;
constexpr int kMaxChunk = 32768;       // scores of a row one CTA keeps in shared memory
constexpr int kMaxCluster = 8;
constexpr int kMaxHalo = 64;           // (pool_kernel - 1) / 2 the pooling path handles
constexpr int kMaxPerThread = kMaxChunk / kThreads;
constexpr int kStage = 2048;           // neighbour-list entries staged in shared memory at a time
constexpr int kMergeWarps = 8;         // groups of four warps of a CTA, one source each at a time
constexpr int kSurvCap = 256;          // merged candidates one warp ranks in shared memory
static_assert(kMergeWarps * kSurvCap * sizeof(Cand) <= 2 * kStage * 4, "survivors reuse the staging area");

// Shared-memory carve-up common to both kernels (dynamic shared memory, 16-byte aligned).
struct Smem {
    uint32_t *hist;       // [kBins] this CTA's digit histogram
    uint32_t *tot;        // [kBins] cluster-wide histogram (every CTA holds a copy)
    uint32_t *wcnt;       // [2 * kWarps] per-warp counts
    uint32_t *misc;       // [16] broadcast words and this CTA's published counts
    int *st_idx;          // [kStage] staged neighbour positions, relative to the chunk
    float *st_f;          // [kStage] their decay factors
    float *vals;          // [halo + chunk + halo]
};

__host__ __device__ inline size_t smem_bytes(int chunk, int halo)
{
    return (size_t)(2 * kBins + 2 * kWarps + 16 + 2 * kStage) * 4 + (size_t)(chunk + 2 * halo + 8) * 4;
}

__device__ __forceinline__ Smem carve(uint8_t *raw, int halo)
{
    Smem s;
    s.hist = reinterpret_cast<uint32_t *>(raw);
    s.tot = s.hist + kBins;
    s.wcnt = s.tot + kBins;
    s.misc = s.wcnt + 2 * kWarps;
    s.st_idx = reinterpret_cast<int *>(s.misc + 16);
    s.st_f = reinterpret_cast<float *>(s.st_idx + kStage);
    s.vals = s.st_f + kStage;
    (void)halo;
    return s;
}

// Result of the radix search: elements whose masked key exceeds `prefix` are kept, and of those
// whose masked key equals it the `remaining` lowest indices.
struct Threshold {
    uint32_t prefix, mask, remaining;
};

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// k-th largest of the cluster's row.  vals: this CTA's chunk (n_local elements, shared memory).
// All CTAs of the cluster call this with the same k (1 <= k <= elements in the row) and return
// the same Threshold.  Executes the same number of cluster barriers in every CTA.
__device__ Threshold cluster_kth(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                 const float *vals, int n_local, uint32_t k)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    Threshold th{0u, 0u, k};
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t nb = pass == 2 ? 1024u : 2048u;
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0u;
        __syncthreads();
        for (int i0 = 0; i0 < n_local; i0 += kThreads) {
            const int i = i0 + tid;
            bool valid = i < n_local;
            uint32_t bin = 0;
            if (valid) {
                const uint32_t u = float_to_key(vals[i]);
                valid = (u & th.mask) == th.prefix;
                bin = (u >> shift) & (nb - 1u);
            }
            // lanes sharing the first valid lane's digit are counted with one atomic (scores of a
            // row often crowd into one digit); the others add for themselves
            const unsigned vm = __ballot_sync(0xffffffffu, valid);
            if (vm) {
                const int leader = __ffs(vm) - 1;
                const uint32_t lbin = __shfl_sync(0xffffffffu, bin, leader);
                const bool same = valid && bin == lbin;
                const unsigned sm = __ballot_sync(0xffffffffu, same);
                if (lane == leader) atomicAdd(&s.hist[lbin], (uint32_t)__popc(sm));
                else if (valid && !same) atomicAdd(&s.hist[bin], 1u);
            }
        }
        __syncthreads();
        const uint32_t *total = s.hist;
        if (C > 1) {
            cl.sync();                                   // every CTA's histogram is complete
            const int slice = kBins / C;
            if (tid < slice) {
                const int bin = rank * slice + tid;
                uint32_t sum = 0;
                for (int p = 0; p < C; ++p) sum += cl.map_shared_rank(s.hist, p)[bin];
                for (int p = 0; p < C; ++p) cl.map_shared_rank(s.tot, p)[bin] = sum;
            }
            cl.sync();                                   // every CTA's copy of the totals is complete
            total = s.tot;
        }
        // walk the digits from the largest down: thread t owns digits nb-1-2t and nb-2-2t
        uint32_t c0 = 0, c1 = 0;
        if (2 * tid < (int)nb) {
            c0 = total[nb - 1 - 2 * tid];
            c1 = total[nb - 2 - 2 * tid];
        }
        uint32_t incl = warp_incl_scan(c0 + c1, lane);
        if (lane == 31) s.wcnt[warp] = incl;
        __syncthreads();
        if (warp == 0) s.wcnt[lane] = warp_incl_scan(s.wcnt[lane], lane);
        __syncthreads();
        incl += warp == 0 ? 0u : s.wcnt[warp - 1];
        const uint32_t before0 = incl - c0 - c1, before1 = before0 + c0;
        if (before0 < th.remaining && before0 + c0 >= th.remaining) {
            s.misc[0] = nb - 1 - 2 * tid;
            s.misc[1] = th.remaining - before0;
            s.misc[2] = c0;
        } else if (before1 < th.remaining && before1 + c1 >= th.remaining) {
            s.misc[0] = nb - 2 - 2 * tid;
            s.misc[1] = th.remaining - before1;
            s.misc[2] = c1;
        }
        __syncthreads();
        th.prefix |= s.misc[0] << shift;
        th.mask |= (nb - 1u) << shift;
        th.remaining = s.misc[1];
        const bool whole_class = s.misc[2] == th.remaining;
        __syncthreads();
        if (whole_class) break;       // every element of the threshold class is kept
    }
    return th;
}

// Ascending positions of the kept elements of the cluster's row -> out[0..k).  Returns nothing;
// ends with the writes of this CTA issued (callers fence before another CTA reads them).
// One cluster barrier.
__device__ void cluster_emit_sorted(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                    const float *vals, int n_local, int base, Threshold th,
                                    int *out)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // warp w owns the contiguous segment [w * seg, (w + 1) * seg) of the chunk
    const int seg = ((n_local + kWarps - 1) / kWarps + 31) & ~31;
    const int lo = min(warp * seg, n_local), hi = min(lo + seg, n_local);
    uint32_t gt = 0, eq = 0;
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        uint32_t mk = 0;
        const bool in = i < hi;
        if (in) mk = float_to_key(vals[i]) & th.mask;
        gt += __popc(__ballot_sync(0xffffffffu, in && mk > th.prefix));
        eq += __popc(__ballot_sync(0xffffffffu, in && mk == th.prefix));
    }
    if (lane == 0) {
        s.wcnt[warp] = gt;
        s.wcnt[kWarps + warp] = eq;
    }
    __syncthreads();
    if (warp == 0) {
        const uint32_t g = s.wcnt[lane], e = s.wcnt[kWarps + lane];
        const uint32_t gi = warp_incl_scan(g, lane), ei = warp_incl_scan(e, lane);
        s.wcnt[lane] = gi - g;                  // exclusive prefix over warps
        s.wcnt[kWarps + lane] = ei - e;
        if (lane == 31) {
            s.misc[4] = gi;                     // this CTA's totals, read by the other ranks
            s.misc[5] = ei;
        }
    }
    __syncthreads();
    uint32_t gt_before = s.wcnt[warp], eq_before = s.wcnt[kWarps + warp];
    if (C > 1) {
        cl.sync();
        for (int p = 0; p < rank; ++p) {
            const uint32_t *pm = cl.map_shared_rank(s.misc, p);
            gt_before += pm[4];
            eq_before += pm[5];
        }
    }
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        uint32_t mk = 0;
        const bool in = i < hi;
        if (in) mk = float_to_key(vals[i]) & th.mask;
        const bool is_gt = in && mk > th.prefix, is_eq = in && mk == th.prefix;
        const unsigned bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
        const unsigned below = (1u << lane) - 1u;
        const uint32_t g = gt_before + __popc(bg & below), e = eq_before + __popc(be & below);
        if (is_gt || (is_eq && e < th.remaining)) out[g + min(e, th.remaining)] = base + i;
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
}

// The m largest edges (cosine descending, position ascending) of the lists when too many tie at
// the bound: exact m-th largest by bisection over the lists themselves.  One warp; returns the
// number of survivors written (m, or fewer when fewer edges are listed).
__device__ int merge_exact(const Cand *cand, int slots, int m, Cand *surv)
{
    const int lane = threadIdx.x & 31;
    int ns = 0;
    {
        // too many ties at the bound: exact m-th largest by bisection over the lists themselves
        unsigned long long t64 = 0ull;
        for (int bit = 63; bit >= 0; --bit) {
            const unsigned long long cut = t64 | (1ull << bit);
            int n = 0;
            for (int i = lane; i < slots; i += 32) {
                const unsigned long long raw = __ldcg(reinterpret_cast<const unsigned long long *>(cand + i));
                const float e = __uint_as_float(static_cast<uint32_t>(raw));
                n += e >= -1.0f && edge_key(e, static_cast<int>(raw >> 32)) >= cut;
            }
            n = __reduce_add_sync(0xffffffffu, n);
            if (n >= m) t64 = cut;
        }
        ns = 0;
        for (int i0 = 0; i0 < slots; i0 += 32) {
            const int i = i0 + lane;
            bool keep = false;
            Cand cd{0.f, 0};
            if (i < slots) {
                const unsigned long long raw = __ldcg(reinterpret_cast<const unsigned long long *>(cand + i));
                cd.e = __uint_as_float(static_cast<uint32_t>(raw));
                cd.j = static_cast<int>(raw >> 32);
                keep = cd.e >= -1.0f && edge_key(cd.e, cd.j) >= t64;
            }
            const unsigned bm = __ballot_sync(0xffffffffu, keep);
            const int pos = ns + __popc(bm & ((1u << lane) - 1u));
            if (keep && pos < kSurvCap) surv[pos] = cd;
            ns += __popc(bm);
        }
    }
    __syncwarp();
    return min(ns, kSurvCap);
}

// Eq. 3 for one source: the m largest edges (cosine descending, position ascending) among the
// candidate lists its key chunks wrote.  One warp; `surv` holds kSurvCap entries of shared memory.
// The lists together hold every member of the top-m, and `hist` counts the listed edges per cosine
// bin: the highest bin b with at least m listed edges in bins >= b bounds the m-th largest from
// below, so only edges with e >= b / kCandBins need ranking.
__device__ void merge_neighbours(const Cand *cand, const uint32_t *hist, int chunks, int m,
                                 Cand *surv, int *ns_sh, int bar_id, int wg, int *nbr_idx, float *nbr_e)
{
    const int lane = threadIdx.x & 31;
    constexpr int kPer = kCandBins / 32;
    // lane l holds bins [l * kPer, (l + 1) * kPer); walk down from the top bin
    uint32_t h[kPer], mine = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        h[q] = __ldcg(hist + lane * kPer + q);
        mine += h[q];
    }
    uint32_t above = 0;                       // listed edges in the lanes above this one
    {
        uint32_t incl = mine;              // suffix sum over lanes, log steps
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_down_sync(0xffffffffu, incl, o);
            if (lane + o < 32) incl += t;
        }
        above = incl - mine;
    }
    int bstar = -1;
    uint32_t run = above;
#pragma unroll
    for (int q = kPer - 1; q >= 0; --q) {
        run += h[q];
        if (bstar < 0 && run >= (uint32_t)m) bstar = lane * kPer + q;
    }
    // the answer is the highest bin found by any lane
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bstar = max(bstar, __shfl_xor_sync(0xffffffffu, bstar, o));
    const float bound = bstar <= 0 ? -1.0f : (float)bstar / (float)kCandBins;

    // the four warps of the group take interleaved blocks of 256 slots, eight loads in flight per lane
    if (wg == 0 && lane == 0) *ns_sh = 0;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    const int slots = chunks * kCandCap;
    for (int i0 = wg * 256; i0 < slots; i0 += 4 * 256) {
        unsigned long long raw[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + q * 32 + lane;
            raw[q] = i < slots ? __ldcg(reinterpret_cast<const unsigned long long *>(cand + i)) : 0ull;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + q * 32 + lane;
            const Cand cd{__uint_as_float(static_cast<uint32_t>(raw[q])), static_cast<int>(raw[q] >> 32)};
            const bool keep = i < slots && cd.e >= bound;
            const unsigned bm = __ballot_sync(0xffffffffu, keep);
            if (bm) {
                int basep = 0;
                if (lane == 0) basep = atomicAdd(ns_sh, __popc(bm));
                basep = __shfl_sync(0xffffffffu, basep, 0);
                const int pos = basep + __popc(bm & ((1u << lane) - 1u));
                if (keep && pos < kSurvCap) surv[pos] = cd;
            }
        }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    int ns = *ns_sh;
    if (ns > kSurvCap) {
        if (wg == 0) ns = merge_exact(cand, slots, m, surv);
        if (wg == 0 && lane == 0) *ns_sh = ns;
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        ns = *ns_sh;
    }
    // rank by counting: all keys are distinct (distinct positions)
    for (int i = wg * 32 + lane; i < ns; i += 128) {
        const Cand me = surv[i];
        const unsigned long long k = edge_key(me.e, me.j);
        int rank = 0;
        for (int t = 0; t < ns; ++t) rank += edge_key(surv[t].e, surv[t].j) > k;
        if (rank < m) {
            nbr_idx[rank] = me.j;
            nbr_e[rank] = me.e;
        }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");      // the list may be reused
}

// vals[i] = row[base + i] for i in [lo, hi) (positions outside [0, N) read as `fill`), all threads
// of the CTA, eight loads in flight per thread ahead of the shared-memory stores.
__device__ __forceinline__ void load_chunk(const float *row, int base, int lo, int hi, int N,
                                           float *vals, float fill)
{
    for (int i0 = lo + (int)threadIdx.x; i0 < hi; i0 += 8 * kThreads) {
        float r[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int i = i0 + k * kThreads, j = base + i;
            r[k] = (i < hi && j >= 0 && j < N) ? __ldcg(row + j) : fill;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int i = i0 + k * kThreads;
            if (i < hi) vals[i] = r[k];
        }
    }
}

struct PoolSelectArgs {
    Dims d;
    int C, chunk, halo;
    int unit0;
    const float *a;        // [units][N] attention mass before pooling, or nullptr: no pooling
    float *s;              // [units][N] scores: written when pooling, read otherwise
    int k;                 // sources to pick (0: none)
    int *src_out;          // [units][k] ascending positions
    const uint32_t *mass_hist;  // optional [units][kBins]: histogram of values the scores dominate
    uint32_t *zero;        // optional: [units][zero_words] words this launch clears for later kernels
    int zero_words;
    int wait_prior;        // launched with programmatic stream serialization
};

// grid = units * C CTAs in clusters of C; block kThreads.  kPer >= chunk / kThreads: elements of
// the chunk a thread pools (a power of two up to kMaxPerThread).
// Top-k of the cluster's row when a histogram of values that the row dominates elementwise is at
// hand (the pooled scores against the histogram of the attention mass before pooling: pooling only
// raises values, so the k-th largest pooled score is at least the k-th largest mass).  The highest
// digit b with k histogram entries in digits >= b therefore bounds the k-th largest row value from
// below; the row's elements with digit >= b are few (at most pool_kernel times the histogram's
// count); each CTA lists its own, the first CTA pulls the lists through distributed shared memory
// and ranks them by counting.  Returns false (in every CTA alike, nothing written) when they exceed kThreads; the
// caller then runs the radix search.  `mass_hist`: kBins counts of the top 11 bits.
// c0, c1: the histogram's counts of digits kBins-1-2t and kBins-2-2t for thread t (the caller loads
// them early, ahead of the pooling).
__device__ bool cluster_topk_bounded(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                     const float *vals, int n_local, int base, int k,
                                     uint32_t c0, uint32_t c1, int *out)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // digit b: walk the histogram from the top (thread t owns digits kBins-1-2t and kBins-2-2t)
    uint32_t incl = warp_incl_scan(c0 + c1, lane);
    if (lane == 31) s.wcnt[warp] = incl;
    if (tid == 0) {
        s.misc[0] = 0u;          // digit 0 when the histogram holds fewer than k entries
        s.misc[7] = 0u;          // this CTA's candidate counter
    }
    __syncthreads();
    if (warp == 0) s.wcnt[lane] = warp_incl_scan(s.wcnt[lane], lane);
    __syncthreads();
    incl += warp == 0 ? 0u : s.wcnt[warp - 1];
    const uint32_t before0 = incl - c0 - c1, before1 = before0 + c0;
    if (before0 < (uint32_t)k && before0 + c0 >= (uint32_t)k) s.misc[0] = kBins - 1 - 2 * tid;
    else if (before1 < (uint32_t)k && before1 + c1 >= (uint32_t)k) s.misc[0] = kBins - 2 - 2 * tid;
    __syncthreads();
    const uint32_t bdigit = s.misc[0];
    // this CTA's candidates -> its own lists (keys in hist, positions in tot)
    for (int i0 = 0; i0 < n_local; i0 += kThreads) {
        const int i = i0 + tid;
        uint32_t key = 0;
        bool cand = false;
        if (i < n_local) {
            key = float_to_key(vals[i]);
            cand = (key >> 21) >= bdigit;
        }
        const unsigned bm = __ballot_sync(0xffffffffu, cand);
        if (bm) {
            uint32_t basep = 0;
            if (lane == 0) basep = atomicAdd(&s.misc[7], (uint32_t)__popc(bm));
            basep = __shfl_sync(0xffffffffu, basep, 0);
            const uint32_t pos = basep + __popc(bm & ((1u << lane) - 1u));
            if (cand && pos < (uint32_t)kThreads) {
                s.hist[pos] = key;
                s.tot[pos] = (uint32_t)(base + i);
            }
        }
    }
    __syncthreads();
    if (C > 1) cl.sync();
    // candidate t of the concatenated lists; every CTA learns the total, the first CTA pulls them
    // (lane p reads CTA p's count, so the remote reads overlap; the walk runs on the copies)
    uint32_t n_lane = 0;
    if (lane < C) n_lane = C > 1 ? cl.map_shared_rank(s.misc, lane)[7] : s.misc[7];
    uint32_t total = 0;
    int mine_p = -1, mine_j = 0;
    for (int p = 0; p < C; ++p) {
        const uint32_t n_p = __shfl_sync(0xffffffffu, n_lane, p);
        if (n_p > (uint32_t)kThreads) total = 0x40000000u;       // a list overflowed
        if (tid >= (int)total && tid < (int)(total + n_p)) {
            mine_p = p;
            mine_j = tid - (int)total;
        }
        total += n_p;
    }
    if (total > (uint32_t)kThreads || total < (uint32_t)k) {
        if (C > 1) cl.sync();                              // nobody still reads another CTA's counter
        return false;
    }
    if (rank == 0) {
        uint32_t key = 0, pos = 0;
        if (mine_p >= 0) {
            key = (C > 1 ? cl.map_shared_rank(s.hist, mine_p) : s.hist)[mine_j];
            pos = (C > 1 ? cl.map_shared_rank(s.tot, mine_p) : s.tot)[mine_j];
        }
        __syncthreads();                                   // own list read before it is overwritten
        uint32_t *ck = s.hist, *ci = s.tot;
        if (mine_p >= 0) {
            ck[tid] = key;
            ci[tid] = pos;
        }
        __syncthreads();
        // a warp per candidate: its rank among all (value descending, position ascending)
        int *kept = s.st_idx;                              // [k] positions of the kept, unordered
        if (tid == 0) s.misc[3] = 0u;      // (word 7 may still be read by the other CTAs)
        __syncthreads();
        if (total <= (uint32_t)(kThreads / 4)) {
            // few candidates: four threads each, every one walking a quarter of the list
            const int t = tid >> 2, sub = tid & 3;
            const bool live = t < (int)total;
            const uint32_t kt = live ? ck[t] : 0u, pt = live ? ci[t] : 0u;
            int r = 0;
            if (live) {
#pragma unroll 4
                for (int u = sub; u < (int)total; u += 4) {
                    const uint32_t ku = ck[u], pu = ci[u];
                    r += (int)(ku > kt) | ((int)(ku == kt) & (int)(pu < pt));
                }
            }
            r += __shfl_xor_sync(0xffffffffu, r, 1);
            r += __shfl_xor_sync(0xffffffffu, r, 2);
            if (live && sub == 0 && r < k) kept[atomicAdd(&s.misc[3], 1u)] = (int)pt;
        } else {
            for (int t = warp; t < (int)total; t += kWarps) {
                const uint32_t kt = ck[t], pt = ci[t];
                int r = 0;
                for (int u = lane; u < (int)total; u += 32) {
                    const uint32_t ku = ck[u], pu = ci[u];
                    r += (int)(ku > kt) | ((int)(ku == kt) & (int)(pu < pt));
                }
                r = __reduce_add_sync(0xffffffffu, r);
                if (lane == 0 && r < k) kept[atomicAdd(&s.misc[3], 1u)] = (int)pt;
            }
        }
        __syncthreads();
        // ascending positions: thread t places kept[t] by counting the smaller ones
        if (tid < k) {
            const int pt = kept[tid];
            int o = 0;
            for (int u = 0; u < k; ++u) o += kept[u] < pt;
            out[o] = pt;
        }
    }
    return true;
}

template <int kPer>
__global__ void __launch_bounds__(kThreads, 1) pool_select_kernel(PoolSelectArgs a)
{
    extern __shared__ __align__(16) uint8_t cs_smem[];
    cg::cluster_group cl = cg::this_cluster();
    const int C = a.C, rank = C > 1 ? (int)cl.block_rank() : 0;
    const int unit = a.unit0 + blockIdx.x / C;
    const Smem s = carve(cs_smem, a.halo);
    const int N = a.d.N, tid = threadIdx.x;
    const int base = rank * a.chunk;
    const int n_local = max(0, min(a.chunk, N - base));
    float *vals = s.vals + a.halo;
    float *row_s = a.s + (long long)unit * N;
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    if (a.zero)
        for (int i = rank * kThreads + tid; i < a.zero_words; i += C * kThreads)
            a.zero[(long long)unit * a.zero_words + i] = 0u;
    // this thread's two counts of the mass histogram, on their way while the row is pooled
    const bool bounded = a.mass_hist && a.k > 0 && a.k <= kThreads;
    uint32_t hc0 = 0, hc1 = 0;
    if (bounded) {
        const uint32_t *mh = a.mass_hist + (long long)unit * kBins;
        hc0 = __ldcg(mh + kBins - 1 - 2 * tid);
        hc1 = __ldcg(mh + kBins - 2 - 2 * tid);
    }
    if (a.a) {
        const float *row_a = a.a + (long long)unit * N;
        const int half = a.halo;
        if (n_local > 0) load_chunk(row_a, base, -half, n_local + half, N, vals, -INFINITY);
        __syncthreads();
        float pooled[kPer];
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int i = q * kThreads + tid;
            if (i < n_local) {
                float best = vals[i - half];
                for (int t = 1 - half; t <= half; ++t) best = fmaxf(best, vals[i + t]);
                pooled[q] = best;
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int i = q * kThreads + tid;
            if (i < n_local) {
                vals[i] = pooled[q];
                row_s[base + i] = pooled[q];
            }
        }
    } else {
        load_chunk(row_s, base, 0, n_local, N, vals, 0.f);
    }
    __syncthreads();
    if (a.k > 0) {
        int *out = a.src_out + (long long)unit * a.k;
        const bool done = bounded && cluster_topk_bounded(cl, C, rank, s, vals, n_local, base, a.k, hc0, hc1, out);
        if (!done) {
            const Threshold th = cluster_kth(cl, C, rank, s, vals, n_local, (uint32_t)a.k);
            cluster_emit_sorted(cl, C, rank, s, vals, n_local, base, th, out);
        }
    }
    if (C > 1) cl.sync();      // no CTA leaves while its shared memory may still be read
}

struct FinishArgs {
    Dims d;
    int C, chunk;
    int unit0;
    float *s;                  // [units][N] scores (decayed in place when has_graph)
    int *nbr_idx;              // [units][K_src][m] neighbour lists (has_graph); written when merging
    float *nbr_e;              // [units][K_src][m] their cosines
    int has_graph;             // apply the decay rounds
    int merge;                 // build the neighbour lists from the per-chunk candidate lists first
    const Cand *cand;          // [units][K_src][cand_chunks][kCandCap]
    const uint32_t *cand_hist; // [units][K_src][kCandBins]
    int cand_chunks;
    int do_select;             // pick the budget and gather
    int *idx_out;              // [units][B]
    int elem_bytes;
    const unsigned char *K, *V;
    unsigned char *K_out, *V_out;
    int wait_prior;            // launched with programmatic stream serialization
};

// grid = units * C CTAs in clusters of C; block kThreads.
__global__ void __launch_bounds__(kThreads, 1) finish_kernel(FinishArgs a)
{
    extern __shared__ __align__(16) uint8_t cs_smem[];
    cg::cluster_group cl = cg::this_cluster();
    const Dims &d = a.d;
    const int C = a.C, rank = C > 1 ? (int)cl.block_rank() : 0;
    const int unit = a.unit0 + blockIdx.x / C;
    const Smem s = carve(cs_smem, 0);
    const int N = d.N, tid = threadIdx.x;
    const int base = rank * a.chunk;
    const int n_local = max(0, min(a.chunk, N - base));
    float *vals = s.vals;
    float *row_s = a.s + (long long)unit * N;
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    load_chunk(row_s, base, 0, n_local, N, vals, 0.f);
    __syncthreads();

    if (a.has_graph && a.merge) {
        // Eq. 3: the four warps of group g of rank r merge sources (g + kMergeWarps * t) * C + r
        const int warp = tid >> 5, grp = warp >> 2, wg = warp & 3;
        Cand *surv = reinterpret_cast<Cand *>(s.st_idx) + grp * kSurvCap;
        int *ns_sh = reinterpret_cast<int *>(s.misc) + 8 + grp;
        for (int src = grp * C + rank; src < d.K_src; src += kMergeWarps * C) {
            const long long slot = ((long long)unit * d.K_src + src) * a.cand_chunks;
            merge_neighbours(a.cand + slot * kCandCap,
                             a.cand_hist + ((long long)unit * d.K_src + src) * kCandBins,
                             a.cand_chunks, d.m, surv, ns_sh, 1 + grp, wg,
                             a.nbr_idx + ((long long)unit * d.K_src + src) * d.m,
                             a.nbr_e + ((long long)unit * d.K_src + src) * d.m);
        }
        __threadfence();
        if (C > 1) cl.sync(); else __syncthreads();
    }

    if (a.has_graph) {
        // Eq. 5 over the fixed graph: source after source (a source's neighbours are distinct, so
        // one source is applied by parallel threads), the T rounds folded into a power.
        const int *ni = a.nbr_idx + (long long)unit * d.K_src * d.m;
        const float *ne = a.nbr_e + (long long)unit * d.K_src * d.m;
        const int per = d.m <= kStage ? kStage / d.m : 0;      // sources staged together
        if (per > 0) {
            for (int src0 = 0; src0 < d.K_src; src0 += per) {
                const int ns = min(per, d.K_src - src0);
                for (int i = tid; i < ns * d.m; i += kThreads) {
                    const float f = 1.0f - d.lambda * fmaxf(__ldcg(ne + src0 * d.m + i), 0.f);
                    float pw = f;
                    for (int t = 1; t < d.T; ++t) pw *= f;
                    s.st_idx[i] = __ldcg(ni + src0 * d.m + i) - base;
                    s.st_f[i] = pw;
                }
                __syncthreads();
                for (int q = 0; q < ns; ++q) {
                    for (int u = tid; u < d.m; u += kThreads) {
                        const int j = s.st_idx[q * d.m + u];
                        if (j >= 0 && j < n_local) vals[j] *= s.st_f[q * d.m + u];
                    }
                    __syncthreads();
                }
            }
        } else {
            for (int src = 0; src < d.K_src; ++src) {
                for (int u = tid; u < d.m; u += kThreads) {
                    const int j = ni[src * d.m + u] - base;
                    if (j >= 0 && j < n_local) {
                        const float f = 1.0f - d.lambda * fmaxf(ne[src * d.m + u], 0.f);
                        float pw = f;
                        for (int t = 1; t < d.T; ++t) pw *= f;
                        vals[j] *= pw;
                    }
                }
                __syncthreads();
            }
        }
        for (int i = tid; i < n_local; i += kThreads) row_s[base + i] = vals[i];
    }

    if (a.do_select) {
        int *idx = a.idx_out + (long long)unit * d.B;
        const Threshold th = cluster_kth(cl, C, rank, s, vals, n_local, (uint32_t)d.B);
        cluster_emit_sorted(cl, C, rank, s, vals, n_local, base, th, idx);
        __threadfence();
        if (C > 1) cl.sync(); else __syncthreads();
        // gather: the cluster's threads share the 16-byte pieces of the B + W output rows
        if (a.K || a.V) {
            const int vec_per_row = kHeadDim * a.elem_bytes / 16;
            const int rows_out = d.B + d.W;
            const long long row_bytes = (long long)kHeadDim * a.elem_bytes;
            const int b = unit / d.hkv, h = unit % d.hkv;
            const long long total = (long long)rows_out * vec_per_row;
            const long long stride = (long long)C * kThreads;
            for (long long p0 = (long long)rank * kThreads + tid; p0 < total; p0 += 4 * stride) {
                uint4 kv[4], vv[4];
                long long dst[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const long long p = p0 + u * stride;
                    dst[u] = -1;
                    if (p < total) {
                        const int c = (int)(p % vec_per_row);
                        const int t = (int)(p / vec_per_row);
                        const int src_row = t < d.B ? __ldcg(idx + t) : N + (t - d.B);
                        dst[u] = ((long long)unit * rows_out + t) * row_bytes + c * 16;
                        if (a.K)
                            kv[u] = *reinterpret_cast<const uint4 *>(
                                a.K + (b * d.ks[0] + h * d.ks[1] + src_row * d.ks[2]) * a.elem_bytes + c * 16);
                        if (a.V)
                            vv[u] = *reinterpret_cast<const uint4 *>(
                                a.V + (b * d.vs[0] + h * d.vs[1] + src_row * d.vs[2]) * a.elem_bytes + c * 16);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (dst[u] >= 0) {
                        if (a.K) *reinterpret_cast<uint4 *>(a.K_out + dst[u]) = kv[u];
                        if (a.V) *reinterpret_cast<uint4 *>(a.V_out + dst[u]) = vv[u];
                    }
                }
            }
        }
    }
    if (C > 1) cl.sync();      // no CTA leaves while its shared memory may still be read
}

}  // namespace cs
}  // namespace graphkv
