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
constexpr int kMaxBudgets = 64;        // batch elements with a budget of their own per launch
constexpr int kFineBins = 8192;        // one-pass selection: histogram over the top 13 bits of the ordered image
constexpr int kFineShift = 19;
constexpr int kTotWords = kFineBins / 2;   // a CTA's slice of the cluster-wide fine histogram (C >= 2)
static_assert(kMergeWarps * kSurvCap * sizeof(Cand) <= 2 * kStage * 4, "survivors reuse the staging area");

// Shared-memory carve-up common to both kernels (dynamic shared memory, 16-byte aligned).
struct Smem {
    uint32_t *hist;       // [kBins] this CTA's digit histogram
    uint32_t *tot;        // [kTotWords] cluster-wide histogram (every CTA holds a copy / its slice)
    uint32_t *fine;       // [kFineBins] this CTA's fine histogram
    uint32_t *wcnt;       // [2 * kWarps] per-warp counts
    uint32_t *misc;       // [32] broadcast words and this CTA's published counts
    int *st_idx;          // [kStage] staging: neighbour positions / candidate positions / survivors
    float *st_f;          // [kStage] staging: decay factors / survivors
    int *nb_j;            // [stage_cap] the unit's neighbour lists, positions (every CTA holds a copy)
    float *nb_f;          // [stage_cap] their decay factors over all rounds
    int stage_cap;        // words of nb_j and of nb_f (at least kStage)
    float *vals;          // [halo + chunk + halo]
};

__host__ __device__ inline size_t smem_bytes(int chunk, int halo, int stage_cap = kStage)
{
    return (size_t)(kBins + kTotWords + kFineBins + 2 * kWarps + 32 + 2 * kStage + 2 * stage_cap) * 4 +
           (size_t)(chunk + 2 * halo + 8) * 4;
}

__device__ __forceinline__ Smem carve(uint8_t *raw, int halo, int stage_cap = kStage)
{
    Smem s;
    s.hist = reinterpret_cast<uint32_t *>(raw);
    s.tot = s.hist + kBins;
    s.fine = s.tot + kTotWords;
    s.wcnt = s.fine + kFineBins;
    s.misc = s.wcnt + 2 * kWarps;
    s.st_idx = reinterpret_cast<int *>(s.misc + 32);
    s.st_f = reinterpret_cast<float *>(s.st_idx + kStage);
    s.nb_j = reinterpret_cast<int *>(s.st_f + kStage);
    s.nb_f = reinterpret_cast<float *>(s.nb_j + stage_cap);
    s.vals = s.nb_f + stage_cap;
    s.stage_cap = stage_cap;
    (void)halo;
    return s;
}

// Result of the radix search: elements whose masked key exceeds `prefix` are kept, and of those
// whose masked key equals it the `remaining` lowest indices.
struct Threshold {
    uint32_t prefix, mask, remaining;
};

// The elements a selection ranks: all n of a chunk in shared memory (list == nullptr), or the n
// of them whose chunk-relative positions `list` holds in ascending order.
// (kListed as a template argument of the loops that walk a view keeps the unlisted case free of
// the indirection.)
struct RowView {
    const float *vals;
    const int *list;
    int n;
    template <bool kListed> __device__ __forceinline__ int pos(int t) const { return kListed ? list[t] : t; }
    template <bool kListed> __device__ __forceinline__ float at(int t) const { return vals[pos<kListed>(t)]; }
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
template <bool kListed>
__device__ Threshold cluster_kth_t(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                   const RowView &row, uint32_t k)
{
    const int n_local = row.n;
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
                const uint32_t u = float_to_key(row.at<kListed>(i));
                valid = (u & th.mask) == th.prefix;
                bin = (u >> shift) & (nb - 1u);
            }
            // the lanes of a warp that share a digit are counted with one addition by the first of
            // them (scores of a row crowd into few digits: additions to one word serialise)
            const unsigned vm = __ballot_sync(0xffffffffu, valid);
            if (valid) {
                const unsigned peers = __match_any_sync(vm, bin);
                if (lane == __ffs(peers) - 1) atomicAdd(&s.hist[bin], (uint32_t)__popc(peers));
            }
        }
        __syncthreads();
        const uint32_t *total = s.hist;
        if (C > 1) {
            cl.sync();                                   // every CTA's histogram is complete
            const int slice = kBins / C;
            if (tid < slice) {
                const int bin = rank * slice + tid;
                // (all peers' counts requested before any is added: one round trip, not C)
                uint32_t part[kMaxCluster];
#pragma unroll
                for (int p = 0; p < kMaxCluster; ++p) part[p] = p < C ? cl.map_shared_rank(s.hist, p)[bin] : 0u;
                uint32_t sum = 0;
#pragma unroll
                for (int p = 0; p < kMaxCluster; ++p) sum += part[p];
#pragma unroll
                for (int p = 0; p < kMaxCluster; ++p)
                    if (p < C) cl.map_shared_rank(s.tot, p)[bin] = sum;
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

__device__ __forceinline__ Threshold cluster_kth(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                                 const RowView &row, uint32_t k)
{
    return row.list ? cluster_kth_t<true>(cl, C, rank, s, row, k) : cluster_kth_t<false>(cl, C, rank, s, row, k);
}

// Candidates for the k largest of a chunk in shared memory.  The chunk's elements fall into
// groups (a thread's strided elements, cut into runs); the k-th largest of the groups' maxima
// bounds the k-th largest element from below, because distinct groups hold distinct elements.
// The bound is taken as the lower edge of the fine-histogram bin of that maximum; the elements
// that reach it (about twice k when a group holds n / 2k elements) are listed by ascending
// position in `list`.  Returns their number, or -1 when grouping cannot help (k above a quarter
// of the chunk) or the list would outgrow `cap`; the caller then ranks the whole chunk.
// Any chunk's bound also holds for a longer row the chunk is part of.
__device__ int filter_candidates(const Smem &s, const float *vals, int n_local, uint32_t k,
                                 int *list, int cap)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = ceil_div(n_local, kThreads);                       // strided elements per thread
    const int gpt = min(per, ceil_div(2 * (int)k, kThreads));          // groups per thread
    const int g = gpt > 0 ? ceil_div(per, gpt) : 0;                    // elements per group
    if (g < 2 || k > (uint32_t)n_local) return -1;
    for (int i = tid; i < kFineBins; i += kThreads) s.fine[i] = 0u;
    __syncthreads();
    for (int q0 = 0; q0 < per; q0 += g) {
        float best = -INFINITY;
        bool any = false;
        for (int q = q0; q < min(q0 + g, per); ++q) {
            const int i = q * kThreads + tid;
            if (i < n_local) {
                best = fmaxf(best, vals[i]);
                any = true;
            }
        }
        if (any) atomicAdd(&s.fine[float_to_key(best) >> kFineShift], 1u);
    }
    __syncthreads();
    // the bin of the k-th largest maximum: thread t owns bins kFineBins-1-8t-q, q < 8
    uint32_t c[8], sum = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        c[q] = s.fine[kFineBins - 1 - (tid * 8 + q)];
        sum += c[q];
    }
    uint32_t incl = warp_incl_scan(sum, lane);
    if (lane == 31) s.wcnt[warp] = incl;
    if (tid == 0) s.misc[23] = 0u;              // bin 0 (everything passes) with fewer than k groups
    __syncthreads();
    if (warp == 0) s.wcnt[lane] = warp_incl_scan(s.wcnt[lane], lane);
    __syncthreads();
    incl += warp == 0 ? 0u : s.wcnt[warp - 1];
    uint32_t run = incl - sum;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        if (run < k && run + c[q] >= k) s.misc[23] = (uint32_t)(kFineBins - 1 - (tid * 8 + q));
        run += c[q];
    }
    __syncthreads();
    const uint32_t bound = s.misc[23] << kFineShift;
    // ordered listing: warp w owns the contiguous segment [w * seg, (w + 1) * seg)
    const int seg = ((n_local + kWarps - 1) / kWarps + 31) & ~31;
    const int lo = min(warp * seg, n_local), hi = min(lo + seg, n_local);
    uint32_t cnt = 0;
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        cnt += __popc(__ballot_sync(0xffffffffu, i < hi && float_to_key(vals[i]) >= bound));
    }
    if (lane == 0) s.wcnt[kWarps + warp] = cnt;
    __syncthreads();
    if (warp == 0) {
        const uint32_t v = s.wcnt[kWarps + lane], vi = warp_incl_scan(v, lane);
        s.wcnt[kWarps + lane] = vi - v;
        if (lane == 31) s.misc[23] = vi;
    }
    __syncthreads();
    const int total = (int)s.misc[23];
    if (total > cap) return -1;
    uint32_t off = s.wcnt[kWarps + warp];
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        const bool keep = i < hi && float_to_key(vals[i]) >= bound;
        const unsigned bm = __ballot_sync(0xffffffffu, keep);
        if (keep) list[off + __popc(bm & ((1u << lane) - 1u))] = i;
        off += __popc(bm);
    }
    __syncthreads();
    return total;
}

// k-th largest of the cluster's row in one histogram pass: a kFineBins histogram over the top 13
// bits of the ordered image (sign, exponent, four mantissa bits: sixteen bins per octave), reduced
// across the cluster in slices; the bin b* that holds the k-th largest is located by every CTA
// alike; the elements above it are kept, and the few inside it are pulled by every CTA and
// ranked by counting (value descending, position ascending), which gives the exact threshold
// value and the number of its ties to keep.  Falls back to the three-digit search when b* holds
// more than a few hundred elements (large budgets, rows with massive ties).  Same contract as cluster_kth.
template <bool kListed>
__device__ Threshold cluster_kth_fine_t(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                        const RowView &row, int base, uint32_t k, PhaseClock &pc)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_local = row.n;
    for (int i = tid; i < kFineBins; i += kThreads) s.fine[i] = 0u;
    if (tid == 0) s.misc[17] = 0u;                     // this CTA's candidate counter
    __syncthreads();
    for (int i0 = 0; i0 < n_local; i0 += kThreads) {
        const int i = i0 + tid;
        const bool valid = i < n_local;
        const uint32_t bin = valid ? float_to_key(row.at<kListed>(i)) >> kFineShift : 0u;
        // the lanes of a warp that share a bin are counted with one addition by the first of them
        const unsigned vm = __ballot_sync(0xffffffffu, valid);
        if (valid) {
            const unsigned peers = __match_any_sync(vm, bin);
            if (lane == __ffs(peers) - 1) atomicAdd(&s.fine[bin], (uint32_t)__popc(peers));
        }
    }
    __syncthreads();
    pc.mark();
    // cluster-wide counts of this CTA's slice of the bins, and the slice's total
    const int slice = kFineBins / C;
    uint32_t mine = 0;
    if (C > 1) {
        cl.sync();                                       // every CTA's histogram is complete
        for (int b = tid; b < slice; b += kThreads) {
            uint32_t part[kMaxCluster];
#pragma unroll
            for (int p = 0; p < kMaxCluster; ++p)
                part[p] = p < C ? cl.map_shared_rank(s.fine, p)[rank * slice + b] : 0u;
            uint32_t sum = 0;
#pragma unroll
            for (int p = 0; p < kMaxCluster; ++p) sum += part[p];
            s.tot[b] = sum;
            mine += sum;
        }
    } else {
        for (int b = tid; b < slice; b += kThreads) mine += s.fine[b];
    }
    mine = __reduce_add_sync(0xffffffffu, mine);
    if (lane == 0) s.wcnt[warp] = mine;
    __syncthreads();
    if (warp == 0) {
        const uint32_t t = __reduce_add_sync(0xffffffffu, s.wcnt[lane]);
        if (lane == 0) s.misc[16] = t;
    }
    __syncthreads();
    pc.mark();
    if (C > 1) cl.sync();                                // slices and their totals are complete
    pc.mark();
    // the slice that holds the k-th largest (rank C-1 has the highest bins)
    uint32_t s_lane = 0;
    if (lane < C) s_lane = C > 1 ? cl.map_shared_rank(s.misc, lane)[16] : s.misc[16];
    uint32_t above = 0;
    int rstar = 0;
    for (int p = C - 1; p >= 0; --p) {
        const uint32_t sp = __shfl_sync(0xffffffffu, s_lane, p);
        if (above + sp >= k) { rstar = p; break; }
        above += sp;
    }
    // walk that slice from its top bin: thread t owns bins slice-1-t*per-q, q < per
    const uint32_t *tt = C > 1 ? cl.map_shared_rank(s.tot, rstar) : s.fine;
    const int per = slice / kThreads;                    // 1, 2, 4 or 8
    uint32_t c[8], sum = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        c[q] = q < per ? tt[slice - 1 - (tid * per + q)] : 0u;
        sum += c[q];
    }
    uint32_t incl = warp_incl_scan(sum, lane);
    if (lane == 31) s.wcnt[kWarps + warp] = incl;
    __syncthreads();
    if (warp == 0) s.wcnt[kWarps + lane] = warp_incl_scan(s.wcnt[kWarps + lane], lane);
    __syncthreads();
    incl += warp == 0 ? 0u : s.wcnt[kWarps + warp - 1];
    uint32_t run = above + incl - sum;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        if (q < per && run < k && run + c[q] >= k) {
            s.misc[20] = (uint32_t)(rstar * slice + slice - 1 - (tid * per + q));
            s.misc[21] = run;
            s.misc[22] = c[q];
        }
        run += c[q];
    }
    __syncthreads();
    pc.mark();
    const uint32_t bstar = s.misc[20], n_above = s.misc[21], n_in = s.misc[22];
    const uint32_t need = k - n_above;                   // of the n_in elements in bin b*
    if (need == n_in) return Threshold{bstar << kFineShift, (uint32_t)(kFineBins - 1) << kFineShift, n_in};
    if (n_in > (uint32_t)kThreads / 4) return cluster_kth_t<kListed>(cl, C, rank, s, row, k);   // too many to rank by counting
    // this CTA's elements of bin b* -> its own lists (keys and positions in the two halves of hist):
    // every warp counts its own first, a scan over the warps gives each its slots
    uint32_t *ck = s.hist;
    int *ci = reinterpret_cast<int *>(s.hist + kThreads);
    uint32_t mine_n = 0;
    for (int i0 = 0; i0 < n_local; i0 += kThreads) {
        const int i = i0 + tid;
        const bool cand = i < n_local && (float_to_key(row.at<kListed>(i)) >> kFineShift) == bstar;
        mine_n += __popc(__ballot_sync(0xffffffffu, cand));
    }
    if (lane == 0) s.wcnt[warp] = mine_n;
    __syncthreads();
    if (warp == 0) {
        const uint32_t v = s.wcnt[lane], vi = warp_incl_scan(v, lane);
        s.wcnt[lane] = vi - v;
        if (lane == 31) s.misc[17] = vi;
    }
    __syncthreads();
    uint32_t slot0 = s.wcnt[warp];
    for (int i0 = 0; i0 < n_local; i0 += kThreads) {
        const int i = i0 + tid;
        uint32_t key = 0;
        bool cand = false;
        int at = 0;
        if (i < n_local) {
            at = row.pos<kListed>(i);
            key = float_to_key(row.vals[at]);
            cand = (key >> kFineShift) == bstar;
        }
        const unsigned bm = __ballot_sync(0xffffffffu, cand);
        if (cand) {
            const uint32_t slot = slot0 + __popc(bm & ((1u << lane) - 1u));
            ck[slot] = key;
            ci[slot] = base + at;
        }
        slot0 += __popc(bm);
    }
    __syncthreads();
    pc.mark();
    if (C > 1) cl.sync();                                // every CTA's list is complete
    pc.mark();
    // every CTA pulls all lists (into the two halves of `tot`, idle by now) and ranks them itself:
    // the same answer everywhere without another exchange
    uint32_t *ak = s.tot;
    int *ai = reinterpret_cast<int *>(s.tot + kThreads);
    {
        uint32_t n_lane = 0;
        if (lane < C) n_lane = C > 1 ? cl.map_shared_rank(s.misc, lane)[17] : s.misc[17];
        uint32_t total = 0;
        int mine_p = -1, mine_j = 0;
        for (int p = 0; p < C; ++p) {
            const uint32_t n_p = __shfl_sync(0xffffffffu, n_lane, p);
            if (tid >= (int)total && tid < (int)(total + n_p)) {
                mine_p = p;
                mine_j = tid - (int)total;
            }
            total += n_p;
        }
        if (mine_p >= 0) {
            ak[tid] = (C > 1 ? cl.map_shared_rank(ck, mine_p) : ck)[mine_j];
            ai[tid] = (C > 1 ? cl.map_shared_rank(ci, mine_p) : ci)[mine_j];
        }
        __syncthreads();
        {
            // few candidates (at most kThreads / 4): four threads each, every one walking a quarter of the list
            const int t = tid >> 2, sub = tid & 3;
            const bool live = t < (int)total;
            const uint32_t kt = live ? ak[t] : 0u;
            const int pt = live ? ai[t] : 0;
            uint32_t r = 0, n_gt = 0;                    // rank among all; candidates with a larger value
            if (live) {
#pragma unroll 4
                for (int u = sub; u < (int)total; u += 4) {
                    const uint32_t ku = ak[u];
                    const int pu = ai[u];
                    n_gt += ku > kt;
                    r += (ku > kt) | ((ku == kt) & (pu < pt));
                }
            }
            r += __shfl_xor_sync(0xffffffffu, r, 1);
            r += __shfl_xor_sync(0xffffffffu, r, 2);
            n_gt += __shfl_xor_sync(0xffffffffu, n_gt, 1);
            n_gt += __shfl_xor_sync(0xffffffffu, n_gt, 2);
            if (live && sub == 0 && r == need - 1) {
                s.misc[18] = kt;
                s.misc[19] = need - n_gt;
            }
        }
        __syncthreads();
    }
    pc.mark();
    return Threshold{s.misc[18], 0xffffffffu, s.misc[19]};
}

__device__ __forceinline__ Threshold cluster_kth_fine(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                                      const RowView &row, int base, uint32_t k, PhaseClock &pc)
{
    return row.list ? cluster_kth_fine_t<true>(cl, C, rank, s, row, base, k, pc)
                    : cluster_kth_fine_t<false>(cl, C, rank, s, row, base, k, pc);
}

// Ascending positions of the kept elements of the cluster's row -> out[0..k).  Returns nothing;
// ends with the writes of this CTA issued (callers fence before another CTA reads them).
// One cluster barrier.  `mirror` (optional): every kept position also goes into that array in the
// shared memory of each of the cluster's `n_mirror` CTAs, complete after the cluster's next barrier.
template <bool kListed>
__device__ void cluster_emit_sorted_t(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                      const RowView &row, int base, Threshold th, int *out,
                                      int *mirror = nullptr, int n_mirror = 1)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_local = row.n;
    // warp w owns the contiguous segment [w * seg, (w + 1) * seg) of the chunk
    const int seg = ((n_local + kWarps - 1) / kWarps + 31) & ~31;
    const int lo = min(warp * seg, n_local), hi = min(lo + seg, n_local);
    uint32_t gt = 0, eq = 0;
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        uint32_t mk = 0;
        const bool in = i < hi;
        if (in) mk = float_to_key(row.at<kListed>(i)) & th.mask;
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
        // lane p reads rank p's totals, so the remote reads overlap
        uint32_t g = 0, e = 0;
        if (lane < rank) {
            const uint32_t *pm = cl.map_shared_rank(s.misc, lane);
            g = pm[4];
            e = pm[5];
        }
        gt_before += __reduce_add_sync(0xffffffffu, g);
        eq_before += __reduce_add_sync(0xffffffffu, e);
    }
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        uint32_t mk = 0;
        const bool in = i < hi;
        int at = 0;
        if (in) {
            at = row.pos<kListed>(i);
            mk = float_to_key(row.vals[at]) & th.mask;
        }
        const bool is_gt = in && mk > th.prefix, is_eq = in && mk == th.prefix;
        const unsigned bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
        const unsigned below = (1u << lane) - 1u;
        const uint32_t gi = gt_before + __popc(bg & below), e = eq_before + __popc(be & below);
        const bool keep = is_gt || (is_eq && e < th.remaining);
        const int t = (int)(gi + min(e, th.remaining));
        if (keep) {
            out[t] = base + at;
            if (mirror) {
                if (n_mirror > 1)
                    for (int p = 0; p < n_mirror; ++p) cl.map_shared_rank(mirror, p)[t] = base + at;
                else
                    mirror[t] = base + at;
            }
        }
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
}

__device__ __forceinline__ void cluster_emit_sorted(cg::cluster_group &cl, int C, int rank, const Smem &s,
                                                    const RowView &row, int base, Threshold th, int *out,
                                                    int *mirror = nullptr, int n_mirror = 1)
{
    if (row.list) cluster_emit_sorted_t<true>(cl, C, rank, s, row, base, th, out, mirror, n_mirror);
    else cluster_emit_sorted_t<false>(cl, C, rank, s, row, base, th, out, mirror, n_mirror);
}

// The m largest edges (cosine descending, position ascending) of the lists when too many tie at
// the bound: the exact m-th largest 64-bit edge key (keys are distinct: distinct positions) by a
// byte-wise radix search over the lists themselves, eight rounds of a 256-bin histogram of the byte
// among the keys that share the bytes found so far.  The four warps of a merging group (`wg` of
// them, barrier `bar_id`); `rh`: 264 words of shared memory of the group; the number of survivors
// written (m, or fewer when fewer edges are listed) is left in *ns_sh.
__device__ void merge_exact(const Cand *cand, int slots, int m, Cand *surv, uint32_t *rh, int *ns_sh,
                            int bar_id, int wg)
{
    const int lane = threadIdx.x & 31, t = wg * 32 + lane;
    unsigned long long t64 = 0ull;
    uint32_t remaining = (uint32_t)m;
    for (int byte = 7; byte >= 0; --byte) {
        const unsigned long long hi_mask = byte == 7 ? 0ull : ~0ull << (8 * (byte + 1));
        rh[t] = 0u;
        rh[t + 128] = 0u;
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        for (int i0 = 0; i0 < slots; i0 += 128) {
            const int i = i0 + t;
            bool valid = false;
            uint32_t bin = 0;
            if (i < slots) {
                const unsigned long long raw = __ldcg(reinterpret_cast<const unsigned long long *>(cand + i));
                const float e = __uint_as_float(static_cast<uint32_t>(raw));
                const unsigned long long key = edge_key(e, static_cast<int>(raw >> 32));
                valid = e >= -1.0f && (key & hi_mask) == t64;
                bin = (uint32_t)(key >> (8 * byte)) & 0xffu;
            }
            // tied cosines share their digits: one addition for the lanes with the first valid lane's
            const unsigned vm = __ballot_sync(0xffffffffu, valid);
            if (vm) {
                const int leader = __ffs(vm) - 1;
                const uint32_t lbin = __shfl_sync(0xffffffffu, bin, leader);
                const bool same = valid && bin == lbin;
                const unsigned sm = __ballot_sync(0xffffffffu, same);
                if (lane == leader) atomicAdd(&rh[lbin], (uint32_t)__popc(sm));
                else if (valid && !same) atomicAdd(&rh[bin], 1u);
            }
        }
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        if (wg == 0) {
            // lane l holds digits 255 - 8 l - q (q < 8)
            uint32_t c8[8], sum = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                c8[q] = rh[255 - 8 * lane - q];
                sum += c8[q];
            }
            const uint32_t incl = warp_incl_scan(sum, lane);
            const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
            uint32_t run = incl - sum;
            if (lane == 0) {
                rh[256] = 0u;                               // fewer edges than m: all are kept
                rh[257] = remaining;
            }
            __syncwarp();
            if (total >= remaining) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (run < remaining && run + c8[q] >= remaining) {
                        rh[256] = (uint32_t)(255 - 8 * lane - q);
                        rh[257] = remaining - run;
                    }
                    run += c8[q];
                }
            }
        }
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        t64 |= (unsigned long long)rh[256] << (8 * byte);
        remaining = rh[257];
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    }
    if (t == 0) *ns_sh = 0;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    for (int i0 = 0; i0 < slots; i0 += 128) {
        const int i = i0 + t;
        bool keep = false;
        Cand cd{0.f, 0};
        if (i < slots) {
            const unsigned long long raw = __ldcg(reinterpret_cast<const unsigned long long *>(cand + i));
            cd.e = __uint_as_float(static_cast<uint32_t>(raw));
            cd.j = static_cast<int>(raw >> 32);
            keep = cd.e >= -1.0f && edge_key(cd.e, cd.j) >= t64;
        }
        const unsigned bm = __ballot_sync(0xffffffffu, keep);
        if (bm) {
            int basep = 0;
            if (lane == 0) basep = atomicAdd(ns_sh, __popc(bm));
            basep = __shfl_sync(0xffffffffu, basep, 0);
            const int pos = basep + __popc(bm & ((1u << lane) - 1u));
            if (keep && pos < kSurvCap) surv[pos] = cd;
        }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    if (t == 0) *ns_sh = min(*ns_sh, kSurvCap);
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
}

// Eq. 3 for one source: the m largest edges (cosine descending, position ascending) among the
// candidate lists its key chunks wrote.  One warp; `surv` holds kSurvCap entries of shared memory.
// The lists together hold every member of the top-m, and `hist` counts the listed edges per cosine
// bin: the highest bin b with at least m listed edges in bins >= b bounds the m-th largest from
// below, so only edges with e >= b / kCandBins need ranking.
// The final list also goes, as (position, decay factor over all rounds), into slots
// [slot0, slot0 + m) of the nb_j / nb_f arrays of the CTAs of the cluster that hold the row (slots past the listed
// edges get position -1).
struct PushLists {
    int C;          // cluster size
    int R;          // ranks 0 .. R-1 receive the lists
    int *nb_j;
    float *nb_f;
    int slot0;
    float lambda;
    int T;
    int signal;
};

__device__ void merge_neighbours(cg::cluster_group &cl, const Cand *cand, const uint32_t *hist,
                                 int chunks, int m, Cand *surv, int *ns_sh, int bar_id, int wg,
                                 int *nbr_idx, float *nbr_e, const PushLists &push, uint32_t *rh)
{
    const int lane = threadIdx.x & 31;
    constexpr int kPer = kCandBins / 32;
    // lane l holds bins [l * kPer, (l + 1) * kPer); walk down from the top bin
    // the histogram and the group's first block of 256 slots per warp are requested together: one
    // round trip to memory instead of two
    const int slots = chunks * kCandCap;
    uint32_t h[kPer], mine = 0;
    unsigned long long raw[8];
#pragma unroll
    for (int q = 0; q < kPer; ++q) h[q] = __ldcg(hist + lane * kPer + q);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int i = wg * 256 + q * 32 + lane;
        raw[q] = i < slots ? __ldcg(reinterpret_cast<const unsigned long long *>(cand + i)) : 0ull;
    }
#pragma unroll
    for (int q = 0; q < kPer; ++q) mine += h[q];
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

    // the four warps of the group take interleaved blocks of 256 slots; a warp reserves the places
    // of a block's survivors with one addition
    if (wg == 0 && lane == 0) *ns_sh = 0;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    for (int i0 = wg * 256; i0 < slots; i0 += 4 * 256) {
        if (i0 != wg * 256) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int i = i0 + q * 32 + lane;
                raw[q] = i < slots ? __ldcg(reinterpret_cast<const unsigned long long *>(cand + i)) : 0ull;
            }
        }
        unsigned bm[8];
        int total = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + q * 32 + lane;
            const float e = __uint_as_float(static_cast<uint32_t>(raw[q]));
            bm[q] = __ballot_sync(0xffffffffu, i < slots && e >= bound);
            total += __popc(bm[q]);
        }
        if (total == 0) continue;
        int basep = 0;
        if (lane == 0) basep = atomicAdd(ns_sh, total);
        basep = __shfl_sync(0xffffffffu, basep, 0);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int pos = basep + __popc(bm[q] & ((1u << lane) - 1u));
            if (((bm[q] >> lane) & 1u) && pos < kSurvCap)
                surv[pos] = Cand{__uint_as_float(static_cast<uint32_t>(raw[q])), static_cast<int>(raw[q] >> 32)};
            basep += __popc(bm[q]);
        }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    int ns = *ns_sh;
    if (ns > kSurvCap) {
        merge_exact(cand, slots, m, surv, rh, ns_sh, bar_id, wg);
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
            const float pw = signal_factor(me.e, push.lambda, push.T, push.signal);
            for (int p = 0; p < push.R; ++p) {
                (push.C > 1 ? cl.map_shared_rank(push.nb_j, p) : push.nb_j)[push.slot0 + rank] = me.j;
                (push.C > 1 ? cl.map_shared_rank(push.nb_f, p) : push.nb_f)[push.slot0 + rank] = pw;
            }
        }
    }
    for (int u = ns + wg * 32 + lane; u < m; u += 128)
        for (int p = 0; p < push.R; ++p)
            (push.C > 1 ? cl.map_shared_rank(push.nb_j, p) : push.nb_j)[push.slot0 + u] = -1;
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
    PhaseClock pc(threadIdx.x == 0 && rank == 0);
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    pc.mark();
    if (a.zero)
        for (int i = rank * kThreads + tid; i < a.zero_words; i += C * kThreads)
            a.zero[(long long)unit * a.zero_words + i] = 0u;
    // this thread's two counts of the mass histogram, on their way while the row is pooled
    // (the bound from the mass histogram needs pooling that only raises values: max pooling)
    const bool bounded = a.mass_hist && a.k > 0 && a.k <= kThreads && !a.d.pool_avg;
    uint32_t hc0 = 0, hc1 = 0;
    if (bounded) {
        const uint32_t *mh = a.mass_hist + (long long)unit * kBins;
        hc0 = __ldcg(mh + kBins - 1 - 2 * tid);
        hc1 = __ldcg(mh + kBins - 2 - 2 * tid);
    }
    if (a.a) {
        const float *row_a = a.a + (long long)unit * N;
        const int half = a.halo;
        const bool avg = a.d.pool_avg != 0;
        if (n_local > 0) load_chunk(row_a, base, -half, n_local + half, N, vals, avg ? 0.f : -INFINITY);
        __syncthreads();
        float pooled[kPer];
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int i = q * kThreads + tid;
            if (i < n_local) {
                float best = vals[i - half];
                if (avg) {
                    // ascending positions, zeros outside the row, divided by the kernel size
                    for (int t = 1 - half; t <= half; ++t) best += vals[i + t];
                    best /= (float)(2 * half + 1);
                } else {
                    for (int t = 1 - half; t <= half; ++t) best = fmaxf(best, vals[i + t]);
                }
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
    pc.mark();
    if (a.k > 0) {
        int *out = a.src_out + (long long)unit * a.k;
        const bool done = bounded && cluster_topk_bounded(cl, C, rank, s, vals, n_local, base, a.k, hc0, hc1, out);
        if (!done) {
            const RowView row{vals, nullptr, n_local};
            const Threshold th = cluster_kth(cl, C, rank, s, row, (uint32_t)a.k);
            cluster_emit_sorted(cl, C, rank, s, row, base, th, out);
        }
    }
    pc.mark();
    if (C > 1) cl.sync();      // no CTA leaves while its shared memory may still be read
    pc.mark();
    pc.flush(3);
}

struct FinishArgs {
    Dims d;
    int C;                     // CTAs per cluster (one cluster per unit)
    int R;                     // ranks 0 .. R-1 hold a chunk of the row each: 1 (the others only
                               // merge neighbour lists and gather) or C
    int chunk, halo;
    int unit0;
    const float *a;            // optional [units][N]: attention mass to pool into the scores first
    float *s;                  // [units][N] scores: read unless pooling; written when pooling or decaying
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
    int stage_cap;             // words of each staging array in shared memory (K_src * m when it fits)
    int keep_scores;           // write the pooled / decayed scores back to `s` (0: nobody reads them)
    int per_batch_budget;      // budgets differ per batch element: budget_of[unit / hkv] (d.B: output rows)
    int budget_of[kMaxBudgets];
};

// Chunk [base, base + n_local) of a unit's scores into shared memory; returns `vals` with
// vals[i] = score of element base + i.  With `row_a` the scores are the attention mass max-pooled
// over [j - half, j + half] (positions outside the row ignored): the raw values are staged first
// and the pooled value of element i replaces a slot at or below raw slot i, in rounds whose
// inputs are all read before any is overwritten (element i reads raw slots i .. i + 2 half, so a
// later round never needs what an earlier one has replaced).  Global reads are 16-byte loads; the
// staging offset inside `buf` (16-byte aligned, chunk + 2 half + 8 words) is chosen so that the
// returned values sit at the same offset modulo 16 bytes as the elements of the global row.
// Ends with the CTA synchronised.
__device__ float *load_pool_chunk(const float *row_a, const float *row_s, int base, int n_local,
                                  int N, int half, float *buf)
{
    const int tid = threadIdx.x;
    const float *row = row_a ? row_a : row_s;
    const int h = row_a ? half : 0;
    const int j0 = base - h, j1 = base + n_local + h;          // staged span, row positions
    const int lo = max(j0, 0), hi = min(j1, N);
    const int e2 = (4 - (h & 3)) & 3;                          // pooled element i goes to slot i - e2
    const int gcls = (int)((reinterpret_cast<uintptr_t>(row + lo) >> 2) & 3);
    int pad = (gcls - (lo - j0)) & 3;
    while (pad < e2) pad += 4;
    float *dst = buf + pad;                                    // dst[j - j0] = row[j]
    if (n_local > 0) {
        for (int j = j0 + tid; j < lo; j += kThreads) dst[j - j0] = -INFINITY;
        for (int j = max(hi, j0) + tid; j < j1; j += kThreads) dst[j - j0] = -INFINITY;
        const int head = min(hi - lo, (4 - gcls) & 3);
        if (tid < head) dst[lo + tid - j0] = __ldcg(row + lo + tid);
        const int v0 = lo + head, nv = (hi - v0) >> 2;
        const float4 *rv = reinterpret_cast<const float4 *>(row + v0);
        float4 *dv = reinterpret_cast<float4 *>(dst + (v0 - j0));
        for (int i0 = tid; i0 < nv; i0 += 8 * kThreads) {
            float4 r[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (i0 + k * kThreads < nv) r[k] = __ldcg(rv + i0 + k * kThreads);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (i0 + k * kThreads < nv) dv[i0 + k * kThreads] = r[k];
        }
        const int t0 = v0 + 4 * nv;
        if (tid < hi - t0) dst[t0 + tid - j0] = __ldcg(row + t0 + tid);
    }
    __syncthreads();
    if (h == 0) return dst;
    for (int r0 = 0; r0 < n_local; r0 += 8 * kThreads) {
        float pooled[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = r0 + q * kThreads + tid;
            pooled[q] = 0.f;
            if (i < n_local) {
                float best = dst[i];
                for (int t = 1; t <= 2 * h; ++t) best = fmaxf(best, dst[i + t]);
                pooled[q] = best;
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = r0 + q * kThreads + tid;
            if (i < n_local) dst[i - e2] = pooled[q];
        }
        __syncthreads();
    }
    return dst - e2;
}

// row[i] = vals[i] for i < n: 16-byte stores where the two sides share their offset modulo 16 bytes.
__device__ void store_chunk(float *row, const float *vals, int n)
{
    const int tid = threadIdx.x;
    const uintptr_t g = reinterpret_cast<uintptr_t>(row), sm = reinterpret_cast<uintptr_t>(vals);
    if (((g ^ sm) & 15) != 0) {
        for (int i = tid; i < n; i += kThreads) row[i] = vals[i];
        return;
    }
    const int head = min(n, (int)((4 - ((g >> 2) & 3)) & 3));
    if (tid < head) row[tid] = vals[tid];
    const int nv = (n - head) >> 2;
    float4 *rv = reinterpret_cast<float4 *>(row + head);
    const float4 *sv = reinterpret_cast<const float4 *>(vals + head);
    for (int i = tid; i < nv; i += kThreads) rv[i] = sv[i];
    const int t0 = head + 4 * nv;
    if (tid < n - t0) row[t0 + tid] = vals[t0 + tid];
}

// Eq. 5 on the chunk in shared memory: the unit's lists are in s.nb_j / s.nb_f as (position,
// factor over all rounds); with the evicted signal every listed position becomes -inf instead.  A position that only one listed edge points to (counted per slot of a
// small table, so a slot shared with another position counts as contested) takes its factor at
// once; the contested ones are applied by one warp, source after source (a source's neighbours are
// distinct), so that overlapping neighbourhoods multiply in a fixed order.  Uses s.fine as
// scratch.  Ends with the CTA synchronised.
__device__ void apply_lists(const Smem &s, float *vals, int base, int n_local, int K_src, int m,
                            bool evict)
{
    const int tid = threadIdx.x;
    const int pairs = K_src * m;                           // fits the staging arrays
    if (pairs > kStage) {
        // hundreds of sources, whose neighbourhoods overlap heavily (counting the edges per position
        // would serialise on the few positions they share): every warp walks the whole list, 32
        // entries at a time, and applies the entries of the positions it owns (a position belongs to
        // one warp, so its factors are applied in list order, whatever the other warps do)
        const int warp = tid >> 5, lane = tid & 31;
        for (int i0 = 0; i0 < pairs; i0 += 32) {
            const int i = i0 + lane;
            int j = -1;
            float f = 1.f;
            if (i < pairs) {
                j = s.nb_j[i] - base;
                f = s.nb_f[i];
            }
            const bool own = j >= 0 && j < n_local && ((j >> 2) & 31) == warp;
            const unsigned ob = __ballot_sync(0xffffffffu, own);
            if (ob == 0) continue;
            if ((ob & (ob - 1)) == 0) {                       // one entry: no order to keep
                if (own) vals[j] = evict ? -INFINITY : vals[j] * f;
                continue;
            }
            if (own) {
                // lanes that hold the same position take turns, lowest lane first
                const unsigned peers = __match_any_sync(ob, j);
                unsigned todo = peers;
                while (todo) {
                    if (__ffs(todo) - 1 == lane) vals[j] = evict ? -INFINITY : vals[j] * f;
                    todo &= todo - 1;
                    __syncwarp(peers);
                }
            }
        }
        __syncthreads();
        return;
    }
    uint32_t *cnt = s.fine;                                // [4096] edges per table slot
    uint32_t *src_mask = s.fine + 4096;                    // [K_src / 32] sources with a contested edge
    for (int i = tid; i < 4096 + (K_src + 31) / 32; i += kThreads) cnt[i] = 0u;
    __syncthreads();
    for (int p = tid; p < pairs; p += kThreads) {
        const int j = s.nb_j[p] - base;
        if (j >= 0 && j < n_local) atomicAdd(&cnt[j & 4095], 1u);
    }
    __syncthreads();
    for (int p = tid; p < pairs; p += kThreads) {
        const int j = s.nb_j[p] - base;
        if (j >= 0 && j < n_local) {
            if (evict) {
                vals[j] = -INFINITY;                       // the evicted signal: no order to keep
            } else if (cnt[j & 4095] == 1u) {
                vals[j] *= s.nb_f[p];
            } else {
                const int q = p / m;
                atomicOr(&src_mask[q >> 5], 1u << (q & 31));
            }
        }
    }
    __syncthreads();
    if (tid < 32) {
        for (int w = 0; w * 32 < K_src; ++w) {
            uint32_t mask = src_mask[w];
            while (mask) {
                const int q = w * 32 + __ffs(mask) - 1;
                mask &= mask - 1;
                for (int u = tid; u < m; u += 32) {
                    const int j = s.nb_j[q * m + u] - base;
                    if (j >= 0 && j < n_local && cnt[j & 4095] != 1u) vals[j] *= s.nb_f[q * m + u];
                }
                __syncwarp();
            }
        }
    }
    __syncthreads();
}

// grid = units * C CTAs in clusters of C; block kThreads.
__global__ void __launch_bounds__(kThreads, 1) finish_kernel(FinishArgs a)
{
    extern __shared__ __align__(16) uint8_t cs_smem[];
    cg::cluster_group cl = cg::this_cluster();
    const Dims &d = a.d;
    const int C = a.C, R = a.R, rank = C > 1 ? (int)cl.block_rank() : 0;
    const int unit = a.unit0 + blockIdx.x / C;
    const Smem s = carve(cs_smem, 0, a.stage_cap);
    const int N = d.N, tid = threadIdx.x;
    const bool holds = rank < R;                           // this CTA keeps a chunk of the row
    const int base = rank * a.chunk;
    const int n_local = holds ? max(0, min(a.chunk, N - base)) : 0;
    float *vals = s.vals;
    float *row_s = a.s + (long long)unit * N;
    PhaseClock pc(tid == 0);
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    pc.mark();
    const int b = unit / d.hkv, h = unit % d.hkv;
    const long long row_bytes = (long long)d.D * a.elem_bytes;
    const int rows_out = d.B + d.W;                        // rows the outputs hold per unit
    const int B = a.per_batch_budget ? a.budget_of[b] : d.B;   // this unit's budget
    const int vpr = (int)(row_bytes >> 4);                 // 16-byte pieces per row
    const unsigned char *k0 = a.K ? a.K + (b * d.ks[0] + h * d.ks[1]) * a.elem_bytes : nullptr;
    const unsigned char *v0 = a.V ? a.V + (b * d.vs[0] + h * d.vs[1]) * a.elem_bytes : nullptr;
    unsigned char *k_out = a.K_out ? a.K_out + (long long)unit * rows_out * row_bytes : nullptr;
    unsigned char *v_out = a.V_out ? a.V_out + (long long)unit * rows_out * row_bytes : nullptr;
    const long long k_stride = d.ks[2] * a.elem_bytes, v_stride = d.vs[2] * a.elem_bytes;
    // copies the 16-byte pieces [p0, p1) of output rows [t0, ...): piece p is (row t0 + p / (2 vpr),
    // K or V, column piece); `src_of(t)` gives the input row.  Four pieces in flight per thread.
    auto copy_rows = [&](int t0, long long n_pieces, auto src_of) {
        const long long stride = (long long)C * kThreads;
        for (long long p0 = (long long)rank * kThreads + tid; p0 < n_pieces; p0 += 4 * stride) {
            uint4 v[4];
            unsigned char *dst[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long p = p0 + u * stride;
                dst[u] = nullptr;
                if (p < n_pieces) {
                    const int t = t0 + (int)(p / (2 * vpr)), pp = (int)(p % (2 * vpr));
                    const bool is_v = pp >= vpr;
                    const int c = is_v ? pp - vpr : pp;
                    const unsigned char *in = is_v ? v0 : k0;
                    if (in) {
                        v[u] = *reinterpret_cast<const uint4 *>(in + src_of(t) * (is_v ? v_stride : k_stride) + c * 16);
                        dst[u] = (is_v ? v_out : k_out) + (long long)t * row_bytes + c * 16;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (dst[u]) *reinterpret_cast<uint4 *>(dst[u]) = v[u];
        }
    };
    const bool gathers = a.do_select && (a.K || a.V);
    if (holds)
        vals = load_pool_chunk(a.a ? a.a + (long long)unit * N : nullptr, row_s, base, n_local, N, a.halo, s.vals);
    pc.mark();

    if (a.has_graph) {
        int *ni = a.nbr_idx + (long long)unit * d.K_src * d.m;
        float *ne = a.nbr_e + (long long)unit * d.K_src * d.m;
        const int pairs = d.K_src * d.m;
        const bool staged = pairs <= s.stage_cap;          // the lists fit the shared-memory staging
        // Eq. 3, then Eq. 5 over the fixed graph with the T rounds folded into a power: the
        // CTAs that hold the row get the unit's lists as (position, factor) in shared memory
        if (a.merge) {
            // the four warps of group g of merging rank r take sources (g + kMergeWarps * t) * M + r;
            // a first CTA that holds the whole row leaves the merging to the others
            const int warp = tid >> 5, grp = warp >> 2, wg = warp & 3;
            Cand *surv = reinterpret_cast<Cand *>(s.st_idx) + grp * kSurvCap;
            int *ns_sh = reinterpret_cast<int *>(s.misc) + 8 + grp;
            const bool spare_first = R == 1 && C > 1;
            const int M = spare_first ? C - 1 : C, mr = spare_first ? rank - 1 : rank;
            for (int src = grp * M + mr; mr >= 0 && src < d.K_src; src += kMergeWarps * M) {
                const long long slot = ((long long)unit * d.K_src + src) * a.cand_chunks;
                const PushLists push{C, staged ? R : 0, s.nb_j, s.nb_f, src * d.m, d.lambda, d.T, d.signal};
                merge_neighbours(cl, a.cand + slot * kCandCap,
                                 a.cand_hist + ((long long)unit * d.K_src + src) * kCandBins,
                                 a.cand_chunks, d.m, surv, ns_sh, 1 + grp, wg, ni + src * d.m,
                                 ne + src * d.m, push, s.fine + grp * 264);
            }
            pc.mark();
            if (!staged) __threadfence();                     // the lists are read back from global memory
            if (C > 1) cl.sync(); else __syncthreads();       // every list has arrived
            pc.mark();
        } else if (staged && holds) {
            for (int i = tid; i < pairs; i += kThreads) {
                s.nb_j[i] = __ldcg(ni + i);
                s.nb_f[i] = signal_factor(__ldcg(ne + i), d.lambda, d.T, d.signal);
            }
            __syncthreads();
        }
        if (staged) {
            if (holds) apply_lists(s, vals, base, n_local, d.K_src, d.m, d.signal == GRAPHKV_SIGNAL_EVICT);
        } else if (holds) {
            for (int src = 0; src < d.K_src; ++src) {
                for (int u = tid; u < d.m; u += kThreads) {
                    const int j = __ldcg(ni + src * d.m + u) - base;
                    if (j >= 0 && j < n_local)
                        vals[j] = d.signal == GRAPHKV_SIGNAL_EVICT
                                      ? -INFINITY
                                      : vals[j] * signal_factor(__ldcg(ne + src * d.m + u), d.lambda, d.T, d.signal);
                }
                __syncthreads();
            }
        }
    }
    pc.mark();
    // the window rows do not depend on the selection (their loads return while the scores are stored)
    if (gathers) copy_rows(B, (long long)d.W * 2 * vpr, [&](int t) { return (long long)(N + (t - B)); });
    if ((a.a || a.has_graph) && holds && a.keep_scores) store_chunk(row_s + base, vals, n_local);
    pc.mark();

    if (a.do_select) {
        int *idx = a.idx_out + (long long)unit * d.B;
        // the kept positions also go into every CTA's shared memory (the fine histogram's words,
        // idle by then), so that the gather neither waits for global writes of other CTAs to become
        // visible nor for a load of the index ahead of every row
        int *idx_s = reinterpret_cast<int *>(s.fine);
        const bool mirrored = gathers && B <= kFineBins;
        if (holds) {
            // rank only the elements that reach a lower bound of the B-th largest, where one is at hand
            // (the staging arrays of the lists are free by now)
            int *list = s.st_idx;
            // (a short chunk is ranked whole: the passes that list candidates would cost more,
            // and a budget above a sixteenth of the chunk leaves too many to gain anything)
            const bool sparse = (long long)B * 16 <= a.chunk;
            const int n_c = a.chunk >= 4 * kStage && sparse
                                ? filter_candidates(s, vals, n_local, (uint32_t)B, list, 4 * kStage) : -1;
            pc.mark();
            const RowView row{vals, n_c >= 0 ? list : nullptr, n_c >= 0 ? n_c : n_local};
            // a sparse selection takes the one-pass search, a dense one the digit-by-digit search
            // (its threshold bin would hold too many elements to rank by counting)
            const Threshold th = sparse ? cluster_kth_fine(cl, R, rank, s, row, base, (uint32_t)B, pc)
                                        : cluster_kth(cl, R, rank, s, row, (uint32_t)B);
            cluster_emit_sorted(cl, R, rank, s, row, base, th, idx, mirrored ? idx_s : nullptr, C);
        }
        pc.mark();
        if (!mirrored) __threadfence();
        if (C > 1) cl.sync(); else __syncthreads();
        pc.mark();
        // gather: the cluster's threads share the 16-byte pieces of the B kept rows
        if (gathers)
            copy_rows(0, (long long)B * 2 * vpr,
                      [&](int t) { return (long long)(mirrored ? idx_s[t] : __ldcg(idx + t)); });
    }
    pc.mark();
    if (C > 1) cl.sync();      // no CTA leaves while its shared memory may still be read
    pc.mark();
    pc.flush(rank == 0 ? 4 : 6);      // the first CTA of a cluster and the others apart
}

}  // namespace cs
}  // namespace graphkv
