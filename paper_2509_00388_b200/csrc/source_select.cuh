// Eq. 2 without a kernel of its own: the source nodes of a unit, the top-k of the POOLED scores
// s_j = max(a[j - h .. j + h]), found without pooling the whole row.
//
// Every CTA of the emit sweep lists, at its tail, the elements of its key chunk whose attention
// mass reaches the chunk's own k-th largest (first by the chunk's mass histogram, then exactly
// among those: k of them plus ties).  Every CTA of the similarity sweep that follows merges the
// lists of its unit for itself, before it gathers the source keys.  Let v be the k-th largest
// mass of the unit (it is among the listed: an element that k others of its own chunk exceed
// cannot be it).  Pooling only raises values, so k positions have s >= v and every source has
// s_j >= v; such a position lies within h of an element with a >= v.  The elements with a >= v
// (k of them plus ties) are all listed, so the merge pools exactly the positions within h of
// them, ranks those (score descending, position ascending) and keeps k.  Rows with massive ties
// (more than kSrcPeaks elements at or above v, or a chunk list that outgrew its slots) take a
// plain radix search over the pooled row instead: rare, and slow.
#pragma once

#include "common.cuh"

namespace graphkv {
namespace tc {

constexpr int kSrcCap = 128;          // listed elements per chunk
constexpr int kSrcMaxK = 64;          // source counts this path serves
constexpr int kSrcPeaks = 256;        // elements at or above v the merge pools around
constexpr int kSrcPool = 2048;        // pooled positions the merge ranks
constexpr int kSrcMerge = 4096;       // listed elements of a unit the merge holds

struct SrcCand {
    float a;
    int j;
};

struct SourceArgs {
    int k;                  // sources per unit (0: this tail does nothing)
    int halo;               // h = (pool_kernel - 1) / 2
    int *src_out;           // [units][k] ascending positions
    SrcCand *cand;          // [units][chunk_slots][kSrcCap] listed elements per chunk
    int *cand_n;            // [units][chunk_slots] their number (kSrcCap + 1: the list overflowed)
    int chunk_slots;
    int chunks;             // lists per unit (the key chunks of the emit sweep)
};

// Shared memory the tail needs, in bytes (it reuses the stage ring of the sweep, idle by then).
constexpr int kSrcSmemBytes = kSrcMerge * 8 + kSrcPeaks * 4 + kSrcPool * 8 + 2048 * 4 + 256;

// pooled score of position j from the unit's mass row in global memory
__device__ __forceinline__ float pooled_at(const float *a_row, int j, int h, int N)
{
    float best = -INFINITY;
    for (int t = max(j - h, 0); t <= min(j + h, N - 1); ++t) best = fmaxf(best, __ldcg(a_row + t));
    return best;
}

// Top-k of the pooled row by a radix search over the row in global memory (11 + 11 + 10 bits),
// all threads of the CTA; positions come out ascending in src_out.  `hist` holds 2048 words,
// `list` k ints, `misc` 8 words of shared memory.
__device__ void source_select_general(const float *a_row, int N, int h, int k, int *src_out,
                                      uint32_t *hist, int *list, uint32_t *misc)
{
    const int tid = threadIdx.x, nthr = blockDim.x;
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)k;
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t nb = pass == 2 ? 1024u : 2048u;
        for (int i = tid; i < 2048; i += nthr) hist[i] = 0u;
        __syncthreads();
        for (int j = tid; j < N; j += nthr) {
            const uint32_t u = float_to_key(pooled_at(a_row, j, h, N));
            if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & (nb - 1u)], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            uint32_t run = 0;
            int b = (int)nb - 1;
            for (; b > 0; --b) {
                if (run + hist[b] >= remaining) break;
                run += hist[b];
            }
            misc[0] = (uint32_t)b;
            misc[1] = remaining - run;
        }
        __syncthreads();
        prefix |= misc[0] << shift;
        mask |= (nb - 1u) << shift;
        remaining = misc[1];
        __syncthreads();
    }
    // positions above the threshold in any order, then the `remaining` lowest positions at it
    if (tid == 0) {
        misc[2] = 0u;
        misc[3] = 0u;
    }
    __syncthreads();
    for (int j = tid; j < N; j += nthr)
        if (float_to_key(pooled_at(a_row, j, h, N)) > prefix) list[atomicAdd(&misc[2], 1u)] = j;
    __syncthreads();
    const int n_gt = (int)misc[2];
    for (int j0 = 0; j0 < N && (int)misc[3] < (int)remaining; j0 += nthr) {
        const int j = j0 + tid;
        const bool eq = j < N && float_to_key(pooled_at(a_row, j, h, N)) == prefix;
        // ordered slots inside the block of positions: count the equal ones at lower positions
        __shared__ uint32_t warp_cnt[32];
        const unsigned bm = __ballot_sync(0xffffffffu, eq);
        if ((tid & 31) == 0) warp_cnt[tid >> 5] = __popc(bm);
        __syncthreads();
        uint32_t before = misc[3];
        for (int w = 0; w < (tid >> 5); ++w) before += warp_cnt[w];
        before += __popc(bm & ((1u << (tid & 31)) - 1u));
        if (eq && before < remaining) list[n_gt + (int)before] = j;
        __syncthreads();
        if (tid == 0) {
            uint32_t tot = 0;
            for (int w = 0; w < (nthr + 31) / 32; ++w) tot += warp_cnt[w];
            misc[3] += tot;
        }
        __syncthreads();
    }
    for (int i = tid; i < k; i += nthr) {
        const int p = list[i];
        int o = 0;
        for (int u = 0; u < k; ++u) o += list[u] < p;
        src_out[o] = p;
    }
}

// Called by all threads of an emit CTA after its tile loop (the chunk's mass values are in global
// memory, its mass histogram in `mass_hist`): lists the chunk's candidates for the merge.
// `scratch`: kSrcSmemBytes of shared memory.
__device__ void source_list_chunk(const SourceArgs &sa, const Dims &d, int unit, int chunk,
                                  int j_begin, int j_end, const float *a_row,
                                  const uint32_t *mass_hist, uint8_t *scratch)
{
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int k = sa.k;
    (void)d;
    SrcCand *merged = reinterpret_cast<SrcCand *>(scratch);                    // [kSrcMerge]
    uint32_t *misc = reinterpret_cast<uint32_t *>(merged + kSrcMerge);         // [64]
    // 1. the chunk's threshold bin: the highest bin with k of its elements in or above it
    if (tid == 0) {
        misc[0] = 0u;
        misc[1] = 0u;
    }
    __syncthreads();
    {
        // thread t < 512 owns bins 2047 - 4t - q; a suffix count over warps through shared memory
        uint32_t c[4] = {0u, 0u, 0u, 0u}, sum = 0;
        if (tid < 512)
            for (int q = 0; q < 4; ++q) {
                c[q] = mass_hist[2047 - 4 * tid - q];
                sum += c[q];
            }
        uint32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31 && warp < 16) misc[8 + warp] = incl;
        __syncthreads();
        uint32_t before = 0;
        for (int w = 0; w < warp && w < 16; ++w) before += misc[8 + w];
        uint32_t run = before + incl - sum;
        if (tid < 512)
            for (int q = 0; q < 4; ++q) {
                if (run < (uint32_t)k && run + c[q] >= (uint32_t)k) misc[0] = (uint32_t)(2047 - 4 * tid - q);
                run += c[q];
            }
        __syncthreads();
    }
    const uint32_t b_loc = misc[0];
    // 2. list the chunk's elements of the bins >= b_loc
    SrcCand *mine = merged;                                 // the own list is staged here first
    for (int j0 = j_begin; j0 < j_end; j0 += nthr) {
        const int j = j0 + tid;
        if (j < j_end) {
            const float av = __ldcg(a_row + j);
            if ((float_to_key(av) >> 21) >= b_loc) {
                const uint32_t slot = atomicAdd(&misc[1], 1u);
                if (slot < (uint32_t)kSrcCap) mine[slot] = SrcCand{av, j};
            }
        }
    }
    __syncthreads();
    int n_mine = (int)misc[1];
    const long long slot0 = (long long)unit * sa.chunk_slots + chunk;
    if (n_mine > k && n_mine <= kSrcCap) {
        // the bin is coarse: keep only the elements at or above the chunk's exact k-th largest
        // (rank by counting: mass descending, position ascending)
        SrcCand me{0.f, 0};
        if (tid < n_mine) {
            me = mine[tid];
            int r = 0;
            for (int u = 0; u < n_mine; ++u) {
                const SrcCand o = mine[u];
                r += (o.a > me.a) | ((o.a == me.a) & (o.j < me.j));
            }
            if (r == k - 1) misc[7] = __float_as_uint(me.a);
        }
        if (tid == 0) misc[1] = 0u;
        __syncthreads();
        const float v_loc = __uint_as_float(misc[7]);
        if (tid < n_mine && me.a >= v_loc) sa.cand[slot0 * kSrcCap + atomicAdd(&misc[1], 1u)] = me;
        __syncthreads();
        n_mine = (int)misc[1];
    } else {
        for (int i = tid; i < min(n_mine, kSrcCap); i += nthr) sa.cand[slot0 * kSrcCap + i] = mine[i];
    }
    if (tid == 0) sa.cand_n[slot0] = n_mine > kSrcCap ? kSrcCap + 1 : n_mine;
}

// Called by all threads of a CTA (at least kSrcPeaks of them) once every list of the unit is
// complete: the unit's k sources by ascending position into `out` (shared memory) and, when
// `out_global` is given, into global memory too.  `scratch`: kSrcSmemBytes of shared memory.
// Ends with the CTA synchronised.
__device__ void source_merge(const SourceArgs &sa, const Dims &d, int unit, const float *a_row,
                             uint8_t *scratch, int *out, int *out_global)
{
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int k = sa.k, h = sa.halo, N = d.N, chunks = sa.chunks;
    SrcCand *merged = reinterpret_cast<SrcCand *>(scratch);                    // [kSrcMerge]
    int *peaks = reinterpret_cast<int *>(merged + kSrcMerge);                  // [kSrcPeaks]
    SrcCand *pool = reinterpret_cast<SrcCand *>(peaks + kSrcPeaks);            // [kSrcPool]
    uint32_t *hist = reinterpret_cast<uint32_t *>(pool + kSrcPool);            // [2048]
    uint32_t *misc = hist + 2048;                                              // [64]
    if (tid == 0) {
        misc[3] = 0u;                                       // merged elements
        misc[4] = 0u;                                       // 1: take the general path
        misc[5] = 0u;                                       // peaks
        misc[6] = 0u;                                       // pooled positions
    }
    __syncthreads();
    for (int c = warp; c < chunks; c += nthr / 32) {
        const int n = __ldcg(sa.cand_n + (long long)unit * sa.chunk_slots + c);
        uint32_t base = 0;
        if (lane == 0) {
            if (n > kSrcCap) misc[4] = 1u;
            else base = atomicAdd(&misc[3], (uint32_t)n);
        }
        base = __shfl_sync(0xffffffffu, base, 0);
        if (n <= kSrcCap && base + n <= (uint32_t)kSrcMerge) {
            const unsigned long long *src =
                reinterpret_cast<const unsigned long long *>(sa.cand + ((long long)unit * sa.chunk_slots + c) * kSrcCap);
            for (int i = lane; i < n; i += 32)
                reinterpret_cast<unsigned long long *>(merged)[base + i] = __ldcg(src + i);
        }
    }
    __syncthreads();
    const int M = (int)misc[3];
    bool general = misc[4] != 0u || M > kSrcMerge || M < k;
    if (!general) {
        // v: the value of the element of rank k-1 (mass descending, position ascending)
        for (int i = tid; i < M; i += nthr) {
            const SrcCand me = merged[i];
            int r = 0;
            for (int u = 0; u < M; ++u) {
                const SrcCand o = merged[u];
                r += (o.a > me.a) | ((o.a == me.a) & (o.j < me.j));
            }
            if (r == k - 1) misc[7] = __float_as_uint(me.a);
        }
        __syncthreads();
        const float v = __uint_as_float(misc[7]);
        // the elements at or above v, by ascending position
        for (int i = tid; i < M; i += nthr)
            if (merged[i].a >= v) {
                const uint32_t slot = atomicAdd(&misc[5], 1u);
                if (slot < (uint32_t)kSrcPeaks) peaks[slot] = merged[i].j;
            }
        __syncthreads();
        const int nP = (int)misc[5];
        general = nP > kSrcPeaks || nP * (2 * h + 1) > kSrcPool;
        if (!general) {
            int *sorted = reinterpret_cast<int *>(merged);      // the merged list is no longer needed
            int my_pos = 0, my_rank = 0;                        // nP <= kSrcPeaks <= threads of the CTA
            if (tid < nP) {
                my_pos = peaks[tid];
                for (int u = 0; u < nP; ++u) my_rank += peaks[u] < my_pos;
            }
            __syncthreads();
            if (tid < nP) sorted[my_rank] = my_pos;
            __syncthreads();
            // pool the positions within h of them, each position once
            const int kp = 2 * h + 1;
            for (int w = tid; w < nP * kp; w += nthr) {
                const int i = w / kp, j = sorted[i] + (w - i * kp) - h;
                const bool dup = i > 0 && j <= sorted[i - 1] + h;
                if (j >= 0 && j < N && !dup) {
                    const uint32_t slot = atomicAdd(&misc[6], 1u);
                    pool[slot] = SrcCand{pooled_at(a_row, j, h, N), j};
                }
            }
            __syncthreads();
            const int nS = (int)misc[6];
            // keep the k best (score descending, position ascending), emit by ascending position
            int *kept = peaks;                                  // k <= kSrcMaxK <= kSrcPeaks
            if (tid == 0) misc[5] = 0u;
            __syncthreads();
            for (int i = tid; i < nS; i += nthr) {
                const SrcCand me = pool[i];
                int r = 0;
                for (int u = 0; u < nS; ++u) {
                    const SrcCand o = pool[u];
                    r += (o.a > me.a) | ((o.a == me.a) & (o.j < me.j));
                }
                if (r < k) kept[atomicAdd(&misc[5], 1u)] = me.j;
            }
            __syncthreads();
            if (tid < k) {
                const int p = kept[tid];
                int o = 0;
                for (int u = 0; u < k; ++u) o += kept[u] < p;
                out[o] = p;
                if (out_global) out_global[o] = p;
            }
            __syncthreads();
            return;
        }
    }
    __syncthreads();
    source_select_general(a_row, N, h, k, out, hist, reinterpret_cast<int *>(merged), misc);
    __syncthreads();
    if (out_global)
        for (int i = tid; i < k; i += nthr) out_global[i] = out[i];
    __syncthreads();
}

}  // namespace tc
}  // namespace graphkv
