// Steps (II)+(III), first half, on the tensor cores (bf16 inputs): the edges e_ij of Eq. 1 between
// the source nodes of a head and every prefix key, and per key chunk the candidates for each
// source's top-m neighbourhood (Eq. 3).  The edge matrix never leaves the SM.
//
// One CTA owns a chunk of at most 512 / NP key tiles of one head (NP = source count padded to
// 16, 32 or 64; a head with more sources is swept once per 64 of them, by CTAs of their own).  Each 128-key tile arrives by TMA, one tcgen05.mma block computes its
// 128 x NP dot products against the source keys into its own TMEM columns, and the epilogue
// threads (thread = key) take the key's norm from the staged tile.  When the sweep is over the
// chunk's whole edge block still sits in TMEM, and the CTA
//   1. takes, per source, a threshold bin that at least m eligible edges of the chunk reach:
//      the highest cosine bin such that m+1 of the per-thread maxima lie in or above it (distinct
//      threads hold distinct keys, and at most one of them is the source itself);
//   2. re-reads TMEM and lists the edges whose bin (the same expression as in step 1, so that a
//      counted maximum is always listed) reaches it, excluding the source itself;
//   3. if a list outgrows its capacity (many ties), finds that source's exact m-th largest
//      (edge descending, position ascending) by a byte-wise radix search over TMEM and lists
//      exactly those m.
// The lists of all chunks hold every member of the head-wide top-m.  Each listed edge is also
// counted in a per-source histogram over the cosine, from which the row-wise finishing kernel
// takes a bound that leaves it a few dozen edges to rank.
#pragma once

#include "source_select.cuh"
#include "tc_common.cuh"

namespace graphkv {
namespace tc {

constexpr int kSimThreads = 320;
constexpr int kSimEpiThreads = 256;
constexpr int kSimMaxNeighbors = 32;    // m this path handles
constexpr int kSimMaxTiles = 32;        // tiles per CTA at NP = 16 (512 TMEM columns)
constexpr int kMaxBins = 256;           // cosine bins over [-1, 1] for the per-thread maxima

struct SimTcArgs {
    Dims d;
    const __nv_bfloat16 *S;   // tensor the source nodes' vectors are read from (the swept tensor comes
                              // through the tensor map)
    long long ss[3];          // its element strides: batch, head, token
    const int *src;        // [units][K_src] source positions
    Cand *cand;            // [units][K_src][chunks][kCandCap]; unused slots hold e = kCandEmpty
    uint32_t *cand_hist;   // [units][K_src][kCandBins] listed edges per cosine bin (zeroed before)
    int *status;
    int unit0;
    int chunks;            // CTAs per unit
    int n_tiles;           // 128-key tiles per unit
    int stages;
    int wait_prior;        // launched with programmatic stream serialization
    long long wait_cycles; // limit of every wait of the kernel, in clocks
    SourceArgs merge;      // merge.k > 0: the sources are not in `src` yet; every CTA merges the candidate
                           // lists the emit sweep left (Eq. 2) and the first chunk of a unit writes them to `src`
    const float *a_mass;   // [units][N] attention mass the merge pools (merge.k > 0)
};

template <int NP> __host__ __device__ constexpr int sim_tiles_cap() { return 512 / NP; }

// Dynamic shared memory (1024-byte aligned base):
//   [0, NP*256)                      source keys, K-major 128-byte swizzle (two 64-column halves)
//   [.., + stages*32 KB)             key tiles in flight; reused for the per-thread maxima
//   barriers, inverse norms of the chunk's keys, source bookkeeping, candidate lists
template <int NP> __host__ __device__ inline size_t sim_smem_bytes(int stages)
{
    return 1024 + (size_t)NP * 256 + (size_t)stages * kTileBytes + (8 + 8 + kSimMaxTiles) * 8 + 16 +
           (size_t)sim_tiles_cap<NP>() * 128 * 4 + (size_t)NP * 6 * 4 + (size_t)NP * kCandCap * 8 + 64;
}

template <int NP>
__device__ __forceinline__ void tmem_ld_np(uint32_t taddr, float (&v)[NP])
{
    if constexpr (NP == 16) {
        tmem_ld16(taddr, v);
    } else {
#pragma unroll
        for (int c = 0; c < NP / 32; ++c) {
            float t[32];
            tmem_ld32(taddr + c * 32, t);
#pragma unroll
            for (int i = 0; i < 32; ++i) v[c * 32 + i] = t[i];
        }
    }
}

template <int NP>
__global__ void __launch_bounds__(kSimThreads, 1)
similarity_tc(const __grid_constant__ CUtensorMap tmK, SimTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kTilesCap = sim_tiles_cap<NP>();
    const Dims &d = a.d;
    const long long lim = a.wait_cycles;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t s_src = base;
    const uint32_t s_stage0 = s_src + NP * 256;
    const uint32_t s_full0 = s_stage0 + a.stages * kTileBytes;
    const uint32_t s_empty0 = s_full0 + 8 * 8;
    const uint32_t s_done0 = s_empty0 + 8 * 8;
    const uint32_t s_tmem = s_done0 + kSimMaxTiles * 8;
    const uint32_t s_invn = s_tmem + 16;
    const uint32_t s_book = s_invn + kTilesCap * 128 * 4;
    const uint32_t s_list = s_book + NP * 6 * 4;
    float *inv_norm = reinterpret_cast<float *>(gen + (s_invn - base));        // [tile][128]
    int *src_pos = reinterpret_cast<int *>(gen + (s_book - base));              // [NP]
    float *src_inv = reinterpret_cast<float *>(src_pos + NP);                   // [NP]
    float *tau = src_inv + NP;                                                  // [NP] threshold cosine
    int *cnt = reinterpret_cast<int *>(tau + NP);                               // [NP]
    int *tau_bin = cnt + NP;                                                    // [NP] bin whose lower edge tau is
    float *src_norm = reinterpret_cast<float *>(tau_bin + NP);                  // [NP] max(|k_c|, eps)
    Cand *list = reinterpret_cast<Cand *>(gen + (s_list - base));               // [NP][kCandCap]
    // after the sweep the stage memory holds the bins of the maxima and the threads' edge queues
    // (a key position takes 26 bits there: rows this kernel is given are shorter than 2^18 keys)
    constexpr int kQueueCap = 32;                                               // edges per thread
    uint32_t *max_bin = reinterpret_cast<uint32_t *>(gen + (s_stage0 - base));  // [NP / 4][256] bytes = 4 sources
    uint2 *queue = reinterpret_cast<uint2 *>(max_bin + (NP / 4) * kSimEpiThreads);  // [kQueueCap][256]
    int *xchg = reinterpret_cast<int *>(gen + (s_tmem - base)) + 2;             // 2 words

    PhaseClock pc(threadIdx.x == 64);
    pc.mark();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    const int per = a.n_tiles / a.chunks, rem = a.n_tiles % a.chunks;
    const int t0 = chunk * per + min(chunk, rem);
    const int n_local = per + (chunk < rem ? 1 : 0);
    const __nv_bfloat16 *Sh = a.S + b * a.ss[0] + (long long)h * a.ss[1];
    // a head with more than NP sources is swept once per NP of them: grid.z counts those sweeps
    const int src0 = blockIdx.z * NP;
    const int *src = a.src + (long long)unit * d.K_src + src0;
    const int n_src = min(NP, d.K_src - src0);               // sources of this CTA

    int n_ahead = 0;                 // tiles thread 0 has requested before the roles split
    if (threadIdx.x == 0) {
        for (int i = 0; i < a.stages; ++i) {
            mbar_init(s_full0 + 8 * i, 1);
            mbar_init(s_empty0 + 8 * i, 1 + 4);       // MMA commit + the four norm warps of a tile
        }
        for (int i = 0; i < kSimMaxTiles; ++i) mbar_init(s_done0 + 8 * i, 1);
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        // the first ring-full of key tiles is under way while the sources are gathered (keys are an
        // input of the call: no wait for the kernels before)
        // (a merge of candidate lists borrows the last two stages as scratch first)
        n_ahead = min(a.merge.k > 0 ? a.stages - 2 : a.stages, n_local);
        for (int i = 0; i < n_ahead; ++i) {
            const uint32_t dst = s_stage0 + i * kTileBytes;
            mbar_expect_tx(s_full0 + 8 * i, kTileBytes);
            tma_load_4d(dst, &tmK, s_full0 + 8 * i, 0, (t0 + i) * kTileKeys, h, b);
            tma_load_4d(dst + kHalfBytes, &tmK, s_full0 + 8 * i, 64, (t0 + i) * kTileKeys, h, b);
        }
    }
    if (warp == 1) {
        tmem_alloc(s_tmem, 512);
        tmem_relinquish();
    }
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    pc.mark();
    if (a.merge.k > 0) {
        static_assert(2 * kTileBytes >= kSrcSmemBytes, "the merge's scratch fits two stages");
        source_merge(a.merge, d, unit, a.a_mass + (long long)unit * d.N,
                     gen + (s_stage0 - base) + (a.stages - 2) * kTileBytes, src_pos,
                     chunk == 0 ? const_cast<int *>(src) : nullptr);
    }
    // source keys -> swizzled operand rows (rows >= K_src are zero), their positions and norms
    // (16 consecutive threads share a row: the row's squared norm is reduced among them)
    for (int i0 = 0; i0 < NP * 16; i0 += kSimThreads) {
        const int i = i0 + threadIdx.x;
        const int r = i >> 4, c16 = i & 15;
        const bool in = i < NP * 16;
        uint4 v = make_uint4(0, 0, 0, 0);
        int pos = -1;
        if (in && r < n_src) {
            pos = a.merge.k > 0 ? src_pos[r] : src[r];
            v = *reinterpret_cast<const uint4 *>(Sh + (long long)pos * a.ss[2] + c16 * 8);
        }
        if (in) *reinterpret_cast<uint4 *>(gen + sw128_offset(NP, r, c16)) = v;
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float n2 = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float lo = __uint_as_float(w[q] << 16), hi = __uint_as_float(w[q] & 0xffff0000u);
            n2 = fmaf(lo, lo, fmaf(hi, hi, n2));
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
        if (in && c16 == 0) {
            src_pos[r] = pos;
            src_norm[r] = fmaxf(sqrtf(n2), kNormEps);
            src_inv[r] = 1.0f / fmaxf(sqrtf(n2), kNormEps);
            cnt[r] = 0;
        }
    }
    if (threadIdx.x == 0) xchg[0] = 1;
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(gen + (s_tmem - base));
    bool ok = true;
    pc.mark();

    if (warp == 0) {
        if (lane == 0) {
            int issued = n_ahead;
            for (int i = n_ahead; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                if (!mbar_wait(s_empty0 + 8 * st, ph ^ 1, lim)) { ok = false; break; }
                const uint32_t dst = s_stage0 + st * kTileBytes;
                mbar_expect_tx(s_full0 + 8 * st, kTileBytes);
                tma_load_4d(dst, &tmK, s_full0 + 8 * st, 0, (t0 + i) * kTileKeys, h, b);
                tma_load_4d(dst + kHalfBytes, &tmK, s_full0 + 8 * st, 64, (t0 + i) * kTileKeys, h, b);
                ++issued;
            }
            if (!ok)        // gave up: let the copies already in flight land before the CTA exits
                for (int i = max(0, issued - a.stages); i < issued; ++i)
                    mbar_wait(s_full0 + 8 * (i % a.stages), (i / a.stages) & 1, lim);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, NP);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                if (!mbar_wait(s_full0 + 8 * st, ph, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t kt = s_stage0 + st * kTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
                    const uint32_t soff = (k >> 2) * (NP * 128) + (k & 3) * 32;
                    umma_bf16(tmem_base + i * NP, umma_desc_sw128(kt + koff),
                              umma_desc_sw128(s_src + soff), idesc, k > 0);
                }
                umma_commit(s_empty0 + 8 * st);
                umma_commit(s_done0 + 8 * i);
            }
        }
    } else {
        // ---- epilogue threads: thread = key (TMEM lane); the two warp sets alternate tiles ----
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int key_lane = quad * 32 + lane;
        const int et = set * 128 + key_lane;                   // epilogue thread id, 0..255
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        float best[NP];                     // per source: max over this thread's keys of dot / |k_j|
#pragma unroll
        for (int c = 0; c < NP; ++c) best[c] = -INFINITY;
        bool alive = true;
        for (int i = set; i < n_local; i += 2) {
            const int st = i % a.stages, ph = (i / a.stages) & 1;
            float inv = 0.f;
            if (alive) alive = __all_sync(0xffffffffu, mbar_wait(s_full0 + 8 * st, ph, lim));
            if (alive) {
                // squared norm of this thread's key from the staged tile
                const uint8_t *tile = gen + (s_stage0 - base) + st * kTileBytes;
                float n0 = 0.f, n1 = 0.f;
#pragma unroll
                for (int c16 = 0; c16 < 16; ++c16) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(tile + sw128_offset(128, key_lane, c16));
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float lo = __uint_as_float(w[q] << 16), hi = __uint_as_float(w[q] & 0xffff0000u);
                        n0 = fmaf(lo, lo, n0);
                        n1 = fmaf(hi, hi, n1);
                    }
                }
                inv = 1.0f / fmaxf(sqrtf(n0 + n1), kNormEps);
                inv_norm[i * 128 + key_lane] = inv;
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty0 + 8 * st);
                alive = __all_sync(0xffffffffu, mbar_wait(s_done0 + 8 * i, 0, lim));
            }
            if (alive) {
                tc_fence_after();
                float v[NP];
                tmem_ld_np<NP>(lane_addr + i * NP, v);
                if ((t0 + i) * kTileKeys + key_lane < d.N) {
#pragma unroll
                    for (int c = 0; c < NP; ++c) best[c] = fmaxf(best[c], v[c] * inv);
                }
            }
        }
        ok = alive;
        pc.mark();
        // every tile's copies and MMAs are complete once both sets are here: the stage memory is free
        if (!alive && lane == 0) xchg[0] = 0;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const bool all_alive = xchg[0] != 0;
        if (all_alive) {
            if (et == 0) xchg[1] = 0;
            // 1. thresholds.  The cosine of a thread's best key for source c is the rounded product
            //    of its best dot / |k_j| with 1 / |k_c| (rounding is monotone).  Every thread leaves
            //    the cosine bins (of kMaxBins over [-1, 1]) of its maxima, four sources to a word; a
            //    warp takes two sources at a time and finds for each, by bisection over the bin index, the
            //    highest bin with m+1 maxima in or above it; tau is that bin's lower edge.
            //    (A thread without keys counts in bin 0, which only matters when tau is -1 anyway.)
#pragma unroll
            for (int g = 0; g < NP / 4; ++g) {
                uint32_t word = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int c = g * 4 + q;
                    int bin = 0;
                    if (c < n_src && best[c] > -INFINITY) {
                        const float e = fminf(fmaxf(best[c] * src_inv[c], -1.0f), 1.0f);
                        bin = min(max(static_cast<int>((e + 1.0f) * (kMaxBins / 2)), 0), kMaxBins - 1);
                    }
                    word |= (uint32_t)bin << (8 * q);
                }
                max_bin[g * kSimEpiThreads + et] = word;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            pc.mark();
            const int ew = warp - 2;
            for (int pr = ew; pr * 2 < n_src; pr += 8) {
                const int g = pr >> 1, sh = (pr & 1) * 16;       // the pair's word and its two bytes there
                uint32_t w8[8];              // this lane's eight threads' bins of sources 4g .. 4g+3
                {
                    const uint4 lo = *reinterpret_cast<const uint4 *>(max_bin + g * kSimEpiThreads + lane * 8);
                    const uint4 hi = *reinterpret_cast<const uint4 *>(max_bin + g * kSimEpiThreads + lane * 8 + 4);
                    w8[0] = lo.x; w8[1] = lo.y; w8[2] = lo.z; w8[3] = lo.w;
                    w8[4] = hi.x; w8[5] = hi.y; w8[6] = hi.z; w8[7] = hi.w;
                }
                uint32_t bstar[2] = {0u, 0u};
#pragma unroll
                for (int bit = 7; bit >= 0; --bit) {
                    int n[2];
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const uint32_t cand = bstar[q] | (1u << bit);
                        n[q] = 0;
#pragma unroll
                        for (int k = 0; k < 8; ++k) n[q] += ((w8[k] >> (sh + 8 * q)) & 0xffu) >= cand ? 1 : 0;
                    }
                    // both counts in one reduction (each at most 256)
                    const uint32_t both = __reduce_add_sync(0xffffffffu, (uint32_t)n[0] | ((uint32_t)n[1] << 16));
                    if ((int)(both & 0xffffu) >= d.m + 1) bstar[0] |= 1u << bit;
                    if ((int)(both >> 16) >= d.m + 1) bstar[1] |= 1u << bit;
                }
                if (lane < 2 && pr * 2 + lane < n_src) {
                    const uint32_t bs = lane == 0 ? bstar[0] : bstar[1];
                    tau[pr * 2 + lane] = bs == 0 ? -1.0f : (float)bs * (2.0f / kMaxBins) - 1.0f;
                    tau_bin[pr * 2 + lane] = (int)bs;
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            pc.mark();
            // 2. list the edges that reach the threshold bin.  theta is the bin's lower edge brought to
            //    the scale of dot / |k_j|, lowered (the bin index rounds: a cosine a few 1e-8 under
            //    the edge still lands in the bin) so that no edge of the bin is missed.
            //    Straight-line code: a thread appends the few edges of its keys that pass, as
            //    (value, source and key), to a queue of its own; afterwards it turns each into a
            //    cosine, checks its bin against the threshold bin and adds it to the source's list (the order
            //    within a list carries no meaning).  A queue that fills up sends every source of the
            //    chunk down the exact path of step 3.
            float theta[NP];
#pragma unroll
            for (int c = 0; c < NP; ++c) {
                // (times the norm instead of divided by its rounded reciprocal: within 1.2e-7 of it,
                // inside the margin taken off below)
                const float q = c < n_src ? (tau[c] - 2.4e-7f) * src_norm[c] : INFINITY;
                theta[c] = q - fabsf(q) * 3.6e-7f - 1e-30f;
            }
            // (the store and the count under one predicate; a key past the end of the row gets a NaN
            // factor, which fails every comparison)
            uint2 *const q0 = queue + et;
            const uint32_t q_first = smem_u32(q0), q_step = kSimEpiThreads * sizeof(uint2);
            const uint32_t q_last = q_first + (kQueueCap - 1) * q_step;
            uint32_t qa = q_first;
            auto list_tile = [&](int i, const float (&v)[NP]) {
                const int j = (t0 + i) * kTileKeys + key_lane;
                const float inv = j < d.N ? inv_norm[i * 128 + key_lane] : __int_as_float(0x7fc00000);
                // few keys pass any threshold: the independent comparisons first, the appends (a
                // dependent chain through the queue's address) only for a key with an edge to list
                if constexpr (NP <= 32) {
                    bool any = false;
#pragma unroll
                    for (int c = 0; c < NP; ++c) any |= v[c] * inv >= theta[c];
                    if (!any) return;
                }
#pragma unroll
                for (int c = 0; c < NP; ++c) {
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t.reg .u32 a;\n\t"
                        "setp.ge.f32 p, %1, %3;\n\t"
                        "min.u32 a, %0, %4;\n\t"
                        "@p st.shared.v2.b32 [a], {%1, %2};\n\t"
                        "@p add.u32 %0, %0, %5;\n\t}"
                        : "+r"(qa)
                        : "f"(v[c] * inv), "r"(((uint32_t)c << 26) | (uint32_t)j), "f"(theta[c]), "r"(q_last),
                          "r"(q_step)
                        : "memory");
                }
            };
            if constexpr (NP <= 32) {
                // the loads of two tiles are in flight together (a deeper unrolled body costs more in
                // instruction fetches than it hides: the body runs a few times per CTA)
                constexpr int kDepth = 2;
                for (int i0 = set; i0 < n_local; i0 += 2 * kDepth) {
                    uint32_t raw[kDepth][NP];
#pragma unroll
                    for (int q = 0; q < kDepth; ++q)
                        if (i0 + 2 * q < n_local) {                  // uniform over the warp
                            if constexpr (NP == 16) tmem_ld16_issue(lane_addr + (i0 + 2 * q) * NP, raw[q]);
                            else tmem_ld32_issue(lane_addr + (i0 + 2 * q) * NP, raw[q]);
                        }
#pragma unroll
                    for (int q = 0; q < kDepth; ++q) tmem_ld_fence(raw[q]);
#pragma unroll
                    for (int q = 0; q < kDepth; ++q)
                        if (i0 + 2 * q < n_local) {
                            float v[NP];
#pragma unroll
                            for (int c = 0; c < NP; ++c) v[c] = __uint_as_float(raw[q][c]);
                            list_tile(i0 + 2 * q, v);
                        }
                }
            } else {
                for (int i = set; i < n_local; i += 2) {
                    float v[NP];
                    tmem_ld_np<NP>(lane_addr + i * NP, v);
                    list_tile(i, v);
                }
            }
            pc.mark();
            const int n_queued = static_cast<int>((qa - q_first) / q_step);
            if (n_queued > kQueueCap) xchg[1] = 1;                    // entries were lost
            for (int k = 0; k < min(n_queued, kQueueCap); ++k) {
                const uint2 en = q0[k * kSimEpiThreads];
                const int c = en.y >> 26, j = en.y & 0x3ffffffu;
                const float e = fminf(fmaxf(__uint_as_float(en.x) * src_inv[c], -1.0f), 1.0f);
                const int bin = min(max(static_cast<int>((e + 1.0f) * (kMaxBins / 2)), 0), kMaxBins - 1);
                if (bin >= tau_bin[c] && j != src_pos[c]) {
                    const int pos = atomicAdd(&cnt[c], 1);
                    if (pos < kCandCap) list[c * kCandCap + pos] = Cand{e, j};
                }
            }
            pc.mark();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            {
                const bool lost = xchg[1] != 0;
                asm volatile("bar.sync 1, 256;" ::: "memory");
                for (int c = et; c < n_src; c += kSimEpiThreads) {
                    if (lost) cnt[c] = kCandCap + 1;
                    if (cnt[c] > kCandCap) xchg[1] = 1;               // some list overflowed
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            // 3. a list that outgrew its capacity: exact m-th largest (edge desc, position asc)
            const bool any_overflow = xchg[1] != 0;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            for (int c = 0; c < n_src && any_overflow; ++c) {
                if (cnt[c] <= kCandCap) continue;                 // uniform: shared memory value
                // the m-th largest 64-bit edge key of the chunk (keys are distinct: distinct positions),
                // a byte at a time from the top: a 256-bin histogram of the byte among the keys that
                // share the bytes found so far, the digit that holds the m-th largest, eight rounds
                unsigned long long t64 = 0ull;
                const float sinv = src_inv[c];
                const int self = src_pos[c];
                uint32_t *rh = max_bin;                           // [256] (the stage memory is idle)
                uint32_t remaining = (uint32_t)d.m;
                for (int byte = 7; byte >= 0; --byte) {
                    const unsigned long long hi_mask = byte == 7 ? 0ull : ~0ull << (8 * (byte + 1));
                    rh[et] = 0u;
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    for (int i = set; i < n_local; i += 2) {
                        const int j = (t0 + i) * kTileKeys + key_lane;
                        const float dot = tmem_ld1(lane_addr + i * NP + c);
                        const float e = fminf(fmaxf(dot * inv_norm[i * 128 + key_lane] * sinv, -1.0f), 1.0f);
                        const unsigned long long key = edge_key(e, j);
                        const bool valid = j < d.N && j != self && (key & hi_mask) == t64;
                        const uint32_t bin = (uint32_t)(key >> (8 * byte)) & 0xffu;
                        // (cosines of a chunk crowd into few digits: the lanes that share the first
                        // valid lane's digit are counted with one addition)
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
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    if (warp == 2) {
                        // lane l holds digits 255 - 8 l - q (q < 8): counts above each digit by a scan
                        uint32_t c8[8], sum = 0;
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            c8[q] = rh[255 - 8 * lane - q];
                            sum += c8[q];
                        }
                        uint32_t incl = sum;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= o) incl += t;
                        }
                        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
                        uint32_t run = incl - sum;
                        if (lane == 0) {
                            xchg[0] = 0;                            // fewer keys than m: every key is kept
                            xchg[1] = (int)remaining;
                        }
                        __syncwarp();
                        if (total >= remaining) {
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                if (run < remaining && run + c8[q] >= remaining) {
                                    xchg[0] = 255 - 8 * lane - q;
                                    xchg[1] = (int)(remaining - run);
                                }
                                run += c8[q];
                            }
                        }
                    }
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    t64 |= (unsigned long long)(uint32_t)xchg[0] << (8 * byte);
                    remaining = (uint32_t)xchg[1];
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
                if (et == 0) cnt[c] = 0;
                asm volatile("bar.sync 1, 256;" ::: "memory");
                for (int i = set; i < n_local; i += 2) {
                    const int j = (t0 + i) * kTileKeys + key_lane;
                    const float dot = tmem_ld1(lane_addr + i * NP + c);
                    const float e = fminf(fmaxf(dot * inv_norm[i * 128 + key_lane] * sinv, -1.0f), 1.0f);
                    if (j < d.N && j != self && edge_key(e, j) >= t64) {
                        const int pos = atomicAdd(&cnt[c], 1);
                        if (pos < kCandCap) list[c * kCandCap + pos] = Cand{e, j};
                    }
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            pc.mark();
            // write the lists out (unused slots marked empty) and count the listed edges per bin
            for (int idx = et; idx < n_src * kCandCap; idx += kSimEpiThreads) {
                const int c = idx / kCandCap, q = idx % kCandCap;
                const long long slot = ((long long)unit * d.K_src + src0 + c) * a.chunks + chunk;
                Cand cd{kCandEmpty, -1};
                if (q < min(cnt[c], kCandCap)) {
                    cd = list[c * kCandCap + q];
                    atomicAdd(a.cand_hist + ((long long)unit * d.K_src + src0 + c) * kCandBins + cand_bin(cd.e), 1u);
                }
                a.cand[slot * kCandCap + q] = cd;
            }
        } else {
            // a wait ran out: publish empty lists so the merge reads nothing undefined
            for (int i = et; i < n_src * kCandCap; i += kSimEpiThreads) {
                const long long slot = ((long long)unit * d.K_src + src0 + i / kCandCap) * a.chunks + chunk;
                a.cand[slot * kCandCap + i % kCandCap] = Cand{kCandEmpty, -1};
            }
        }
        pc.mark();
        tc_fence_before();
    }
    if (!ok && a.status) atomicExch(a.status, (int)GRAPHKV_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    pc.mark();
    pc.flush(2);
}

}  // namespace tc
}  // namespace graphkv
