// Step (I) on the tensor cores (bf16 inputs): SnapKV-style window-attention scores.
//
// Two sweeps over the keys of a head, both as TMA -> shared memory -> tcgen05.mma -> TMEM
// pipelines with the softmax arithmetic done on the accumulators as they come out of TMEM:
//   score_stats_tc  D = Q K^T  (query rows on TMEM lanes): per-row running max and sum of
//                   2^(l2 - max) over the keys the row may see, l2 = q.k/sqrt(D) * log2(e).
//   score_emit_tc   D = K Q^T  (keys on TMEM lanes): a[j] = sum_r 2^(l2[r][j] - c_r),
//                   c_r = max_r + log2(Z_r), i.e. the softmax probabilities summed over the
//                   window rows and grouped heads, one thread per key.
// The second sweep re-reads K right after the first, so it is served by L2 as far as the keys
// fit there.  The statistics CTAs of a unit leave their partial (max, sum) per row in global
// memory and the last of them to finish (an arrival counter) merges them into c_r.  One
// exponential in four is evaluated by a cubic on the FMA pipe: at 256 query rows per KV head the
// MUFU unit, not HBM, is the ceiling of both sweeps; the multiply-adds around the exponentials
// run on packed pairs (fma.rn.f32x2) to halve their issue slots.  Warp roles (576 threads):
// warp 0 = TMA producer (it starts on the key tiles before the dependency wait: keys are an
// input of the call), warp 1 = MMA issuer and TMEM owner, warps 2..17 = epilogue (four sets of
// four warps covering the four TMEM lane quadrants; a thread takes at most 64 accumulator
// columns of a tile, copies them to registers and frees the TMEM buffer before the arithmetic.
// At 256 query rows all four sets share each tile and two buffers alternate; at 128 or fewer two
// sets share a tile, the two pairs take alternate tiles and four buffers rotate).
#pragma once

#include "source_select.cuh"
#include "tc_common.cuh"

namespace graphkv {
namespace tc {

constexpr int kScoreThreads = 576;       // producer warp, MMA warp, 16 epilogue warps
constexpr int kMassBins = 2048;         // histogram of the attention mass: top 11 bits of float_to_key
constexpr int kEpiWarps = 16;
constexpr int kScratchBytes = 10240;     // row constants (1 KB) + four exchange buffers of 4 x 128 floats

struct ScoreTcArgs {
    Dims d;
    const __nv_bfloat16 *Q;
    float *part;        // [units][stats_chunks][GW][2] row statistics (max, sum) per key chunk
    float *row_c;       // [units][GW] c_r = max_r + log2(Z_r), written by the last stats CTA of a unit
    int *arrivals;      // [2 * units] words: the two-kernel path counts finished statistics CTAs in [unit]
                        // (zero before the launch; reset on the way), the kernel of both sweeps keeps a
                        // 64-bit (tag, count) word per unit there
    float *a_out;       // [units][N] attention mass before pooling
    uint32_t *a_hist;   // optional [units][kMassBins]: counts of a by the top bits of its ordered image
    int *status;        // workspace status word
    int unit0;          // first unit of this launch
    int chunks;         // key chunks (CTAs) per unit
    int n_tiles;        // 128-key tiles per unit in this sweep
    int stats_chunks;   // key chunks of the statistics sweep (partials per row)
    int stages;         // shared-memory K tiles in flight
    int wait_prior;     // launched with programmatic stream serialization: wait for the kernels before
    // emit sweep only: candidate lists for the source nodes of Eq. 2 at its tail (src.k = 0: none), and words to clear
    // for the kernels that follow
    SourceArgs src;
    uint32_t *zero;     // optional [units][zero_words]
    int zero_words;
    int local_hist;     // build the per-CTA mass histogram even without a_hist
    long long wait_cycles;   // limit of every wait of the kernel, in clocks
    int clear_head;          // kernel of both sweeps: clear the status word and the unit's mass histogram on
                             // the way (the caller then needs no memset ahead of the launch)
    uint32_t call_tag;       // kernel of both sweeps: a nonzero value no earlier call on this workspace used
    int withhold_commit;     // test hook (statistics sweep): 1: the MMA issuer leaves out the arrival that
                             // announces its first accumulator, so the wait for it runs out; 2 (kernel of
                             // both sweeps): no CTA announces itself at the hand-over, so that wait runs out
};

struct ScoreSmem {
    uint32_t q, stage0, full0, empty0, tfull0, tempty0, tmem_slot, xbar0, misc;
};

// Carve dynamic shared memory (1024-byte aligned base): Q operand, K stages, barriers.
__device__ __forceinline__ ScoreSmem score_smem_layout(uint8_t *raw, int rows_pad, int stages,
                                                       uint8_t **gen_base)
{
    const uint32_t base = (smem_u32(raw) + 1023u) & ~1023u;
    *gen_base = raw + (base - smem_u32(raw));
    ScoreSmem s;
    s.q = base;
    s.stage0 = s.q + rows_pad * 256;
    s.full0 = s.stage0 + stages * kTileBytes;
    s.empty0 = s.full0 + 8 * 8;
    s.tfull0 = s.empty0 + 8 * 8;
    s.tempty0 = s.tfull0 + 4 * 8;
    s.tmem_slot = s.tempty0 + 4 * 8;
    s.xbar0 = s.tmem_slot + 16;
    s.misc = s.xbar0 + 8 * 8;
    return s;
}

__host__ __device__ inline size_t score_smem_bytes(int rows_pad, int stages)
{
    return 1024 + (size_t)rows_pad * 256 + (size_t)stages * kTileBytes + 8 * 8 * 2 + 4 * 8 * 2 + 16 + 8 * 8 +
           kScratchBytes + 8192 + 64;   // scratch: the CTA's row statistics / row constants and the
                                        // exchange buffers; 8 KB: the emit sweep's histogram of the mass
}

// Q rows of the unit -> K-major swizzled operand (rows >= GW zero-filled).  Threads tid of
// nthreads; loads are issued four at a time ahead of the shared-memory stores.
__device__ __forceinline__ void stage_q(uint8_t *q_gen, int rows_pad, const Dims &d,
                                        const __nv_bfloat16 *Q, int b, int h, int tid, int nthreads)
{
    const __nv_bfloat16 *Qh = Q + b * d.qs[0] + (long long)(h * d.G) * d.qs[1];
    for (int i0 = tid; i0 < rows_pad * 16; i0 += 4 * nthreads) {
        uint4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = i0 + k * nthreads;
            const int r = i >> 4, c16 = i & 15;
            v[k] = make_uint4(0, 0, 0, 0);
            if (i < rows_pad * 16 && r < d.GW) {
                const int g = r / d.W, rw = r - g * d.W;
                v[k] = *reinterpret_cast<const uint4 *>(Qh + g * d.qs[1] + rw * d.qs[2] + c16 * 8);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = i0 + k * nthreads;
            if (i < rows_pad * 16)
                *reinterpret_cast<uint4 *>(q_gen + sw128_offset(rows_pad, i >> 4, i & 15)) = v[k];
        }
    }
}

// Barriers and TMEM of both sweeps, then the CTA synchronised so that every warp may use them.
// Returns the TMEM base address.
__device__ __forceinline__ uint32_t score_setup(const ScoreSmem &s, uint8_t *gen, const CUtensorMap *tmK,
                                                int stages, uint32_t tmem_cols, int tile_warps)
{
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(s.full0 + 8 * i, 1);
            mbar_init(s.empty0 + 8 * i, 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(s.tfull0 + 8 * i, 1);
            mbar_init(s.tempty0 + 8 * i, tile_warps);      // the epilogue warps that work on one tile
        }
        for (int i = 0; i < 8; ++i) mbar_init(s.xbar0 + 8 * i, tile_warps);
        mbar_fence_init();
        tma_prefetch_desc(tmK);
    }
    if ((threadIdx.x >> 5) == 1) {
        tmem_alloc(s.tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    return *reinterpret_cast<volatile uint32_t *>(gen + (s.tmem_slot - s.q));
}

// TMA producer (one thread): key tiles t0+i of (h, b), i in [i_begin, i_end), into the stage ring.
// The keys are an input of the call, so the producer never waits for the kernels before.
__device__ __forceinline__ bool score_produce(const ScoreSmem &s, const CUtensorMap *tmK, int stages,
                                              int t0, int i_begin, int i_end, int h, int b, long long lim)
{
    bool ok = true;
    int issued = i_begin;
    for (int i = i_begin; i < i_end; ++i) {
        const int st = i % stages, ph = (i / stages) & 1;
        if (!mbar_wait(s.empty0 + 8 * st, ph ^ 1, lim)) { ok = false; break; }
        const uint32_t dst = s.stage0 + st * kTileBytes;
        mbar_expect_tx(s.full0 + 8 * st, kTileBytes);
        tma_load_4d(dst, tmK, s.full0 + 8 * st, 0, (t0 + i) * kTileKeys, h, b);
        tma_load_4d(dst + kHalfBytes, tmK, s.full0 + 8 * st, 64, (t0 + i) * kTileKeys, h, b);
        ++issued;
    }
    if (!ok)        // gave up: let the copies already in flight land before the CTA exits
        for (int i = max(0, issued - stages); i < issued; ++i)
            mbar_wait(s.full0 + 8 * (i % stages), (i / stages) & 1, lim);
    return ok;
}

__device__ __forceinline__ void tile_range(int n_tiles, int chunks, int chunk, int *t0, int *t1)
{
    const int base = n_tiles / chunks, rem = n_tiles % chunks;
    *t0 = chunk * base + min(chunk, rem);
    *t1 = *t0 + base + (chunk < rem ? 1 : 0);
}

// One x32 slice of a row's accumulator: fold into the running (max, sum).
__device__ __forceinline__ void stats_fold(float (&v)[32], float scale, float &mx, float &z)
{
    float cm = fmaxf(v[0], v[1]);
#pragma unroll
    for (int i = 2; i < 32; i += 2) cm = fmaxf(cm, fmaxf(v[i], v[i + 1]));
    const float mn = fmaxf(mx, cm * scale);
    z *= ex2(mx - mn);
    mx = mn;
    const uint64_t nm = pack2(-mn, -mn);
    z += ex2_sum32(v, pack2(scale, scale), [&](int) { return make_ulonglong2(nm, nm); });
}

// (max, sum) of a row over the partials of all key chunks of a unit: kTpr consecutive threads of a
// warp share the row, thread `sub` of them takes chunks sub, sub + kTpr, ..., eight loads in flight,
// and the shares are combined with shuffles (every thread of the warp calls this).  Both score
// paths merge this way, so they agree to the bit.
template <int kTpr>
__device__ __forceinline__ float2 merge_row_partials(const float2 *pu, int chunks, int GW, int r, int sub)
{
    float mx = kNegBig, z = 0.f;
    if (r < GW) {
        for (int q0 = sub; q0 < chunks; q0 += 8 * kTpr) {
            float2 v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                v[k] = q0 + k * kTpr < chunks ? __ldcg(pu + (long long)(q0 + k * kTpr) * GW + r)
                                              : make_float2(kNegBig, 0.f);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float mn = fmaxf(mx, v[k].x);
                z = z * ex2(mx - mn) + v[k].y * ex2(v[k].x - mn);
                mx = mn;
            }
        }
    }
#pragma unroll
    for (int o = 1; o < kTpr; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, mx, o), z2 = __shfl_xor_sync(0xffffffffu, z, o);
        const float mn = fmaxf(mx, m2);
        z = z * ex2(mx - mn) + z2 * ex2(m2 - mn);
        mx = mn;
    }
    return make_float2(mx, z);
}

// kRowTiles = 1 (G*W <= 128) or 2 (G*W <= 256).  grid (chunks, units of the launch).
template <int kRowTiles>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_stats_tc(const __grid_constant__ CUtensorMap tmK, ScoreTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    PhaseClock pc(threadIdx.x == 64);
    pc.mark();
    constexpr int kRowsPad = 128 * kRowTiles;
    constexpr int kBufCols = 128 * kRowTiles;        // TMEM columns per accumulator buffer
    constexpr uint32_t kTmemCols = 512;
    // Every epilogue thread takes 64 accumulator columns of a tile.  With two row tiles the 16
    // warps share each tile (two buffers); with one, two groups of 8 warps take alternate tiles
    // (four buffers), so that a round of waiting, loading and releasing covers as much arithmetic.
    constexpr int kBufs = 512 / kBufCols, kGroups = 2 / kRowTiles;
    const Dims &d = a.d;
    const long long lim = a.wait_cycles;
    uint8_t *gen;
    const ScoreSmem s = score_smem_layout(smem_raw, kRowsPad, a.stages, &gen);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    int t0, t1;
    tile_range(a.n_tiles, a.chunks, chunk, &t0, &t1);
    const int n_local = t1 - t0;

    constexpr int kParts = 4 / kRowTiles;            // partial statistics per row
    float2 *cta_part = reinterpret_cast<float2 *>(gen + (s.misc - s.q));      // [kParts][kRowsPad]
    int *s_flag = reinterpret_cast<int *>(gen + (s.tmem_slot - s.q)) + 2;
    const int n_ahead = min(n_local, a.stages);

    const uint32_t tmem_base = score_setup(s, gen, &tmK, a.stages, kTmemCols, kEpiWarps / kGroups);
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = score_produce(s, &tmK, a.stages, t0, 0, n_ahead, h, b, lim);
    } else {
        stage_q(gen, kRowsPad, d, a.Q, b, h, threadIdx.x - 32, kScoreThreads - 32);
        fence_proxy_async();
    }
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pc.mark();
    pdl_launch_dependents();
    __syncthreads();
    pc.mark();

    if (warp == 0) {
        if (lane == 0 && ok) ok = score_produce(s, &tmK, a.stages, t0, n_ahead, n_local, h, b, lim);
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, 128);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                const int buf = i % kBufs, bph = (i / kBufs) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1, lim)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, ph, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t kt = s.stage0 + st * kTileBytes;
#pragma unroll
                for (int rt = 0; rt < kRowTiles; ++rt) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
                        const uint32_t qoff = (k >> 2) * (kRowsPad * 128) + rt * (128 * 128) + (k & 3) * 32;
                        umma_bf16(tmem_base + buf * kBufCols + rt * 128, umma_desc_sw128(s.q + qoff),
                                  umma_desc_sw128(kt + koff), idesc, k > 0);
                    }
                }
                umma_commit(s.empty0 + 8 * st);
                if (!(a.withhold_commit == 1 && i == 0)) umma_commit(s.tfull0 + 8 * buf);
            }
        }
    } else {
        // epilogue: thread = query row (TMEM lane); the four warp sets split the accumulator's
        // columns (row tile, then keys).
        constexpr int kSetCols = 64;
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int grp = set / (4 / kGroups);               // tiles grp, grp + kGroups, ...
        const int row = quad * 32 + lane;
        const int col0 = (set % (4 / kGroups)) * kSetCols, rt = col0 >> 7, key_off = col0 & 127;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        float mx = kNegBig, z = 0.f;
        const int r = rt * 128 + row;
        const int lim = d.N + (r < d.GW ? r % d.W : 0);      // last visible key of the row
        // A thread copies its columns to registers and hands the TMEM buffer back before the
        // arithmetic, so the next MMA never waits for exponentials.
        bool alive = true;
        for (int i = grp; i < n_local && alive; i += kGroups) {
            const int buf = i % kBufs, bph = (i / kBufs) & 1;
            alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, bph, lim));
            if (!alive) break;
            tc_fence_after();
            uint32_t raw[kSetCols / 32][32];
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kBufCols + col0;
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) tmem_ld32_issue(t_row + c * 32, raw[c]);
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) tmem_ld_fence(raw[c]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
            const int key0 = (t0 + i) * kTileKeys + key_off;
            const bool masked = key0 + kSetCols - 1 > d.N;      // window keys or the tail past L
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) {
                float v[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(raw[c][e]);
                if (masked) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (key0 + c * 32 + e > lim) v[e] = -INFINITY;
                }
                stats_fold(v, scale, mx, z);
            }
        }
        ok = alive;
        pc.mark();
        // partial p of row r: the sets (of every group) that hold columns of the row's tile
        cta_part[(kRowTiles == 1 ? set : set & 1) * kRowsPad + r] = make_float2(mx, z);
    }
    if (!ok && a.status) atomicExch(a.status, (int)GRAPHKV_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // this CTA's statistics of each row; the last CTA of the unit to get here merges all chunks
    // into the unit's row constants c_r
    for (int r = threadIdx.x; r < d.GW; r += kScoreThreads) {
        float2 p[kParts];
        float mx = kNegBig;
#pragma unroll
        for (int k = 0; k < kParts; ++k) {
            p[k] = cta_part[k * kRowsPad + r];
            mx = fmaxf(mx, p[k].x);
        }
        float z = 0.f;
#pragma unroll
        for (int k = 0; k < kParts; ++k) z += p[k].y * ex2(p[k].x - mx);
        reinterpret_cast<float2 *>(a.part)[((long long)unit * a.stats_chunks + chunk) * d.GW + r] =
            make_float2(mx, z);
    }
    pc.mark();
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *s_flag = atomicAdd(a.arrivals + unit, 1) == a.chunks - 1;
    __syncthreads();
    if (*s_flag) {
        __threadfence();
        const float2 *pu = reinterpret_cast<const float2 *>(a.part) + (long long)unit * a.stats_chunks * d.GW;
        constexpr int kTpr = 4 / kRowTiles;
        if (threadIdx.x < kRowsPad * kTpr) {
            const int r = threadIdx.x / kTpr, sub = threadIdx.x % kTpr;
            const float2 mz = merge_row_partials<kTpr>(pu, a.chunks, d.GW, r, sub);
            if (sub == 0 && r < d.GW) a.row_c[(long long)unit * d.GW + r] = mz.x + log2f(mz.y);
        }
        if (threadIdx.x == 0) a.arrivals[unit] = 0;      // ready for the next launch
    }
    pc.mark();
    pc.flush(0);
}

// kColTiles = 1 (G*W <= 128) or 2 (G*W <= 256).  grid (chunks, units of the launch).
template <int kColTiles>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_emit_tc(const __grid_constant__ CUtensorMap tmK, ScoreTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    PhaseClock pc(threadIdx.x == 64);
    pc.mark();
    constexpr int kRowsPad = 128 * kColTiles;        // rows of the Q operand (UMMA N)
    constexpr int kBufCols = 128 * kColTiles;
    constexpr uint32_t kTmemCols = 512;
    // Every epilogue thread takes up to 64 accumulator columns of a tile.  With two column tiles
    // the 16 warps share each tile (two buffers); with one, two groups of 8 warps take alternate
    // tiles (four buffers), so that a round of waiting, loading and releasing covers as much
    // arithmetic.
    constexpr int kBufs = 512 / kBufCols, kGroups = 2 / kColTiles, kSets = 4 / kGroups;
    constexpr int kXchg = 16 / kSets;                // exchange buffers in rotation
    const Dims &d = a.d;
    const long long lim = a.wait_cycles;
    uint8_t *gen;
    const ScoreSmem s = score_smem_layout(smem_raw, kRowsPad, a.stages, &gen);
    float *row_c = reinterpret_cast<float *>(gen + (s.misc - s.q));      // [kRowsPad]
    float *xchg = row_c + 256;                                          // [kXchg tiles][kSets][128]
    uint32_t *mass_hist = reinterpret_cast<uint32_t *>(gen + (s.misc - s.q) + kScratchBytes);   // [kMassBins]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    int t0, t1;
    tile_range(a.n_tiles, a.chunks, chunk, &t0, &t1);
    const int n_local = t1 - t0;
    const int n_cols = (d.GW + 31) & ~31;            // UMMA N: every x32 slice read below is written

    const int n_ahead = min(n_local, a.stages);
    const uint32_t tmem_base = score_setup(s, gen, &tmK, a.stages, kTmemCols, kEpiWarps / kGroups);
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = score_produce(s, &tmK, a.stages, t0, 0, n_ahead, h, b, lim);
    } else {
        stage_q(gen, kRowsPad, d, a.Q, b, h, threadIdx.x - 32, kScoreThreads - 32);
        fence_proxy_async();
    }
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pc.mark();
    pdl_launch_dependents();
    const bool want_hist = a.a_hist != nullptr || a.local_hist;
    if (want_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads) mass_hist[i] = 0u;
    if (a.zero) {
        // this CTA's share of the unit's words to clear
        const int per_cta = ceil_div(a.zero_words, a.chunks);
        for (int i = chunk * per_cta + threadIdx.x; i < min((chunk + 1) * per_cta, a.zero_words); i += kScoreThreads)
            a.zero[(long long)unit * a.zero_words + i] = 0u;
    }
    // -c_r of the unit's rows; padding rows contribute 2^-inf = 0
    for (int r = threadIdx.x; r < kRowsPad; r += kScoreThreads)
        row_c[r] = r < d.GW ? -__ldcg(a.row_c + (long long)unit * d.GW + r) : -INFINITY;
    __syncthreads();
    pc.mark();

    if (warp == 0) {
        if (lane == 0 && ok) ok = score_produce(s, &tmK, a.stages, t0, n_ahead, n_local, h, b, lim);
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, n_cols);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                const int buf = i % kBufs, bph = (i / kBufs) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1, lim)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, ph, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t kt = s.stage0 + st * kTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
                    const uint32_t qoff = (k >> 2) * (kRowsPad * 128) + (k & 3) * 32;
                    umma_bf16(tmem_base + buf * kBufCols, umma_desc_sw128(kt + koff),
                              umma_desc_sw128(s.q + qoff), idesc, k > 0);
                }
                umma_commit(s.empty0 + 8 * st);
                umma_commit(s.tfull0 + 8 * buf);
            }
        }
    } else {
        // epilogue: thread = key (TMEM lane); the warp sets of a tile split the query rows (x32
        // column slices, at most two each).
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int grp = set / kSets, part = set % kSets;       // tiles grp, grp + kGroups, ...
        const int key_lane = quad * 32 + lane;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        const uint64_t scale2 = pack2(scale, scale);
        const int n_slices = (d.GW + 31) >> 5;                 // x32 column slices in use (<= 8)
        const int s_begin = (part * n_slices) / kSets, s_end = ((part + 1) * n_slices) / kSets;
        float *a_row = a.a_out + (long long)unit * d.N;
        // A thread copies its slices to registers and hands the TMEM buffer back before the
        // arithmetic, so the next MMA never waits for exponentials.
        const uint32_t t_set = tmem_base + ((uint32_t)(quad * 32) << 16) + s_begin * 32;
        bool alive = true;
        auto sum_slice = [&](const uint32_t (&reg)[32], int sl) {
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(reg[e]);
            const ulonglong2 *c4 = reinterpret_cast<const ulonglong2 *>(row_c + sl * 32);
            return ex2_sum32(v, scale2, [&](int q) { return c4[q]; });
        };
        for (int i = grp; i < n_local && alive; i += kGroups) {
            const int buf = i % kBufs;
            alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, (i / kBufs) & 1, lim));
            if (!alive) break;
            tc_fence_after();
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
            };
            float acc = 0.f;
            if (s_end - s_begin == 2) {
                uint32_t ra[32], rb[32];
                tmem_ld32_issue(t_set + buf * kBufCols, ra);
                tmem_ld32_issue(t_set + buf * kBufCols + 32, rb);
                tmem_ld_fence(ra);
                tmem_ld_fence(rb);
                release();
                acc = sum_slice(ra, s_begin) + sum_slice(rb, s_begin + 1);
            } else if (s_end - s_begin == 1) {
                uint32_t ra[32];
                tmem_ld32_issue(t_set + buf * kBufCols, ra);
                tmem_ld_fence(ra);
                release();
                acc = sum_slice(ra, s_begin);
            } else {
                release();
            }
            // The sets of the tile hold the parts of each key's row sum.  Each leaves its part in
            // the exchange buffer of the tile (kXchg in rotation: a buffer comes round again only
            // after every warp has left the tile that used it) and arrives on that buffer's
            // barrier; the sets take turns waiting for all parts, adding them up and storing the
            // result, so no set waits for another except on its own turn.
            const int xb = i % kXchg;
            xchg[(xb * kSets + part) * 128 + key_lane] = acc;
            __syncwarp();
            if (lane == 0) mbar_arrive(s.xbar0 + 8 * xb);
            if (part != (i / kGroups) % kSets) continue;
            alive = __all_sync(0xffffffffu, mbar_wait(s.xbar0 + 8 * xb, (i / kXchg) & 1, lim));
            const int j = (t0 + i) * kTileKeys + key_lane;
            if (alive && j < d.N) {
                const float *x = xchg + xb * kSets * 128 + key_lane;
                const float aj = kSets == 4 ? (x[0] + x[128]) + (x[256] + x[384]) : x[0] + x[128];
                a_row[j] = aj;
                if (want_hist) atomicAdd(&mass_hist[float_to_key(aj) >> 21], 1u);
            }
        }
        ok = alive;
        pc.mark();
    }
    if (!ok && a.status) atomicExch(a.status, (int)GRAPHKV_ERR_TIMEOUT);
    tc_fence_before();
    const bool all_ok = __syncthreads_and(ok ? 1 : 0) != 0;
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // this CTA's share of the unit's mass histogram (pooling and source selection start from it)
    if (a.a_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads)
            if (mass_hist[i]) atomicAdd(a.a_hist + (long long)unit * kMassBins + i, mass_hist[i]);
    pc.mark();
    // Eq. 2, first half: this chunk's candidates for the unit's source nodes (the stage ring is idle
    // by now and serves as scratch); the similarity sweep merges the lists
    if (a.src.k > 0 && all_ok)
        source_list_chunk(a.src, d, unit, chunk, t0 * kTileKeys, min(t1 * kTileKeys, d.N),
                          a.a_out + (long long)unit * d.N, mass_hist, gen + (s.stage0 - s.q));
    pc.mark();
    pc.flush(1);
}


// Both sweeps in one kernel, for launches whose CTAs are all resident at once (one CTA per SM and
// no more CTAs than SMs; launched cooperatively, so the device starts the grid as a whole): a CTA runs the statistics pass over its key chunk, leaves its partial
// row statistics, announces itself on the unit's counter, waits (bounded, like every wait here)
// until all chunks of the unit have done so, merges the partials into the row constants itself
// and runs the emit pass over the same chunk in reverse tile order, so that the tiles the first
// pass left in the stage ring are used again without a copy.  Against two launches this saves a
// kernel boundary, the second set-up (barriers, tensor memory, the staging of the queries) and
// the re-read of the ring's tiles.  kTiles = 1 (G*W <= 128) or 2 (G*W <= 256); grid (chunks,
// units of the launch); a.arrivals holds one 64-bit word per unit (the call's tag and the count of
// arrived CTAs), whatever its content before the launch.
template <int kTiles>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_fused_tc(const __grid_constant__ CUtensorMap tmK, ScoreTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    PhaseClock pc(threadIdx.x == 64);
    pc.mark();
    constexpr int kRowsPad = 128 * kTiles;
    constexpr int kBufCols = 128 * kTiles;
    constexpr uint32_t kTmemCols = 512;
    constexpr int kBufs = 512 / kBufCols, kGroups = 2 / kTiles, kSets = 4 / kGroups;
    constexpr int kXchg = 16 / kSets;
    constexpr int kParts = 4 / kTiles;               // partial statistics per row within the CTA
    const Dims &d = a.d;
    const long long lim = a.wait_cycles;
    uint8_t *gen;
    const ScoreSmem s = score_smem_layout(smem_raw, kRowsPad, a.stages, &gen);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    const int S = a.stages;
    int t0, t1;
    tile_range(a.n_tiles, a.chunks, chunk, &t0, &t1);
    const int n_local = t1 - t0;                                          // tiles of the statistics pass
    const int n_emit = max(0, min(t1, ceil_div(d.N, kTileKeys)) - t0);    // of them, tiles with prefix keys
    const int n_cols = (d.GW + 31) & ~31;            // UMMA N of the emit pass

    // scratch: first the CTA's partial statistics, after the hand-over the row constants and the
    // exchange buffers of the emit pass
    float2 *cta_part = reinterpret_cast<float2 *>(gen + (s.misc - s.q));      // [kParts][kRowsPad]
    float *row_c = reinterpret_cast<float *>(gen + (s.misc - s.q));           // [kRowsPad]
    float *xchg = row_c + 256;                                                // [kXchg tiles][kSets][128]
    uint32_t *mass_hist = reinterpret_cast<uint32_t *>(gen + (s.misc - s.q) + kScratchBytes);   // [kMassBins]
    int *s_flag = reinterpret_cast<int *>(gen + (s.tmem_slot - s.q)) + 2;
    const int n_ahead = min(n_local, S);

    const uint32_t tmem_base = score_setup(s, gen, &tmK, S, kTmemCols, kEpiWarps / kGroups);
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = score_produce(s, &tmK, S, t0, 0, n_ahead, h, b, lim);
    } else {
        stage_q(gen, kRowsPad, d, a.Q, b, h, threadIdx.x - 32, kScoreThreads - 32);
        fence_proxy_async();
    }
    pc.mark();
    if (a.wait_prior) pdl_wait();
    pc.mark();
    pdl_launch_dependents();
    const bool want_hist = a.a_hist != nullptr || a.local_hist;
    if (want_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads) mass_hist[i] = 0u;
    if (a.clear_head) {
        // (after the wait: nothing of the call before still reads or writes these words; the unit's
        // histogram is added to only after the hand-over, which orders these stores before it)
        if (a.status && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *a.status = 0;
        if (a.a_hist) {
            const int per_cta = ceil_div(kMassBins, a.chunks);
            for (int i = chunk * per_cta + threadIdx.x; i < min((chunk + 1) * per_cta, kMassBins); i += kScoreThreads)
                a.a_hist[(long long)unit * kMassBins + i] = 0u;
        }
    }
    if (a.zero) {
        const int per_cta = ceil_div(a.zero_words, a.chunks);
        for (int i = chunk * per_cta + threadIdx.x; i < min((chunk + 1) * per_cta, a.zero_words); i += kScoreThreads)
            a.zero[(long long)unit * a.zero_words + i] = 0u;
    }
    __syncthreads();
    pc.mark();

    // ---- statistics pass: D = Q K^T, tiles 0 .. n_local-1 in order ----
    if (warp == 0) {
        if (lane == 0 && ok) ok = score_produce(s, &tmK, S, t0, n_ahead, n_local, h, b, lim);
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, 128);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % S, ph = (i / S) & 1;
                const int buf = i % kBufs, bph = (i / kBufs) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1, lim)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, ph, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t kt = s.stage0 + st * kTileBytes;
#pragma unroll
                for (int rt = 0; rt < kTiles; ++rt) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
                        const uint32_t qoff = (k >> 2) * (kRowsPad * 128) + rt * (128 * 128) + (k & 3) * 32;
                        umma_bf16(tmem_base + buf * kBufCols + rt * 128, umma_desc_sw128(s.q + qoff),
                                  umma_desc_sw128(kt + koff), idesc, k > 0);
                    }
                }
                umma_commit(s.empty0 + 8 * st);
                if (!(a.withhold_commit == 1 && i == 0)) umma_commit(s.tfull0 + 8 * buf);
            }
        }
    } else {
        constexpr int kSetCols = 64;
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int grp = set / (4 / kGroups);
        const int row = quad * 32 + lane;
        const int col0 = (set % (4 / kGroups)) * kSetCols, rt = col0 >> 7, key_off = col0 & 127;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        float mx = kNegBig, z = 0.f;
        const int r = rt * 128 + row;
        const int last = d.N + (r < d.GW ? r % d.W : 0);      // last visible key of the row
        bool alive = true;
        for (int i = grp; i < n_local && alive; i += kGroups) {
            const int buf = i % kBufs, bph = (i / kBufs) & 1;
            alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, bph, lim));
            if (!alive) break;
            tc_fence_after();
            uint32_t raw[kSetCols / 32][32];
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kBufCols + col0;
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) tmem_ld32_issue(t_row + c * 32, raw[c]);
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) tmem_ld_fence(raw[c]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
            const int key0 = (t0 + i) * kTileKeys + key_off;
            const bool masked = key0 + kSetCols - 1 > d.N;      // window keys or the tail past L
#pragma unroll
            for (int c = 0; c < kSetCols / 32; ++c) {
                float v[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(raw[c][e]);
                if (masked) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (key0 + c * 32 + e > last) v[e] = -INFINITY;
                }
                stats_fold(v, scale, mx, z);
            }
        }
        ok = alive;
        cta_part[(kTiles == 1 ? set : set & 1) * kRowsPad + r] = make_float2(mx, z);
    }
    pc.mark();

    // ---- hand-over: partials out, every chunk of the unit in, row constants ----
    tc_fence_before();
    bool all_ok = __syncthreads_and(ok ? 1 : 0) != 0;
    unsigned long long *arrived = reinterpret_cast<unsigned long long *>(a.arrivals) + unit;
    unsigned long long seen_early = 0ull;
    if (threadIdx.x == 0)
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(seen_early) : "l"(arrived) : "memory");
    for (int r = threadIdx.x; r < d.GW; r += kScoreThreads) {
        float2 p[kParts];
        float mx = kNegBig;
#pragma unroll
        for (int k = 0; k < kParts; ++k) {
            p[k] = cta_part[k * kRowsPad + r];
            mx = fmaxf(mx, p[k].x);
        }
        float z = 0.f;
#pragma unroll
        for (int k = 0; k < kParts; ++k) z += p[k].y * ex2(p[k].x - mx);
        reinterpret_cast<float2 *>(a.part)[((long long)unit * a.stats_chunks + chunk) * d.GW + r] =
            make_float2(mx, z);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        // The unit's arrival word holds (call tag, count).  A CTA that finds another tag there starts
        // the count for this call (one compare-and-swap, by the unit's first arrivals only), so
        // whatever the word held before (zeros, an earlier call's count, the count of a call that
        // gave up, memory nobody cleared) never counts and nothing has to be reset; with the call's
        // tag in place an arrival is a plain addition.  The word was looked at ahead of the fence
        // (`seen_early`): its tag can only have turned into this call's since.  A CTA whose pass
        // failed still arrives, so that the others do not wait in vain.
        const unsigned long long tag = (unsigned long long)a.call_tag << 32;
        if (a.withhold_commit != 2) {
            unsigned long long cur = seen_early;
            while (true) {
                if ((cur >> 32) == a.call_tag) {
                    atomicAdd(arrived, 1ull);
                    break;
                }
                const unsigned long long prev = atomicCAS(arrived, cur, tag | 1ull);
                if (prev == cur) break;
                cur = prev;
            }
        }
        bool in = false;
        const long long c0 = clock64();
        while (true) {
            unsigned long long seen;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(arrived) : "memory");
            if ((seen >> 32) == a.call_tag && (uint32_t)seen >= (uint32_t)a.chunks) { in = true; break; }
            if (clock64() - c0 > lim) break;
            __nanosleep(20);
        }
        *s_flag = in ? 1 : 0;
    }
    __syncthreads();
    pc.mark();
    if (!*s_flag) { ok = false; all_ok = false; }
    if (all_ok) {
        // every CTA merges the unit's partials itself: kTpr threads per row take the chunks in turn
        constexpr int kTpr = 4 / kTiles;
        const float2 *pu = reinterpret_cast<const float2 *>(a.part) + (long long)unit * a.stats_chunks * d.GW;
        static_assert(kRowsPad * kTpr <= (kScoreThreads & ~31), "whole warps take the rows");
        if (threadIdx.x < kRowsPad * kTpr) {
            const int r = threadIdx.x / kTpr, sub = threadIdx.x % kTpr;
            const float2 mz = merge_row_partials<kTpr>(pu, a.chunks, d.GW, r, sub);
            // -c_r of the unit's rows; padding rows contribute 2^-inf = 0
            if (sub == 0) row_c[r] = r < d.GW ? -(mz.x + log2f(mz.y)) : -INFINITY;
        }
    }
    __syncthreads();
    pc.mark();

    // ---- emit pass: D = K Q^T, the chunk's prefix tiles in reverse order ----
    // Tile tl sits in ring slot tl % S in both passes; uses(st) counts the fills of slot st by the
    // first pass, so the u-th use of a slot keeps the parities of its barriers in step.
    auto slot_use = [&](int tl, int k) { return (n_local - (tl % S) + S - 1) / S + k / S; };
    if (!all_ok) {
        // nothing more to do: a wait ran out somewhere
    } else if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int k = 0; k < n_emit; ++k) {
                const int tl = n_emit - 1 - k, st = tl % S, u = slot_use(tl, k);
                if (!mbar_wait(s.empty0 + 8 * st, (u & 1) ^ 1, lim)) { ok = false; break; }
                if (tl + S >= n_local) {
                    mbar_arrive(s.full0 + 8 * st);            // still there from the first pass
                } else {
                    const uint32_t dst = s.stage0 + st * kTileBytes;
                    mbar_expect_tx(s.full0 + 8 * st, kTileBytes);
                    tma_load_4d(dst, &tmK, s.full0 + 8 * st, 0, (t0 + tl) * kTileKeys, h, b);
                    tma_load_4d(dst + kHalfBytes, &tmK, s.full0 + 8 * st, 64, (t0 + tl) * kTileKeys, h, b);
                }
                ++issued;
            }
            if (!ok)        // gave up: let the copies already in flight land before the CTA exits
                for (int k = max(0, issued - S); k < issued; ++k) {
                    const int tl = n_emit - 1 - k;
                    mbar_wait(s.full0 + 8 * (tl % S), slot_use(tl, k) & 1, lim);
                }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, n_cols);
            for (int k = 0; k < n_emit; ++k) {
                const int tl = n_emit - 1 - k, st = tl % S, u = slot_use(tl, k);
                const int i = n_local + k;                        // accumulator buffers keep rotating
                const int buf = i % kBufs, bph = (i / kBufs) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1, lim)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, u & 1, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t kt = s.stage0 + st * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t koff = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    const uint32_t qoff = (kk >> 2) * (kRowsPad * 128) + (kk & 3) * 32;
                    umma_bf16(tmem_base + buf * kBufCols, umma_desc_sw128(kt + koff),
                              umma_desc_sw128(s.q + qoff), idesc, kk > 0);
                }
                umma_commit(s.empty0 + 8 * st);
                umma_commit(s.tfull0 + 8 * buf);
            }
        }
    } else {
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int grp = set / kSets, part = set % kSets;
        const int key_lane = quad * 32 + lane;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        const uint64_t scale2 = pack2(scale, scale);
        const int n_slices = (d.GW + 31) >> 5;
        const int s_begin = (part * n_slices) / kSets, s_end = ((part + 1) * n_slices) / kSets;
        float *a_row = a.a_out + (long long)unit * d.N;
        const uint32_t t_set = tmem_base + ((uint32_t)(quad * 32) << 16) + s_begin * 32;
        bool alive = true;
        auto sum_slice = [&](const uint32_t (&reg)[32], int sl) {
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(reg[e]);
            const ulonglong2 *c4 = reinterpret_cast<const ulonglong2 *>(row_c + sl * 32);
            return ex2_sum32(v, scale2, [&](int q) { return c4[q]; });
        };
        for (int k = grp; k < n_emit && alive; k += kGroups) {
            const int i = n_local + k, buf = i % kBufs;
            alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, (i / kBufs) & 1, lim));
            if (!alive) break;
            tc_fence_after();
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
            };
            float acc = 0.f;
            if (s_end - s_begin == 2) {
                uint32_t ra[32], rb[32];
                tmem_ld32_issue(t_set + buf * kBufCols, ra);
                tmem_ld32_issue(t_set + buf * kBufCols + 32, rb);
                tmem_ld_fence(ra);
                tmem_ld_fence(rb);
                release();
                acc = sum_slice(ra, s_begin) + sum_slice(rb, s_begin + 1);
            } else if (s_end - s_begin == 1) {
                uint32_t ra[32];
                tmem_ld32_issue(t_set + buf * kBufCols, ra);
                tmem_ld_fence(ra);
                release();
                acc = sum_slice(ra, s_begin);
            } else {
                release();
            }
            // the sets of the tile exchange the parts of each key's row sum (see score_emit_tc)
            const int xb = k % kXchg;
            xchg[(xb * kSets + part) * 128 + key_lane] = acc;
            __syncwarp();
            if (lane == 0) mbar_arrive(s.xbar0 + 8 * xb);
            if (part != (k / kGroups) % kSets) continue;
            alive = __all_sync(0xffffffffu, mbar_wait(s.xbar0 + 8 * xb, (k / kXchg) & 1, lim));
            const int j = (t0 + n_emit - 1 - k) * kTileKeys + key_lane;
            if (alive && j < d.N) {
                const float *x = xchg + xb * kSets * 128 + key_lane;
                const float aj = kSets == 4 ? (x[0] + x[128]) + (x[256] + x[384]) : x[0] + x[128];
                a_row[j] = aj;
                if (want_hist) atomicAdd(&mass_hist[float_to_key(aj) >> 21], 1u);
            }
        }
        ok = alive;
    }
    pc.mark();
    if (!ok && a.status) atomicExch(a.status, (int)GRAPHKV_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (a.a_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads)
            if (mass_hist[i]) atomicAdd(a.a_hist + (long long)unit * kMassBins + i, mass_hist[i]);
    pc.mark();
    pc.flush(5);
}

}  // namespace tc
}  // namespace graphkv
