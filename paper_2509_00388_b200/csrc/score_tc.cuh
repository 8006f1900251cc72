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
// MUFU unit, not HBM, is the ceiling of both sweeps.  Warp roles (320 threads): warp 0 = TMA
// producer (it starts on the key tiles before the dependency wait: keys are an input of the
// call), warp 1 = MMA issuer and TMEM owner, warps 2..9 = epilogue (two sets of four warps
// covering the four TMEM lane quadrants; the sets split the accumulator columns).
#pragma once

#include "tc_common.cuh"

namespace graphkv {
namespace tc {

constexpr int kScoreThreads = 320;
constexpr int kMassBins = 2048;         // histogram of the attention mass: top 11 bits of float_to_key
constexpr int kEpiWarps = 8;

struct ScoreTcArgs {
    Dims d;
    const __nv_bfloat16 *Q;
    float *part;        // [units][stats_chunks][GW][2] row statistics (max, sum) per key chunk
    float *row_c;       // [units][GW] c_r = max_r + log2(Z_r), written by the last stats CTA of a unit
    int *arrivals;      // [units] stats CTAs done per unit (zero before the launch; reset on the way)
    float *a_out;       // [units][N] attention mass before pooling
    uint32_t *a_hist;   // optional [units][kMassBins]: counts of a by the top bits of its ordered image
    int *status;        // workspace status word
    int unit0;          // first unit of this launch
    int chunks;         // key chunks (CTAs) per unit
    int n_tiles;        // 128-key tiles per unit in this sweep
    int stats_chunks;   // key chunks of the statistics sweep (partials per row)
    int stages;         // shared-memory K tiles in flight
    int wait_prior;     // launched with programmatic stream serialization: wait for the kernels before
};

struct ScoreSmem {
    uint32_t q, stage0, full0, empty0, tfull0, tempty0, tmem_slot, misc;
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
    s.tempty0 = s.tfull0 + 2 * 8;
    s.tmem_slot = s.tempty0 + 2 * 8;
    s.misc = s.tmem_slot + 16;
    return s;
}

__host__ __device__ inline size_t score_smem_bytes(int rows_pad, int stages)
{
    return 1024 + (size_t)rows_pad * 256 + (size_t)stages * kTileBytes + 8 * 8 * 2 + 2 * 8 * 2 + 16 +
           8192 + 8192 + 64;   // 8 KB: the CTA's row statistics / row constants and the exchange
                               // buffer; 8 KB: the emit sweep's histogram of the attention mass
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
                                                int stages, uint32_t tmem_cols)
{
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(s.full0 + 8 * i, 1);
            mbar_init(s.empty0 + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s.tfull0 + 8 * i, 1);
            mbar_init(s.tempty0 + 8 * i, 8);       // the eight epilogue warps
        }
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
                                              int t0, int i_begin, int i_end, int h, int b)
{
    bool ok = true;
    int issued = i_begin;
    for (int i = i_begin; i < i_end; ++i) {
        const int st = i % stages, ph = (i / stages) & 1;
        if (!mbar_wait(s.empty0 + 8 * st, ph ^ 1)) { ok = false; break; }
        const uint32_t dst = s.stage0 + st * kTileBytes;
        mbar_expect_tx(s.full0 + 8 * st, kTileBytes);
        tma_load_4d(dst, tmK, s.full0 + 8 * st, 0, (t0 + i) * kTileKeys, h, b);
        tma_load_4d(dst + kHalfBytes, tmK, s.full0 + 8 * st, 64, (t0 + i) * kTileKeys, h, b);
        ++issued;
    }
    if (!ok)        // gave up: let the copies already in flight land before the CTA exits
        for (int i = max(0, issued - stages); i < issued; ++i)
            mbar_wait(s.full0 + 8 * (i % stages), (i / stages) & 1);
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
    float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        z0 += ex2(fmaf(v[i], scale, -mn));
        z1 += ex2(fmaf(v[i + 1], scale, -mn));
        z2 += ex2(fmaf(v[i + 2], scale, -mn));
        z3 += ex2_poly3(fmaf(v[i + 3], scale, -mn));      // one exponential in four off the MUFU unit
    }
    z += (z0 + z1) + (z2 + z3);
}

// kRowTiles = 1 (G*W <= 128) or 2 (G*W <= 256).  grid (chunks, units of the launch).
template <int kRowTiles>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_stats_tc(const __grid_constant__ CUtensorMap tmK, ScoreTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kRowsPad = 128 * kRowTiles;
    constexpr int kBufCols = 128 * kRowTiles;        // TMEM columns per accumulator buffer
    constexpr uint32_t kTmemCols = 2 * kBufCols;
    const Dims &d = a.d;
    uint8_t *gen;
    const ScoreSmem s = score_smem_layout(smem_raw, kRowsPad, a.stages, &gen);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    int t0, t1;
    tile_range(a.n_tiles, a.chunks, chunk, &t0, &t1);
    const int n_local = t1 - t0;

    float2 *cta_part = reinterpret_cast<float2 *>(gen + (s.misc - s.q));      // [2][kRowsPad]
    int *s_flag = reinterpret_cast<int *>(gen + (s.tmem_slot - s.q)) + 2;
    const int n_ahead = min(n_local, a.stages);

    const uint32_t tmem_base = score_setup(s, gen, &tmK, a.stages, kTmemCols);
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = score_produce(s, &tmK, a.stages, t0, 0, n_ahead, h, b);
    } else {
        stage_q(gen, kRowsPad, d, a.Q, b, h, threadIdx.x - 32, kScoreThreads - 32);
        fence_proxy_async();
    }
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    __syncthreads();

    if (warp == 0) {
        if (lane == 0 && ok) ok = score_produce(s, &tmK, a.stages, t0, n_ahead, n_local, h, b);
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, 128);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                const int buf = i & 1, bph = (i >> 1) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, ph)) { ok = false; break; }
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
                umma_commit(s.tfull0 + 8 * buf);
            }
        }
    } else {
        // epilogue: thread = query row (TMEM lane), warp set = half of the key columns
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int row = quad * 32 + lane;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        float mx[kRowTiles], z[kRowTiles];
        int lim[kRowTiles];                      // last visible key of the row
#pragma unroll
        for (int rt = 0; rt < kRowTiles; ++rt) {
            mx[rt] = kNegBig;
            z[rt] = 0.f;
            const int r = rt * 128 + row;
            lim[rt] = d.N + (r < d.GW ? r % d.W : 0);
        }
        bool alive = true;
        for (int i = 0; i < n_local && alive; ++i) {
            const int buf = i & 1, bph = (i >> 1) & 1;
            alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, bph));
            if (!alive) break;
            tc_fence_after();
            const int key0 = (t0 + i) * kTileKeys + set * 64;
            const bool masked = key0 + 63 > d.N;          // window keys or the tail past L
#pragma unroll
            for (int rt = 0; rt < kRowTiles; ++rt) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kBufCols + rt * 128 +
                                  set * 64 + c * 32, v);
                    if (masked) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (key0 + c * 32 + e > lim[rt]) v[e] = -INFINITY;
                    }
                    stats_fold(v, scale, mx[rt], z[rt]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
        }
        ok = alive;
#pragma unroll
        for (int rt = 0; rt < kRowTiles; ++rt) cta_part[set * kRowsPad + rt * 128 + row] = make_float2(mx[rt], z[rt]);
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
        const float2 p0 = cta_part[r], p1 = cta_part[kRowsPad + r];
        const float mx = fmaxf(p0.x, p1.x);
        reinterpret_cast<float2 *>(a.part)[((long long)unit * a.stats_chunks + chunk) * d.GW + r] =
            make_float2(mx, p0.y * ex2(p0.x - mx) + p1.y * ex2(p1.x - mx));
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *s_flag = atomicAdd(a.arrivals + unit, 1) == a.chunks - 1;
    __syncthreads();
    if (*s_flag) {
        __threadfence();
        const float2 *pu = reinterpret_cast<const float2 *>(a.part) + (long long)unit * a.stats_chunks * d.GW;
        for (int r = threadIdx.x; r < d.GW; r += kScoreThreads) {
            float mx = kNegBig, z = 0.f;
            for (int q0 = 0; q0 < a.chunks; q0 += 8) {       // eight loads in flight at a time
                float2 v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    v[k] = q0 + k < a.chunks ? __ldcg(pu + (long long)(q0 + k) * d.GW + r)
                                             : make_float2(kNegBig, 0.f);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float mn = fmaxf(mx, v[k].x);
                    z = z * ex2(mx - mn) + v[k].y * ex2(v[k].x - mn);
                    mx = mn;
                }
            }
            a.row_c[(long long)unit * d.GW + r] = mx + log2f(z);
        }
        if (threadIdx.x == 0) a.arrivals[unit] = 0;      // ready for the next launch
    }
}

// kColTiles = 1 (G*W <= 128) or 2 (G*W <= 256).  grid (chunks, units of the launch).
template <int kColTiles>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_emit_tc(const __grid_constant__ CUtensorMap tmK, ScoreTcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kRowsPad = 128 * kColTiles;        // rows of the Q operand (UMMA N)
    constexpr int kBufCols = 128 * kColTiles;
    constexpr uint32_t kTmemCols = 2 * kBufCols;
    const Dims &d = a.d;
    uint8_t *gen;
    const ScoreSmem s = score_smem_layout(smem_raw, kRowsPad, a.stages, &gen);
    float *row_c = reinterpret_cast<float *>(gen + (s.misc - s.q));      // [kRowsPad]
    float *xchg = row_c + kRowsPad;                                     // [2][128]
    uint32_t *mass_hist = reinterpret_cast<uint32_t *>(gen + (s.misc - s.q) + 8192);   // [kMassBins]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = a.unit0 + blockIdx.y, b = unit / d.hkv, h = unit % d.hkv;
    const int chunk = blockIdx.x;
    int t0, t1;
    tile_range(a.n_tiles, a.chunks, chunk, &t0, &t1);
    const int n_local = t1 - t0;
    const int n_cols = (d.GW + 31) & ~31;            // UMMA N: every x32 slice read below is written

    const int n_ahead = min(n_local, a.stages);
    const uint32_t tmem_base = score_setup(s, gen, &tmK, a.stages, kTmemCols);
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = score_produce(s, &tmK, a.stages, t0, 0, n_ahead, h, b);
    } else {
        stage_q(gen, kRowsPad, d, a.Q, b, h, threadIdx.x - 32, kScoreThreads - 32);
        fence_proxy_async();
    }
    if (a.wait_prior) pdl_wait();
    pdl_launch_dependents();
    if (a.a_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads) mass_hist[i] = 0u;
    // c_r of the unit's rows; padding rows contribute 2^-inf = 0
    for (int r = threadIdx.x; r < kRowsPad; r += kScoreThreads)
        row_c[r] = r < d.GW ? __ldcg(a.row_c + (long long)unit * d.GW + r) : INFINITY;
    __syncthreads();

    if (warp == 0) {
        if (lane == 0 && ok) ok = score_produce(s, &tmK, a.stages, t0, n_ahead, n_local, h, b);
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, n_cols);
            for (int i = 0; i < n_local; ++i) {
                const int st = i % a.stages, ph = (i / a.stages) & 1;
                const int buf = i & 1, bph = (i >> 1) & 1;
                if (!mbar_wait(s.tempty0 + 8 * buf, bph ^ 1)) { ok = false; break; }
                if (!mbar_wait(s.full0 + 8 * st, ph)) { ok = false; break; }
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
        // epilogue: thread = key (TMEM lane), warp set = half of the query rows
        const int quad = warp & 3, set = (warp - 2) >> 2;
        const int key_lane = quad * 32 + lane;
        const float scale = rsqrtf((float)kHeadDim) * kLog2e;
        const int n_slices = (d.GW + 31) >> 5;                 // x32 column slices in use
        const int s_begin = set == 0 ? 0 : (n_slices + 1) >> 1;
        const int s_end = set == 0 ? (n_slices + 1) >> 1 : n_slices;
        float *a_row = a.a_out + (long long)unit * d.N;
        bool alive = true;
        for (int i = 0; i < n_local; ++i) {
            const int buf = i & 1, bph = (i >> 1) & 1;
            float acc = 0.f;
            if (alive) alive = __all_sync(0xffffffffu, mbar_wait(s.tfull0 + 8 * buf, bph));
            if (alive) {
                tc_fence_after();
                for (int sl = s_begin; sl < s_end; ++sl) {
                    float v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kBufCols + sl * 32, v);
                    const float4 *c4 = reinterpret_cast<const float4 *>(row_c + sl * 32);
                    float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float4 c = c4[e];
                        p0 += ex2(fmaf(v[4 * e], scale, -c.x));
                        p1 += ex2(fmaf(v[4 * e + 1], scale, -c.y));
                        p2 += ex2(fmaf(v[4 * e + 2], scale, -c.z));
                        p3 += ex2_poly3(fmaf(v[4 * e + 3], scale, -c.w));
                    }
                    acc += (p0 + p1) + (p2 + p3);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s.tempty0 + 8 * buf);
            }
            // the two sets hold the two halves of each key's row sum
            if (set == 1) xchg[buf * 128 + key_lane] = acc;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (set == 0 && alive) {
                const int j = (t0 + i) * kTileKeys + key_lane;
                if (j < d.N) {
                    const float aj = acc + xchg[buf * 128 + key_lane];
                    a_row[j] = aj;
                    if (a.a_hist) atomicAdd(&mass_hist[float_to_key(aj) >> 21], 1u);
                }
            }
        }
        ok = alive;
    }
    if (!ok && a.status) atomicExch(a.status, (int)GRAPHKV_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // this CTA's share of the unit's mass histogram (pooling and source selection start from it)
    if (a.a_hist)
        for (int i = threadIdx.x; i < kMassBins; i += kScoreThreads)
            if (mass_hist[i]) atomicAdd(a.a_hist + (long long)unit * kMassBins + i, mass_hist[i]);
}

}  // namespace tc
}  // namespace graphkv
