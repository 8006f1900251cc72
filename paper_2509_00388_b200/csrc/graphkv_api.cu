// C ABI of the GraphKV library: argument validation, workspace layout and kernel launches.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "cluster_select.cuh"
#include "common.cuh"
#include "decode_attn.cuh"
#include "gather.cuh"
#include "propagate_simt.cuh"
#include "score_simt.cuh"
#include "score_tc.cuh"
#include "select.cuh"
#include "sim_tc.cuh"

using namespace graphkv;

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kMaxSmem = 227 * 1024;      // dynamic shared memory a CTA may ask for
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Workspace carve-up; every region starts 256-byte aligned.
struct Layout {
    size_t status;      // int status word (256 bytes reserved)
    size_t arrivals;    // counters of score CTAs per unit [2 * units] (directly after the status word)
    size_t a_hist;      // histogram of the attention mass [units][2048] (directly after the counters)
    size_t row_c;       // softmax row constants [units][GW]
    size_t part;        // softmax row statistics per key chunk
    size_t a;           // attention mass before pooling [units][N]
    size_t s;           // scores when the caller gives no array [units][N]
    size_t src;         // source nodes [units][K_src]
    size_t sims;        // edges of the sources [units][K_src][N]
    size_t nbr_idx;     // neighbourhoods [units][K_src][m]
    size_t nbr_e;
    size_t cand;        // per-chunk neighbour candidates [units][K_src][sim_chunks][kCandCap]
    size_t cand_hist;   // [units][K_src][kCandBins]
    size_t src_cand;    // elements the emit sweep lists for the source selection [units][max_parts][kSrcCap]
    size_t src_cnt;     // [units][max_parts]
    size_t total;
    int n_stat_chunks;  // key chunks of the SIMT statistics sweep
    int max_parts;      // partial statistics per row the region can hold
};

graphkv_status resolve(const graphkv_params *p, Dims *d)
{
    if (!p) return GRAPHKV_ERR_INVALID_ARG;
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->window < 1 ||
        p->seq_len <= p->window || p->n_q_heads % p->n_kv_heads != 0)
        return GRAPHKV_ERR_INVALID_ARG;
    const int N = p->seq_len - p->window;
    if (p->budget < 1 || p->budget > N) return GRAPHKV_ERR_INVALID_ARG;
    if (p->pool_kernel < 1 || p->pool_kernel % 2 == 0) return GRAPHKV_ERR_INVALID_ARG;
    if (p->topk_nodes < 0 || p->topk_nodes > N) return GRAPHKV_ERR_INVALID_ARG;
    if (p->neighbors < 0 || p->neighbors > N - 1) return GRAPHKV_ERR_INVALID_ARG;
    if (p->rounds < 0) return GRAPHKV_ERR_INVALID_ARG;
    if (!(p->decay >= 0.0f && p->decay <= 1.0f)) return GRAPHKV_ERR_INVALID_ARG;
    if (p->dtype != GRAPHKV_BF16 && p->dtype != GRAPHKV_F32) return GRAPHKV_ERR_INVALID_ARG;
    if (p->pool_mode != GRAPHKV_POOL_MAX && p->pool_mode != GRAPHKV_POOL_AVG) return GRAPHKV_ERR_INVALID_ARG;
    if (p->signal < GRAPHKV_SIGNAL_DECAY || p->signal > GRAPHKV_SIGNAL_EVICT) return GRAPHKV_ERR_INVALID_ARG;
    if (p->reselect != 0 && p->reselect != 1) return GRAPHKV_ERR_INVALID_ARG;
    if (p->head_dim != kHeadDim && p->head_dim != 64) return GRAPHKV_ERR_UNSUPPORTED;
    const int G = p->n_q_heads / p->n_kv_heads;
    if ((long long)G * p->window > kMaxRows) return GRAPHKV_ERR_UNSUPPORTED;
    if ((long long)p->batch * p->n_kv_heads > 65535) return GRAPHKV_ERR_UNSUPPORTED;
    const int vec = p->dtype == GRAPHKV_BF16 ? 8 : 4;      // elements per 16 bytes
    for (int i = 0; i < 3; ++i) {
        if (p->q_stride[i] < 0 || p->k_stride[i] < 0 || p->v_stride[i] < 0)
            return GRAPHKV_ERR_INVALID_ARG;
        if (p->q_stride[i] % vec || p->k_stride[i] % vec || p->v_stride[i] % vec)
            return GRAPHKV_ERR_INVALID_ARG;
    }
    if (p->q_stride[2] < p->head_dim || p->k_stride[2] < p->head_dim || p->v_stride[2] < p->head_dim)
        return GRAPHKV_ERR_INVALID_ARG;
    d->batch = p->batch; d->hq = p->n_q_heads; d->hkv = p->n_kv_heads; d->G = G; d->D = p->head_dim;
    d->W = p->window; d->L = p->seq_len; d->N = N; d->GW = G * p->window;
    d->B = p->budget; d->kp = p->pool_kernel; d->K_src = p->topk_nodes;
    d->m = graphkv_resolve_neighbors(N, p->neighbors);
    d->T = p->rounds; d->lambda = p->decay; d->units = p->batch * p->n_kv_heads;
    d->bf16 = p->dtype == GRAPHKV_BF16 ? 1 : 0;
    d->pool_avg = p->pool_mode == GRAPHKV_POOL_AVG ? 1 : 0;
    d->signal = p->signal;
    d->reselect = p->reselect;
    for (int i = 0; i < 3; ++i) {
        d->qs[i] = p->q_stride[i]; d->ks[i] = p->k_stride[i]; d->vs[i] = p->v_stride[i];
    }
    return GRAPHKV_OK;
}

int env_int(const char *name, int dflt)
{
    const char *v = getenv(name);
    return v ? atoi(v) : dflt;
}

// Limit of the device-side waits in clocks: about two seconds, or GRAPHKV_WAIT_CYCLES (tests make
// a wait run out with a short one).
long long wait_cycles()
{
    const char *v = getenv("GRAPHKV_WAIT_CYCLES");
    const long long n = v ? atoll(v) : 0;
    return n > 0 ? n : tc::kWaitCycles;
}

// SMs of the current device (queried once per device).
int sm_count()
{
    static std::mutex mu;
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lk(mu);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Units per launch of a sweep.  By default all units go into one launch: measured on B200, the
// fixed cost of extra launches outweighs serving the later sweeps of a small group from L2
// (GRAPHKV_L2_GROUP_MB bounds the keys of a group for experiments).
int units_per_group(const Dims &d)
{
    const double mb = (double)d.L * d.D * 2 / 1.0e6;
    int n = (int)(env_int("GRAPHKV_L2_GROUP_MB", 1 << 20) / mb);
    if (n < 1) n = 1;
    if (n > d.units) n = d.units;
    return n;
}

// Key chunks (CTAs) per unit for a sweep of `tiles` key tiles per unit over `units` units, one CTA
// per SM: the count that minimises waves x (tiles per CTA + a per-CTA overhead of about three
// tile times), with at least min_chunks and at most max_chunks.
int sweep_chunks(int units, int tiles, int min_chunks, int max_chunks)
{
    const int n_sms = sm_count();
    int best = std::max(1, min_chunks);
    long long best_cost = -1;
    const int hi = std::max(best, std::min(tiles, max_chunks));
    for (int c = best; c <= hi; ++c) {
        const long long waves = ceil_div(units * c, n_sms);
        const long long cost = waves * (ceil_div(tiles, c) + 3);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = c;
        }
    }
    return best;
}

// ---- row-wise stages on clusters: which rows fit ----------------------------------------------------
struct ClusterPlan {
    bool ok;            // the row fits the cluster kernels
    int C, chunk, halo;
};

ClusterPlan cluster_plan(const Dims &d)
{
    ClusterPlan p{false, 1, 0, (d.kp - 1) / 2};
    if (env_int("GRAPHKV_NO_CLUSTER", 0)) return p;
    // as many CTAs per row as keep a chunk near 2048 scores (the gather of the kept rows is spread
    // over the cluster's CTAs: 16384-score rows with 2048 kept rows finish in 35 us on 8 CTAs per
    // row against 42 us on 4), but all clusters in one wave of the
    // 148 SMs when the rows allow it (two waves of clusters of 8 measured 1.8x slower than one
    // wave of clusters of 4 for 32 rows of 131072)
    while (p.C < cs::kMaxCluster && ceil_div(d.N, p.C) > 2048) p.C *= 2;
    while (p.C > 1 && d.units * p.C > sm_count() && ceil_div(d.N, p.C / 2) <= cs::kMaxChunk) p.C /= 2;
    // hundreds of sources: their neighbour lists are merged by groups of warps, kMergeWarps per CTA,
    // so more CTAs per row shorten that phase as long as all clusters stay in one wave
    while (d.K_src > 4 * cs::kMergeWarps * p.C && p.C < cs::kMaxCluster && d.units * p.C * 2 <= sm_count() &&
           ceil_div(d.N, p.C * 2) >= 1024)
        p.C *= 2;
    p.chunk = (ceil_div(d.N, p.C) + 31) & ~31;
    p.ok = p.chunk <= cs::kMaxChunk && p.halo <= cs::kMaxHalo;
    return p;
}

// Tensor-core similarity sweep: usable for bf16 keys and up to 32 neighbours; 64 sources per
// sweep of the keys, so a head with more sources (the paper's 0.3 x budget) is swept several times.
constexpr int kSimMaxSources = 4096;
struct SimPlan {
    bool ok;
    int NP;         // sources per sweep padded to 16, 32 or 64
    int chunks;     // CTAs (key chunks) per unit
    int n_tiles;    // 128-key tiles per unit
    int stages;
};

SimPlan sim_plan(const Dims &d, bool bf16)
{
    SimPlan p{false, 16, 1, ceil_div(d.N, tc::kTileKeys), 5};
    if (!bf16 || d.D != kHeadDim || d.K_src < 1 || d.K_src > kSimMaxSources || d.m < 1 ||
        d.m > tc::kSimMaxNeighbors)
        return p;
    if (env_int("GRAPHKV_FORCE_SIMT", 0)) return p;
    if (!cluster_plan(d).ok) return p;          // its candidate lists are merged by the cluster kernel
    // 64 sources per sweep leave a CTA 8 key tiles (the tensor memory holds 512 columns): four keys per
    // epilogue thread, of which the m + 1 best maxima set each source's threshold.  With more than 16
    // neighbours the chunk's candidates then crowd its 64-entry lists and the threads' queues, and
    // overflows take the slow exact path (450 sources, m = 32 at 32K keys: 2.1 ms against 0.35 ms);
    // 32 sources per sweep (16 tiles, eight keys per thread) stay clear of it and measured faster
    // there at every source count, 64 faster for m = 16.
    p.NP = d.K_src <= 16 ? 16 : (d.K_src <= 32 || d.m > 16 ? 32 : 64);
    p.stages = p.NP == 64 ? 4 : 5;
    const int cap = 512 / p.NP;
    const int group = units_per_group(d);
    p.chunks = sweep_chunks(group, p.n_tiles, ceil_div(p.n_tiles, cap), 1 << 20);
    p.ok = true;
    return p;
}

Layout layout_of(const Dims &d)
{
    Layout l;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    l.n_stat_chunks = ceil_div(d.L, kStatsChunk);
    l.max_parts = l.n_stat_chunks > 148 ? l.n_stat_chunks : 148;
    l.status = take(kAlign);
    l.arrivals = take((size_t)d.units * 2 * sizeof(int));
    l.a_hist = take((size_t)d.units * tc::kMassBins * sizeof(uint32_t));
    l.row_c = take((size_t)d.units * d.GW * sizeof(float));
    l.part = take((size_t)d.units * l.max_parts * d.GW * 2 * sizeof(float));
    l.a = take((size_t)d.units * d.N * sizeof(float));
    l.s = take((size_t)d.units * d.N * sizeof(float));
    l.src = take((size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * sizeof(int));
    const size_t pairs = (size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * (d.m > 0 ? d.m : 1);
    // the dense edge rows exist only for the generic similarity path
    const SimPlan sp0 = sim_plan(d, d.bf16 != 0);
    l.sims = take(sp0.ok ? kAlign : (size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * d.N * sizeof(float));
    l.nbr_idx = take(pairs * sizeof(int));
    l.nbr_e = take(pairs * sizeof(float));
    const SimPlan sp = sim_plan(d, d.bf16 != 0);
    const size_t slots = sp.ok ? (size_t)d.units * d.K_src * sp.chunks : 1;
    l.cand = take(slots * kCandCap * sizeof(Cand));
    l.cand_hist = take((size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * kCandBins * sizeof(uint32_t));
    const bool tail = d.bf16 && d.K_src > 0 && d.K_src <= tc::kSrcMaxK;
    l.src_cand = take(tail ? (size_t)d.units * l.max_parts * tc::kSrcCap * sizeof(tc::SrcCand) : kAlign);
    l.src_cnt = take(tail ? (size_t)d.units * l.max_parts * sizeof(int) : kAlign);
    l.total = off;
    return l;
}

graphkv_status check_ws(const Layout &l, const void *ws, size_t ws_bytes)
{
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < l.total)
        return GRAPHKV_ERR_WORKSPACE;
    return GRAPHKV_OK;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline graphkv_status launch_status()
{
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        if (getenv("GRAPHKV_LOG")) fprintf(stderr, "graphkv: launch failed: %s\n", cudaGetErrorString(e));
        return GRAPHKV_ERR_CUDA;
    }
    return GRAPHKV_OK;
}

// ---- launch accounting and optional per-kernel timing -----------------------------------------
std::atomic<long long> g_launches{0};
std::atomic<int> g_trace_on{0};
std::mutex g_trace_mu;
struct TraceEntry { const char *name; cudaEvent_t start, stop; };
std::vector<TraceEntry> g_trace;

// Counts one kernel launch; with tracing on, brackets it with CUDA events on its stream.
struct LaunchScope {
    cudaStream_t st;
    bool traced;
    TraceEntry e;
    LaunchScope(const char *name, cudaStream_t s) : st(s), traced(false)
    {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (!g_trace_on.load(std::memory_order_relaxed)) return;
        e.name = name;
        if (cudaEventCreate(&e.start) != cudaSuccess) return;
        if (cudaEventCreate(&e.stop) != cudaSuccess) { cudaEventDestroy(e.start); return; }
        cudaEventRecord(e.start, st);
        traced = true;
    }
    ~LaunchScope()
    {
        if (!traced) return;
        cudaEventRecord(e.stop, st);
        std::lock_guard<std::mutex> lk(g_trace_mu);
        g_trace.push_back(e);
    }
};
#define GKV_LAUNCH(name, st, ...)        \
    do {                                 \
        LaunchScope _scope(name, st);    \
        __VA_ARGS__;                     \
    } while (0)

template <typename T> inline T *at(void *ws, size_t off)
{
    return reinterpret_cast<T *>(static_cast<unsigned char *>(ws) + off);
}

// ---- launches with attributes -------------------------------------------------------------------
// Kernels of one API call after the first are launched with programmatic stream serialization:
// their prologue (barriers, TMEM, operand staging, the first key tiles) overlaps the tail of the
// kernel before, and they execute griddepcontrol.wait before touching anything an earlier kernel
// of the call wrote.
thread_local int t_launches_in_call = 0;

inline bool next_launch_is_dependent()
{
    static const bool enabled = [] { const char *v = getenv("GRAPHKV_PDL"); return v ? atoi(v) != 0 : true; }();
    const bool dep = enabled && t_launches_in_call > 0 && !g_trace_on.load(std::memory_order_relaxed);
    ++t_launches_in_call;
    return dep;
}

// Set before a launch_ex whose kernel makes its CTAs wait for one another: the launch then asks
// for all CTAs of the grid to be resident together (a cooperative launch), so that no other work
// on the device can keep part of the grid waiting for SMs that the rest of it holds.
thread_local bool t_cooperative = false;

template <typename... KArgs, typename... Args>
graphkv_status launch_ex(const char *name, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                         cudaStream_t st, bool dependent, int cluster_x, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[3];
    int n = 0;
    if (t_cooperative) {
        t_cooperative = false;
        attr[n].id = cudaLaunchAttributeCooperative;
        attr[n].val.cooperative = 1;
        ++n;
    }
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (dependent) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    cudaError_t e;
    GKV_LAUNCH(name, st, (e = cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...)));
    if (e != cudaSuccess) {
        if (getenv("GRAPHKV_LOG")) fprintf(stderr, "graphkv: %s: %s\n", name, cudaGetErrorString(e));
        return GRAPHKV_ERR_CUDA;
    }
    return GRAPHKV_OK;
}

// Runs `setup` once per device (function attributes are per device); returns its result.
template <typename F> bool once_per_device(std::mutex &mu, signed char (&state)[64], F setup)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lk(mu);
    if (state[dev] == 0) state[dev] = setup() ? 1 : -1;
    return state[dev] > 0;
}

template <typename Kern> bool set_smem(Kern k, size_t bytes)
{
    return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

// A value for the arrival words of the kernel of both score sweeps that no earlier call of this
// process has used (never zero; the sequence starts at a clock-derived value, so a word left by
// another process matches it only by a 1 in 2^32 chance).
uint32_t next_call_tag()
{
    static std::atomic<uint32_t> tag{
        static_cast<uint32_t>(std::chrono::steady_clock::now().time_since_epoch().count() * 2654435761u) | 1u};
    uint32_t t = tag.fetch_add(1u) + 1u;
    if (t == 0u) t = tag.fetch_add(1u) + 1u;
    return t;
}

// Status word, arrival counters and the mass histogram start every scoring call at zero: a memset
// ahead of the sweeps, except where the kernel of both sweeps clears them itself.
inline graphkv_status reset_words(const Dims &d, const Layout &l, void *ws, cudaStream_t st)
{
    return cudaMemsetAsync(ws, 0, l.a_hist + (size_t)d.units * tc::kMassBins * sizeof(uint32_t), st) == cudaSuccess
               ? GRAPHKV_OK : GRAPHKV_ERR_CUDA;
}

// ---- step (I) ------------------------------------------------------------------------------
// Attention mass before pooling, a [units][N], SIMT path (any dtype).
template <typename T>
graphkv_status run_mass_simt(const Dims &d, const Layout &l, const T *Q, const T *K, float *a,
                             void *ws, cudaStream_t st)
{
    if (reset_words(d, l, ws, st) != GRAPHKV_OK) return GRAPHKV_ERR_CUDA;
    float *part = at<float>(ws, l.part);
    const int threads = ceil_div(d.GW, 32) * 32;
    const size_t smem = ((size_t)d.GW * d.D + 2 * d.GW) * sizeof(float);
    static std::mutex mu;
    static signed char state[64] = {};
    if (!once_per_device(mu, state, [] {
            const size_t mx = ((size_t)kMaxRows * kHeadDim + 2 * kMaxRows) * sizeof(float);
            return set_smem(score_emit_simt<T, 128>, mx) && set_smem(score_emit_simt<T, 64>, mx);
        }))
        return GRAPHKV_ERR_CUDA;
    const dim3 grid_s(l.n_stat_chunks, d.units), grid_e(ceil_div(d.N, kEmitChunk), d.units);
    if (d.D == 64) {
        GKV_LAUNCH("score_stats_simt", st,
                   (score_stats_simt<T, 64><<<grid_s, threads, 0, st>>>(d, Q, K, part, l.n_stat_chunks,
                                                                        at<int>(ws, l.status))));
        GKV_LAUNCH("score_emit_simt", st,
                   (score_emit_simt<T, 64><<<grid_e, kEmitThreads, smem, st>>>(d, Q, K, part, l.n_stat_chunks, a)));
    } else {
        GKV_LAUNCH("score_stats_simt", st,
                   (score_stats_simt<T, 128><<<grid_s, threads, 0, st>>>(d, Q, K, part, l.n_stat_chunks,
                                                                         at<int>(ws, l.status))));
        GKV_LAUNCH("score_emit_simt", st,
                   (score_emit_simt<T, 128><<<grid_e, kEmitThreads, smem, st>>>(d, Q, K, part, l.n_stat_chunks, a)));
    }
    return launch_status();
}

// ---- step (I), tensor-core path (bf16) -----------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Tensor map over K [batch][hkv][rows][128] bf16 with the caller's strides; boxes of 128 rows x 64
// columns, 128-byte swizzle, zero fill past the last row.
bool make_k_tensormap(CUtensorMap *tm, const void *K, const Dims &d, int rows, const long long *ks = nullptr)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    if (!ks) ks = d.ks;
    const cuuint64_t row_b = (cuuint64_t)ks[2] * 2;
    cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows, (cuuint64_t)d.hkv, (cuuint64_t)d.batch};
    cuuint64_t head_b = (cuuint64_t)ks[1] * 2, batch_b = (cuuint64_t)ks[0] * 2;
    if (d.hkv == 1 || head_b == 0) head_b = row_b * (cuuint64_t)rows;
    if (d.batch == 1 || batch_b == 0) batch_b = head_b * (cuuint64_t)d.hkv;
    cuuint64_t strides[3] = {row_b, head_b, batch_b};
    cuuint32_t box[4] = {64, (cuuint32_t)tc::kTileKeys, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(K), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// What the emit sweep does besides the attention mass: the source nodes of Eq. 2 at its tail
// (k > 0), words cleared for the kernels that follow, the unit's mass histogram for a pooling
// kernel that follows.
struct EmitExtras {
    int k;
    int *list_chunks;   // out: candidate lists per unit the emit sweep leaves (its key chunks)
    int *src_out;
    uint32_t *zero;
    int zero_words;
    bool global_hist;
};

// Attention mass before pooling, a [units][N], tensor-core path (bf16).
graphkv_status run_mass_tc(const Dims &d, const Layout &l, const __nv_bfloat16 *Q,
                           const __nv_bfloat16 *K, float *a, void *ws, cudaStream_t st,
                           const EmitExtras &ex)
{
    CUtensorMap tmK;
    if (!make_k_tensormap(&tmK, K, d, d.L)) return GRAPHKV_ERR_CUDA;
    const int row_tiles = d.GW <= 128 ? 1 : 2;
    const int rows_pad = 128 * row_tiles;
    const int stages = row_tiles == 1 ? 5 : 4;
    const size_t smem = tc::score_smem_bytes(rows_pad, stages);
    static std::mutex mu;
    static signed char state[64] = {};
    if (!once_per_device(mu, state, [] {
        const size_t mx = std::max(tc::score_smem_bytes(256, 4), tc::score_smem_bytes(128, 5));
        return set_smem(tc::score_stats_tc<1>, mx) && set_smem(tc::score_stats_tc<2>, mx) &&
                  set_smem(tc::score_emit_tc<1>, mx) && set_smem(tc::score_emit_tc<2>, mx) &&
                  set_smem(tc::score_fused_tc<1>, mx) && set_smem(tc::score_fused_tc<2>, mx);
        }))
        return GRAPHKV_ERR_CUDA;
    const int tiles_stats = ceil_div(d.L, tc::kTileKeys), tiles_emit = ceil_div(d.N, tc::kTileKeys);
    const int group = units_per_group(d);
    graphkv_status rc = GRAPHKV_OK;
    // the kernel of both sweeps (one launch of all units, all CTAs resident) clears the head of the
    // workspace itself; every other form gets a memset first
    const bool one_kernel = ex.k == 0 && group >= d.units &&
                            d.units * sweep_chunks(d.units, tiles_stats, 1, l.max_parts) <= sm_count() &&
                            !env_int("GRAPHKV_TWO_SCORE_KERNELS", 0);
    if (!one_kernel && reset_words(d, l, ws, st) != GRAPHKV_OK) return GRAPHKV_ERR_CUDA;
    for (int u0 = 0; u0 < d.units && rc == GRAPHKV_OK; u0 += group) {
        const int nu = std::min(group, d.units - u0);
        const int chunks_s = sweep_chunks(nu, tiles_stats, 1, l.max_parts);
        const int chunks_e = sweep_chunks(nu, tiles_emit, 1, l.max_parts);
        tc::ScoreTcArgs sa{d, Q, at<float>(ws, l.part), at<float>(ws, l.row_c), at<int>(ws, l.arrivals), a,
                           ex.global_hist ? at<uint32_t>(ws, l.a_hist) : nullptr, at<int>(ws, l.status), u0,
                           chunks_s, tiles_stats, chunks_s, stages, 0,
                           tc::SourceArgs{0, 0, nullptr, nullptr, nullptr, 0, 0}, nullptr, 0, 0,
                           wait_cycles(), 0, 0u, env_int("GRAPHKV_DEBUG_WITHHOLD_COMMIT", 0)};
        tc::ScoreTcArgs ea = sa;
        ea.chunks = chunks_e;
        ea.n_tiles = tiles_emit;
        ea.src = tc::SourceArgs{ex.k, (d.kp - 1) / 2, ex.src_out, at<tc::SrcCand>(ws, l.src_cand),
                                at<int>(ws, l.src_cnt), l.max_parts, chunks_e};
        if (ex.list_chunks) *ex.list_chunks = chunks_e;
        ea.zero = ex.zero;
        ea.zero_words = ex.zero_words;
        ea.local_hist = ex.k > 0 ? 1 : 0;
        // one kernel for both sweeps when all its CTAs are resident at once (one per SM): the CTAs
        // of a unit wait for one another between the passes, so the launch is a cooperative one
        // (the device starts the grid only when all of it fits beside whatever else is running);
        // a device that refuses it gets the two kernels
        if (one_kernel) {
            tc::ScoreTcArgs fa = ea;
            fa.chunks = chunks_s;
            fa.n_tiles = tiles_stats;
            fa.clear_head = 1;
            fa.call_tag = next_call_tag();
            fa.wait_prior = next_launch_is_dependent();
            t_cooperative = true;
            rc = launch_ex("score_fused_tc", row_tiles == 1 ? tc::score_fused_tc<1> : tc::score_fused_tc<2>,
                           dim3(chunks_s, nu), dim3(tc::kScoreThreads), smem, st, fa.wait_prior != 0, 1, tmK, fa);
            if (rc == GRAPHKV_OK) continue;
            cudaGetLastError();
            if (reset_words(d, l, ws, st) != GRAPHKV_OK) return GRAPHKV_ERR_CUDA;
            rc = GRAPHKV_OK;
        }
        sa.wait_prior = next_launch_is_dependent();
        rc = launch_ex("score_stats_tc", row_tiles == 1 ? tc::score_stats_tc<1> : tc::score_stats_tc<2>,
                       dim3(chunks_s, nu), dim3(tc::kScoreThreads), smem, st, sa.wait_prior != 0, 1, tmK, sa);
        if (rc != GRAPHKV_OK) break;
        ea.wait_prior = next_launch_is_dependent();
        rc = launch_ex("score_emit_tc", row_tiles == 1 ? tc::score_emit_tc<1> : tc::score_emit_tc<2>,
                       dim3(chunks_e, nu), dim3(tc::kScoreThreads), smem, st, ea.wait_prior != 0, 1, tmK, ea);
    }
    return rc;
}

constexpr EmitExtras kPlainEmit{0, nullptr, nullptr, nullptr, 0, true};

inline bool tc_mass(const __nv_bfloat16 *, const Dims &d) { return d.D == kHeadDim && !env_int("GRAPHKV_FORCE_SIMT", 0); }
inline bool tc_mass(const float *, const Dims &) { return false; }

inline graphkv_status run_mass(const Dims &d, const Layout &l, const __nv_bfloat16 *Q,
                               const __nv_bfloat16 *K, float *a, void *ws, cudaStream_t st,
                               const EmitExtras &ex = kPlainEmit)
{
    if (!tc_mass(Q, d)) return run_mass_simt(d, l, Q, K, a, ws, st);
    return run_mass_tc(d, l, Q, K, a, ws, st, ex);
}
inline graphkv_status run_mass(const Dims &d, const Layout &l, const float *Q, const float *K,
                               float *a, void *ws, cudaStream_t st, const EmitExtras & = kPlainEmit)
{
    return run_mass_simt(d, l, Q, K, a, ws, st);
}

// ---- row-wise stages on clusters -------------------------------------------------------------
template <typename Args>
graphkv_status launch_cluster(const char *name, void (*kern)(Args), Args args, int clusters, int C,
                              size_t smem, cudaStream_t st)
{
    static std::mutex mu;
    static signed char state[64] = {};
    if (!once_per_device(mu, state, [] {
        const size_t mx = kMaxSmem;
        return set_smem(cs::pool_select_kernel<1>, mx) && set_smem(cs::pool_select_kernel<2>, mx) &&
                  set_smem(cs::pool_select_kernel<4>, mx) && set_smem(cs::pool_select_kernel<8>, mx) &&
                  set_smem(cs::pool_select_kernel<16>, mx) && set_smem(cs::pool_select_kernel<32>, mx) &&
                  set_smem(cs::finish_kernel, mx);
        }))
        return GRAPHKV_ERR_CUDA;
    args.wait_prior = next_launch_is_dependent();
    return launch_ex(name, kern, dim3(clusters * C), dim3(cs::kThreads), smem, st, args.wait_prior != 0, C,
                     args);
}

// Pooling of a -> s (when a != nullptr) and the k source nodes of Eq. 2 (when k > 0).
// `zero` (optional): zero_words words per unit cleared on the way, for the kernels that follow.
// `mass_hist` (optional): per unit, a histogram of values the scores dominate (see the kernel).
graphkv_status run_pool_sources(const Dims &d, const float *a, float *s, int k, int *src,
                                const uint32_t *mass_hist, uint32_t *zero, int zero_words,
                                cudaStream_t st)
{
    if (!a && k == 0) return GRAPHKV_OK;
    const ClusterPlan cp = cluster_plan(d);
    if (cp.ok) {
        cs::PoolSelectArgs pa{d, cp.C, cp.chunk, a ? cp.halo : 0, 0, a, s, k, src, mass_hist, zero, zero_words, 0};
        const char *name = a ? (k ? "pool_select_sources" : "pool_max") : "select_sources";
        const size_t smem = cs::smem_bytes(cp.chunk, pa.halo);
        const int per = ceil_div(cp.chunk, cs::kThreads);
        void (*kern)(cs::PoolSelectArgs) =
            per <= 1 ? cs::pool_select_kernel<1> : per <= 2 ? cs::pool_select_kernel<2>
            : per <= 4 ? cs::pool_select_kernel<4> : per <= 8 ? cs::pool_select_kernel<8>
            : per <= 16 ? cs::pool_select_kernel<16> : cs::pool_select_kernel<32>;
        return launch_cluster(name, kern, pa, d.units, cp.C, smem, st);
    }
    if (zero && cudaMemsetAsync(zero, 0, (size_t)d.units * zero_words * 4, st) != cudaSuccess)
        return GRAPHKV_ERR_CUDA;
    if (a)
        GKV_LAUNCH("pool_max", st,
                   (pool_max_kernel<<<dim3(ceil_div(d.N, 256), d.units), 256, 0, st>>>(d.N, d.kp, d.pool_avg, a, s)));
    if (k > 0) {
        SelectArgs sa{s, d.N, d.N, k, nullptr, src, nullptr};
        GKV_LAUNCH("select_sources", st, (topk_select_kernel<<<d.units, kSelectThreads, 0, st>>>(sa)));
    }
    return launch_status();
}

// ---- steps (II)+(III): the graph ------------------------------------------------------------------
inline bool graph_active(const Dims &d) { return d.K_src > 0 && d.T > 0 && d.m > 0; }

// Edges of the sources (Eq. 1) and their top-m neighbourhoods (Eq. 3) -> neighbour lists in the
// workspace.  `src` holds the sources in ascending position.
// The tensors an edge compares: the sources' vectors come from S, the swept vectors from A.
template <typename T> struct EdgeOperands {
    const T *S;
    const long long *ss;
    const T *A;
    const long long *as;
};

// `merge` (optional): the sources are still candidate lists the emit sweep left; the similarity
// sweep merges them (tensor-core path, one sweep of at most 64 sources).
template <typename T>
graphkv_status run_graph(const Dims &d, const Layout &l, const EdgeOperands<T> &eo, const int *src, void *ws,
                         cudaStream_t st, const tc::SourceArgs *merge = nullptr, const float *a_mass = nullptr)
{
    const SimPlan sp = sim_plan(d, sizeof(T) == 2);
    if (sp.ok) {
        CUtensorMap tmK;
        if (!make_k_tensormap(&tmK, eo.A, d, d.L, eo.as)) return GRAPHKV_ERR_CUDA;
        static std::mutex mu;
        static signed char state[64] = {};
        if (!once_per_device(mu, state, [] {
            return set_smem(tc::similarity_tc<16>, tc::sim_smem_bytes<16>(5)) &&
                      set_smem(tc::similarity_tc<32>, tc::sim_smem_bytes<32>(5)) &&
                      set_smem(tc::similarity_tc<64>, tc::sim_smem_bytes<64>(4));
            }))
            return GRAPHKV_ERR_CUDA;
        const int group = units_per_group(d);
        for (int u0 = 0; u0 < d.units; u0 += group) {
            const int nu = std::min(group, d.units - u0);
            // one launch takes every source: grid.z counts the sweeps of sp.NP sources each
            tc::SimTcArgs sa{d, reinterpret_cast<const __nv_bfloat16 *>(eo.S), {eo.ss[0], eo.ss[1], eo.ss[2]}, src, at<Cand>(ws, l.cand),
                             at<uint32_t>(ws, l.cand_hist), at<int>(ws, l.status), u0, sp.chunks,
                             sp.n_tiles, sp.stages, 0, wait_cycles(),
                             merge ? *merge : tc::SourceArgs{0, 0, nullptr, nullptr, nullptr, 0, 0}, a_mass};
            sa.wait_prior = next_launch_is_dependent();
            const dim3 grid(sp.chunks, nu, ceil_div(d.K_src, sp.NP)), block(tc::kSimThreads);
            graphkv_status rc;
            if (sp.NP == 16)
                rc = launch_ex("similarity_tc", tc::similarity_tc<16>, grid, block,
                               tc::sim_smem_bytes<16>(sp.stages), st, sa.wait_prior != 0, 1, tmK, sa);
            else if (sp.NP == 32)
                rc = launch_ex("similarity_tc", tc::similarity_tc<32>, grid, block,
                               tc::sim_smem_bytes<32>(sp.stages), st, sa.wait_prior != 0, 1, tmK, sa);
            else
                rc = launch_ex("similarity_tc", tc::similarity_tc<64>, grid, block,
                               tc::sim_smem_bytes<64>(sp.stages), st, sa.wait_prior != 0, 1, tmK, sa);
            if (rc != GRAPHKV_OK) return rc;
        }
        return GRAPHKV_OK;
    }
    float *sims = at<float>(ws, l.sims);
    const dim3 grid_sim(ceil_div(d.N, kSimChunk), d.units);
    const Strides3 st_s{{eo.ss[0], eo.ss[1], eo.ss[2]}}, st_a{{eo.as[0], eo.as[1], eo.as[2]}};
    if (d.D == 64)
        GKV_LAUNCH("similarity_simt", st,
                   (similarity_simt<T, 64><<<grid_sim, kSimThreads, 0, st>>>(d, eo.S, st_s, eo.A, st_a, src, sims)));
    else
        GKV_LAUNCH("similarity_simt", st,
                   (similarity_simt<T, 128><<<grid_sim, kSimThreads, 0, st>>>(d, eo.S, st_s, eo.A, st_a, src, sims)));
    SelectArgs na{sims, d.N, d.N, d.m, src, at<int>(ws, l.nbr_idx), at<float>(ws, l.nbr_e)};
    GKV_LAUNCH("select_neighbors", st,
               (topk_select_kernel<<<d.units * d.K_src, kSelectThreads, 0, st>>>(na)));
    return launch_status();
}

// Decay rounds (when has_graph) on s in place, then (when do_select) the budget selection and
// the gather of the compact cache.
// How the finishing kernel spreads a unit over a cluster: a row of up to kMaxChunk scores is held
// whole by the first CTA (its selection then needs no exchange between CTAs) and the other CTAs of
// the cluster only merge neighbour lists and gather; a longer row is split over all C CTAs.
struct FinishPlan {
    bool ok;
    int C, R, chunk;
};

FinishPlan finish_plan(const Dims &d, int halo)
{
    FinishPlan p{false, 1, 1, 0};
    if (env_int("GRAPHKV_NO_CLUSTER", 0) || halo > cs::kMaxHalo) return p;
    const ClusterPlan cp = cluster_plan(d);
    p.C = p.R = cp.C;
    p.chunk = cp.chunk;
    p.ok = p.chunk <= cs::kMaxChunk;
    return p;
}

// Per-batch-element budgets of the call in flight (graphkv_compress_layers), or none.
thread_local const int32_t *t_budgets = nullptr;
// The caller of the call in flight wants the final scores (graphkv_compress without scores_out
// does not: its last kernel then leaves them in shared memory).
thread_local bool t_keep_scores = true;

graphkv_status run_finish(const Dims &d, const Layout &l, int elem_bytes, const float *a, float *s,
                          bool has_graph, bool merge, bool do_select, const void *K, const void *V,
                          void *K_out, void *V_out, int *idx_out, void *ws, cudaStream_t st)
{
    if (!has_graph && !do_select && !a) return GRAPHKV_OK;
    const int halo = a ? (d.kp - 1) / 2 : 0;
    const FinishPlan fp = finish_plan(d, halo);
    if (fp.ok && cluster_plan(d).ok) {
        cs::FinishArgs fa{d, fp.C, fp.R, fp.chunk, halo, 0, a, s, at<int>(ws, l.nbr_idx), at<float>(ws, l.nbr_e),
                          has_graph ? 1 : 0, has_graph && merge ? 1 : 0, at<Cand>(ws, l.cand),
                          at<uint32_t>(ws, l.cand_hist), sim_plan(d, d.bf16 != 0).chunks, do_select ? 1 : 0, idx_out, elem_bytes,
                          static_cast<const unsigned char *>(K), static_cast<const unsigned char *>(V),
                          static_cast<unsigned char *>(K_out), static_cast<unsigned char *>(V_out), 0, cs::kStage,
                          (t_keep_scores || !do_select) ? 1 : 0, 0, {}};
        if (t_budgets && do_select) {
            fa.per_batch_budget = 1;
            for (int i = 0; i < d.batch; ++i) fa.budget_of[i] = t_budgets[i];
        }
        // the neighbour lists of a unit are staged in shared memory when K_src * m entries fit
        const int pairs = has_graph ? d.K_src * d.m : 0;
        if (pairs > cs::kStage && cs::smem_bytes(fp.chunk, halo, (pairs + 255) & ~255) <= kMaxSmem)
            fa.stage_cap = (pairs + 255) & ~255;
        const char *name = has_graph ? (do_select ? "decay_select_gather" : "decay_rounds") : "select_gather";
        return launch_cluster(name, cs::finish_kernel, fa, d.units, fp.C,
                              cs::smem_bytes(fp.chunk, halo, fa.stage_cap), st);
    }
    if (t_budgets && do_select) return GRAPHKV_ERR_UNSUPPORTED;      // only the cluster kernel takes budgets per layer
    if (a)
        GKV_LAUNCH("pool_max", st,
                   (pool_max_kernel<<<dim3(ceil_div(d.N, 256), d.units), 256, 0, st>>>(d.N, d.kp, d.pool_avg, a, s)));
    if (has_graph)
        GKV_LAUNCH("decay_rounds", st,
                   (decay_rounds_kernel<<<d.units, 256, 0, st>>>(d, at<int>(ws, l.nbr_idx),
                                                                 at<float>(ws, l.nbr_e), s)));
    if (do_select) {
        SelectArgs sa{s, d.N, d.N, d.B, nullptr, idx_out, nullptr};
        GKV_LAUNCH("select_budget", st, (topk_select_kernel<<<d.units, kSelectThreads, 0, st>>>(sa)));
        if (K || V) {
            const long long total = (long long)d.units * (d.B + d.W) * (d.D * elem_bytes / 16);
            const int blocks = (int)std::min<long long>((total + kGatherThreads - 1) / kGatherThreads,
                                                        148LL * 16);
            GKV_LAUNCH("gather_rows", st,
                       (gather_rows_kernel<<<blocks, kGatherThreads, 0, st>>>(
                           d, elem_bytes, static_cast<const unsigned char *>(K),
                           static_cast<const unsigned char *>(V), idx_out,
                           static_cast<unsigned char *>(K_out), static_cast<unsigned char *>(V_out))));
        }
    }
    return launch_status();
}

// ---- the calls, typed ---------------------------------------------------------------------------

template <typename T>
graphkv_status do_score(const Dims &d, const Layout &l, const T *Q, const T *K, float *scores,
                        void *ws, cudaStream_t st)
{
    float *a = d.kp > 1 ? at<float>(ws, l.a) : scores;
    graphkv_status rc = run_mass(d, l, Q, K, a, ws, st);
    if (rc != GRAPHKV_OK || d.kp == 1) return rc;
    return run_pool_sources(d, a, scores, 0, nullptr, nullptr, nullptr, 0, st);
}

// One pass of steps (II)+(III) from the scores as they stand: sources, edges, neighbourhoods,
// d.T rounds over that graph.
template <typename T>
graphkv_status propagate_once(const Dims &d, const Layout &l, const EdgeOperands<T> &eo, float *scores,
                              int *src, void *ws, cudaStream_t st)
{
    const bool tc_graph = graph_active(d) && sim_plan(d, sizeof(T) == 2).ok;
    graphkv_status rc = run_pool_sources(d, nullptr, scores, d.K_src, src, nullptr,
                                         tc_graph ? at<uint32_t>(ws, l.cand_hist) : nullptr,
                                         d.K_src * kCandBins, st);
    if (rc != GRAPHKV_OK || !graph_active(d)) return rc;
    if ((rc = run_graph(d, l, eo, src, ws, st)) != GRAPHKV_OK) return rc;
    return run_finish(d, l, (int)sizeof(T), nullptr, scores, true, sim_plan(d, sizeof(T) == 2).ok, false,
                      nullptr, nullptr, nullptr, nullptr, nullptr, ws, st);
}

// Steps (II)+(III).  With d.reselect every round is a pass of its own: the sources are re-picked
// from the scores the round before left and their neighbourhoods rebuilt (src_out then holds the
// sources of the last round).
template <typename T>
graphkv_status do_propagate(const Dims &d, const Layout &l, const EdgeOperands<T> &eo, float *scores,
                            int *src_out, void *ws, cudaStream_t st)
{
    if (d.K_src == 0) return GRAPHKV_OK;
    int *src = src_out ? src_out : at<int>(ws, l.src);
    if (!d.reselect || d.T <= 1) return propagate_once(d, l, eo, scores, src, ws, st);
    Dims one = d;
    one.T = 1;
    for (int t = 0; t < d.T; ++t) {
        const graphkv_status rc = propagate_once(one, l, eo, scores, src, ws, st);
        if (rc != GRAPHKV_OK) return rc;
    }
    return GRAPHKV_OK;
}

template <typename T>
graphkv_status do_compress(const Dims &d, const Layout &l, const T *Q, const T *K, const void *V,
                           void *K_out, void *V_out, int *idx_out, float *s, void *ws,
                           cudaStream_t st)
{
    const bool graph = graph_active(d);
    float *a = d.kp > 1 ? at<float>(ws, l.a) : s;
    int *src = at<int>(ws, l.src);
    const bool tc_graph = graph && sim_plan(d, sizeof(T) == 2).ok;
    const int halo = (d.kp - 1) / 2;
    // The tensor-core emit sweep can leave candidate lists for the sources at its tail, the
    // similarity sweep merge them and the finishing kernel pool, which saves the pooling kernel
    // (one sweep of at most 64 sources, one launch group, max pooling).  Measured on B200 the
    // merge in front of every similarity CTA costs what the pooling kernel takes (32K keys: 114
    // against 112 us per step; 131072 x 4: 1.25 against 1.13 ms), so it is off by default.
    const bool tail_src = tc_mass(Q, d) && tc_graph && d.K_src <= tc::kSrcMaxK && !d.pool_avg &&
                          units_per_group(d) >= d.units && env_int("GRAPHKV_TAIL_SOURCES", 0);
    const bool finish_pools = d.kp > 1 && !d.pool_avg && (tail_src || !graph) && finish_plan(d, halo).ok &&
                              cluster_plan(d).ok;
    graphkv_status rc;
    int list_chunks = 0;
    if (tail_src || !graph) {
        const EmitExtras ex{tail_src ? d.K_src : 0, &list_chunks, src, tail_src ? at<uint32_t>(ws, l.cand_hist) : nullptr,
                            tail_src ? d.K_src * kCandBins : 0, false};
        if ((rc = run_mass(d, l, Q, K, a, ws, st, ex)) != GRAPHKV_OK) return rc;
        if (d.kp > 1 && !finish_pools &&
            (rc = run_pool_sources(d, a, s, 0, nullptr, nullptr, nullptr, 0, st)) != GRAPHKV_OK)
            return rc;
    } else {
        if ((rc = run_mass(d, l, Q, K, a, ws, st)) != GRAPHKV_OK) return rc;
        // the tensor-core emit sweep leaves a histogram of the attention mass behind
        rc = run_pool_sources(d, d.kp > 1 ? a : nullptr, s, d.K_src, src,
                              tc_mass(Q, d) ? at<uint32_t>(ws, l.a_hist) : nullptr,
                              tc_graph ? at<uint32_t>(ws, l.cand_hist) : nullptr, d.K_src * kCandBins, st);
        if (rc != GRAPHKV_OK) return rc;
    }
    const EdgeOperands<T> eo{K, d.ks, K, d.ks};
    if (graph && d.reselect && d.T > 1) {
        // every round its own pass: the first one rides on the sources picked above, the rounds
        // after it start from the scores in `s`; the last pass also selects and gathers
        Dims one = d;
        one.T = 1;
        const tc::SourceArgs merge1{d.K_src, halo, src, at<tc::SrcCand>(ws, l.src_cand), at<int>(ws, l.src_cnt),
                                    l.max_parts, list_chunks};
        if ((rc = run_graph(one, l, eo, src, ws, st, tail_src ? &merge1 : nullptr, a)) != GRAPHKV_OK) return rc;
        if ((rc = run_finish(one, l, (int)sizeof(T), finish_pools ? a : nullptr, s, true, tc_graph, false,
                             nullptr, nullptr, nullptr, nullptr, nullptr, ws, st)) != GRAPHKV_OK)
            return rc;
        for (int t = 1; t < d.T; ++t)
            if ((rc = propagate_once(one, l, eo, s, src, ws, st)) != GRAPHKV_OK) return rc;
        return run_finish(one, l, (int)sizeof(T), nullptr, s, false, false, true, K, V, K_out, V_out, idx_out,
                          ws, st);
    }
    const tc::SourceArgs merge{d.K_src, halo, src, at<tc::SrcCand>(ws, l.src_cand), at<int>(ws, l.src_cnt),
                               l.max_parts, list_chunks};
    if (graph && (rc = run_graph(d, l, eo, src, ws, st, tail_src ? &merge : nullptr, a)) != GRAPHKV_OK) return rc;
    return run_finish(d, l, (int)sizeof(T), finish_pools ? a : nullptr, s, graph, tc_graph, true, K, V,
                      K_out, V_out, idx_out, ws, st);
}

// ---- KNorm initial score ---------------------------------------------------------------------
// s_j = 1 / max(||k_j||, eps) for the prefix keys: 16 threads share a key row (16 bytes each of a
// bf16 row, 32 of an fp32 row), eight rows in flight per thread.  grid (CTAs per unit, units).
template <typename T, int kD>
__global__ void __launch_bounds__(256) knorm_score_kernel(Dims d, const T *__restrict__ K, float *__restrict__ scores)
{
    constexpr int kTpr = kD / 8;                 // threads per key row, eight elements each
    const int sub = threadIdx.x & (kTpr - 1), unit = blockIdx.y;
    const T *Kh = K + (unit / d.hkv) * d.ks[0] + (long long)(unit % d.hkv) * d.ks[1] + sub * 8;
    float *out = scores + (long long)unit * d.N;
    const int stride = (gridDim.x * blockDim.x) / kTpr;
    for (int j0 = (blockIdx.x * blockDim.x + threadIdx.x) / kTpr; j0 < d.N; j0 += 8 * stride) {
        float n2[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * stride;
            n2[u] = 0.f;
            if (j < d.N) {
                float v[8];
                load8(Kh + (long long)j * d.ks[2], v);
#pragma unroll
                for (int e = 0; e < 8; ++e) n2[u] = fmaf(v[e], v[e], n2[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int o = kTpr / 2; o > 0; o >>= 1) n2[u] += __shfl_xor_sync(0xffffffffu, n2[u], o);
            const int j = j0 + u * stride;
            if (sub == 0 && j < d.N) out[j] = 1.0f / fmaxf(sqrtf(n2[u]), kNormEps);
        }
    }
}

// ---- built-in scratch for graphkv_score_noalloc ---------------------------------------------------
// Device memory that is part of the library image.  In host code the array's name is only a handle
// for cudaGetSymbolAddress; kernels get the address looked up once per device.
static __device__ __align__(256) unsigned char g_builtin_scratch[GRAPHKV_BUILTIN_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_builtin_mu;
void *g_builtin_ptr[kMaxDevices] = {};

// Address of the built-in scratch on the current device (nullptr on failure).
void *builtin_scratch()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lk(g_builtin_mu);
    if (!g_builtin_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess) return nullptr;
        g_builtin_ptr[dev] = p;
    }
    return g_builtin_ptr[dev];
}

}  // namespace

extern "C" {

int32_t graphkv_resolve_neighbors(int32_t n_prefix, int32_t neighbors)
{
    if (neighbors > 0) return neighbors;
    int32_t m = n_prefix / 1000;
    m = m < 1 ? 1 : (m > 32 ? 32 : m);
    if (m > n_prefix - 1) m = n_prefix - 1;
    return m;
}

size_t graphkv_workspace_bytes(const graphkv_params *params)
{
    Dims d;
    if (resolve(params, &d) != GRAPHKV_OK) return 0;
    return layout_of(d).total;
}

graphkv_status graphkv_score(const graphkv_params *params, const void *Qw, const void *K,
                             float *scores, void *workspace, size_t workspace_bytes, void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    t_launches_in_call = 0;
    if (!Qw || !K || !scores || !aligned16(Qw) || !aligned16(K)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->dtype == GRAPHKV_BF16)
        return do_score(d, l, static_cast<const __nv_bfloat16 *>(Qw),
                        static_cast<const __nv_bfloat16 *>(K), scores, workspace, st);
    return do_score(d, l, static_cast<const float *>(Qw), static_cast<const float *>(K), scores,
                    workspace, st);
}

size_t graphkv_builtin_scratch_needed(const graphkv_params *params)
{
    Dims d;
    if (resolve(params, &d) != GRAPHKV_OK) return 0;
    return layout_of(d).s;       // the scoring call uses the regions laid out before `s`
}

graphkv_status graphkv_score_noalloc(const graphkv_params *params, const void *Qw, const void *K,
                                     float *scores, void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    t_launches_in_call = 0;
    if (!Qw || !K || !scores || !aligned16(Qw) || !aligned16(K)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if (l.s > GRAPHKV_BUILTIN_SCRATCH_BYTES) return GRAPHKV_ERR_BUILTIN_SCRATCH;
    void *ws = builtin_scratch();
    if (!ws) return GRAPHKV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->dtype == GRAPHKV_BF16)
        return do_score(d, l, static_cast<const __nv_bfloat16 *>(Qw),
                        static_cast<const __nv_bfloat16 *>(K), scores, ws, st);
    return do_score(d, l, static_cast<const float *>(Qw), static_cast<const float *>(K), scores, ws, st);
}

graphkv_status graphkv_read_status_noalloc(void *stream)
{
    void *ws = builtin_scratch();
    if (!ws) return GRAPHKV_ERR_CUDA;
    return graphkv_read_status(ws, stream);
}

graphkv_status graphkv_propagate_edges(const graphkv_params *params, const void *K, const void *V,
                                       int32_t src_tensor, int32_t all_tensor, float *scores,
                                       int32_t *src_idx_out, void *workspace, size_t workspace_bytes,
                                       void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    t_launches_in_call = 0;
    if ((src_tensor != GRAPHKV_TENSOR_K && src_tensor != GRAPHKV_TENSOR_V) ||
        (all_tensor != GRAPHKV_TENSOR_K && all_tensor != GRAPHKV_TENSOR_V))
        return GRAPHKV_ERR_INVALID_ARG;
    const void *S = src_tensor == GRAPHKV_TENSOR_K ? K : V, *A = all_tensor == GRAPHKV_TENSOR_K ? K : V;
    const long long *ss = src_tensor == GRAPHKV_TENSOR_K ? d.ks : d.vs;
    const long long *as = all_tensor == GRAPHKV_TENSOR_K ? d.ks : d.vs;
    if (!S || !A || !scores || !aligned16(S) || !aligned16(A)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->dtype == GRAPHKV_BF16) {
        const EdgeOperands<__nv_bfloat16> eo{static_cast<const __nv_bfloat16 *>(S), ss,
                                             static_cast<const __nv_bfloat16 *>(A), as};
        return do_propagate(d, l, eo, scores, src_idx_out, workspace, st);
    }
    const EdgeOperands<float> eo{static_cast<const float *>(S), ss, static_cast<const float *>(A), as};
    return do_propagate(d, l, eo, scores, src_idx_out, workspace, st);
}

graphkv_status graphkv_propagate(const graphkv_params *params, const void *K, float *scores,
                                 int32_t *src_idx_out, void *workspace, size_t workspace_bytes,
                                 void *stream)
{
    return graphkv_propagate_edges(params, K, nullptr, GRAPHKV_TENSOR_K, GRAPHKV_TENSOR_K, scores,
                                   src_idx_out, workspace, workspace_bytes, stream);
}

graphkv_status graphkv_score_knorm(const graphkv_params *params, const void *K, float *scores, void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    if (!K || !scores || !aligned16(K)) return GRAPHKV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // about one wave of resident CTAs (eight of 256 threads per SM) over all units
    const int per_unit = std::max(1, std::min(ceil_div(d.N, 16 * 8), ceil_div(sm_count() * 8, d.units)));
    const dim3 grid(per_unit, d.units);
    const __nv_bfloat16 *Kb = static_cast<const __nv_bfloat16 *>(K);
    const float *Kf = static_cast<const float *>(K);
    if (params->dtype == GRAPHKV_BF16 && d.D == 64)
        GKV_LAUNCH("knorm_score", st, (knorm_score_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(d, Kb, scores)));
    else if (params->dtype == GRAPHKV_BF16)
        GKV_LAUNCH("knorm_score", st, (knorm_score_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(d, Kb, scores)));
    else if (d.D == 64)
        GKV_LAUNCH("knorm_score", st, (knorm_score_kernel<float, 64><<<grid, 256, 0, st>>>(d, Kf, scores)));
    else
        GKV_LAUNCH("knorm_score", st, (knorm_score_kernel<float, 128><<<grid, 256, 0, st>>>(d, Kf, scores)));
    return launch_status();
}

graphkv_status graphkv_select_gather(const graphkv_params *params, const float *scores,
                                     const void *K, const void *V, void *K_out, void *V_out,
                                     int32_t *idx_out, void *workspace, size_t workspace_bytes,
                                     void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    t_launches_in_call = 0;
    if (!scores || !idx_out) return GRAPHKV_ERR_INVALID_ARG;
    if ((K == nullptr) != (K_out == nullptr) || (V == nullptr) != (V_out == nullptr))
        return GRAPHKV_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    const int elem = params->dtype == GRAPHKV_BF16 ? 2 : 4;
    return run_finish(d, l, elem, nullptr, const_cast<float *>(scores), false, false, true, K, V, K_out,
                      V_out, idx_out, workspace, static_cast<cudaStream_t>(stream));
}

graphkv_status graphkv_compress(const graphkv_params *params, const void *Qw, const void *K,
                                const void *V, void *K_out, void *V_out, int32_t *idx_out,
                                float *scores_out, void *workspace, size_t workspace_bytes,
                                void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    t_launches_in_call = 0;
    if (!Qw || !K || !V || !K_out || !V_out || !idx_out) return GRAPHKV_ERR_INVALID_ARG;
    if (!aligned16(Qw) || !aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *s = scores_out ? scores_out : at<float>(workspace, l.s);
    t_keep_scores = scores_out != nullptr;
    if (params->dtype == GRAPHKV_BF16)
        rc = do_compress(d, l, static_cast<const __nv_bfloat16 *>(Qw),
                         static_cast<const __nv_bfloat16 *>(K), V, K_out, V_out, idx_out, s, workspace, st);
    else
        rc = do_compress(d, l, static_cast<const float *>(Qw), static_cast<const float *>(K), V, K_out,
                         V_out, idx_out, s, workspace, st);
    t_keep_scores = true;
    return rc;
}

graphkv_status graphkv_compress_layers(const graphkv_params *params, const int32_t *budgets,
                                       const void *Qw, const void *K, const void *V, void *K_out,
                                       void *V_out, int32_t *idx_out, float *scores_out,
                                       void *workspace, size_t workspace_bytes, void *stream)
{
    if (!params || !budgets) return GRAPHKV_ERR_INVALID_ARG;
    if (params->batch > cs::kMaxBudgets) return GRAPHKV_ERR_UNSUPPORTED;
    for (int i = 0; i < params->batch; ++i)
        if (budgets[i] < 1 || budgets[i] > params->budget) return GRAPHKV_ERR_INVALID_ARG;
    t_budgets = budgets;
    const graphkv_status rc = graphkv_compress(params, Qw, K, V, K_out, V_out, idx_out, scores_out,
                                               workspace, workspace_bytes, stream);
    t_budgets = nullptr;
    return rc;
}

static bool decode_shape(const graphkv_params *p, DecodeArgs *a)
{
    if (!p || p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->seq_len < 1 ||
        p->n_q_heads % p->n_kv_heads != 0 || p->head_dim != kHeadDim ||
        p->n_q_heads / p->n_kv_heads > kDecMaxG || (long long)p->batch * p->n_kv_heads > 65535 ||
        (p->dtype != GRAPHKV_BF16 && p->dtype != GRAPHKV_F32))
        return false;
    const int vec = p->dtype == GRAPHKV_BF16 ? 8 : 4;
    for (int i = 0; i < 3; ++i)
        if (p->k_stride[i] < 0 || p->v_stride[i] < 0 || p->k_stride[i] % vec || p->v_stride[i] % vec) return false;
    if (p->q_stride[0] < 0 || p->q_stride[1] < kHeadDim) return false;
    a->batch = p->batch; a->hq = p->n_q_heads; a->hkv = p->n_kv_heads; a->G = p->n_q_heads / p->n_kv_heads;
    a->rows = p->seq_len;
    const int units = p->batch * p->n_kv_heads;
    const int tiles = ceil_div(p->seq_len, kDecTile);
    a->splits = std::max(1, std::min(std::min(tiles, 256), ceil_div(4 * sm_count(), units)));
    a->qs[0] = p->q_stride[0]; a->qs[1] = p->q_stride[1];
    for (int i = 0; i < 3; ++i) { a->ks[i] = p->k_stride[i]; a->vs[i] = p->v_stride[i]; }
    return true;
}

size_t graphkv_decode_workspace_bytes(const graphkv_params *params)
{
    DecodeArgs a;
    if (!decode_shape(params, &a)) return 0;
    return align_up((size_t)a.batch * a.hkv * a.splits * a.G * (2 + kHeadDim) * sizeof(float));
}

graphkv_status graphkv_decode_attention(const graphkv_params *params, const void *q, const void *K,
                                        const void *V, float *out, void *workspace,
                                        size_t workspace_bytes, void *stream)
{
    DecodeArgs a;
    if (!decode_shape(params, &a)) return params && params->head_dim != kHeadDim ? GRAPHKV_ERR_UNSUPPORTED
                                                                                  : GRAPHKV_ERR_INVALID_ARG;
    if (!q || !K || !V || !out || !aligned16(K) || !aligned16(V)) return GRAPHKV_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < graphkv_decode_workspace_bytes(params)) return GRAPHKV_ERR_WORKSPACE;
    a.part = static_cast<float *>(workspace);
    a.out = out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid(a.splits, a.batch * a.hkv);
    if (params->dtype == GRAPHKV_BF16)
        GKV_LAUNCH("decode_partial", st, (decode_partial_kernel<__nv_bfloat16><<<grid, kDecThreads, 0, st>>>(
                                             a, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(K),
                                             static_cast<const __nv_bfloat16 *>(V))));
    else
        GKV_LAUNCH("decode_partial", st, (decode_partial_kernel<float><<<grid, kDecThreads, 0, st>>>(
                                             a, static_cast<const float *>(q), static_cast<const float *>(K),
                                             static_cast<const float *>(V))));
    GKV_LAUNCH("decode_merge", st, (decode_merge_kernel<<<a.batch * a.hkv * a.G, kHeadDim, 0, st>>>(a)));
    return launch_status();
}

graphkv_status graphkv_read_status(const void *workspace, void *stream)
{
    if (!workspace) return GRAPHKV_ERR_WORKSPACE;
    int word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GRAPHKV_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GRAPHKV_ERR_CUDA;
    if (word < 0 || word > GRAPHKV_ERR_TIMEOUT) return GRAPHKV_ERR_CUDA;
    return static_cast<graphkv_status>(word);
}

graphkv_status graphkv_read_neighbors(const graphkv_params *params, const void *workspace,
                                      size_t workspace_bytes, int32_t *nbr_idx_out,
                                      float *nbr_e_out, void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    if (!graph_active(d)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t pairs = (size_t)d.units * d.K_src * d.m;
    const unsigned char *ws = static_cast<const unsigned char *>(workspace);
    if (nbr_idx_out && cudaMemcpyAsync(nbr_idx_out, ws + l.nbr_idx, pairs * sizeof(int),
                                       cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return GRAPHKV_ERR_CUDA;
    if (nbr_e_out && cudaMemcpyAsync(nbr_e_out, ws + l.nbr_e, pairs * sizeof(float),
                                     cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return GRAPHKV_ERR_CUDA;
    return GRAPHKV_OK;
}

int64_t graphkv_launch_count(void) { return g_launches.load(); }

void graphkv_trace_enable(int32_t enable)
{
    g_trace_on.store(enable ? 1 : 0);
}

int32_t graphkv_trace_read(graphkv_trace_record *out, int32_t capacity)
{
    std::lock_guard<std::mutex> lk(g_trace_mu);
    int32_t n = 0;
    for (const TraceEntry &e : g_trace) {
        float ms = -1.f;
        if (cudaEventSynchronize(e.stop) == cudaSuccess) cudaEventElapsedTime(&ms, e.start, e.stop);
        if (out && n < capacity) {
            strncpy(out[n].name, e.name, sizeof(out[n].name) - 1);
            out[n].name[sizeof(out[n].name) - 1] = 0;
            out[n].ms = ms;
            ++n;
        }
        cudaEventDestroy(e.start);
        cudaEventDestroy(e.stop);
    }
    g_trace.clear();
    return n;
}

int32_t graphkv_phase_timing_read(uint64_t *out)
{
#ifdef GRAPHKV_PHASE_TIMING
    if (!out || cudaDeviceSynchronize() != cudaSuccess) return 0;
    constexpr size_t n = (size_t)kPhaseKernels * kPhaseSlots;
    std::vector<unsigned long long> sum(n), mx(n), cnt(kPhaseKernels);
    if (cudaMemcpyFromSymbol(sum.data(), g_phase_sum, n * 8) != cudaSuccess ||
        cudaMemcpyFromSymbol(mx.data(), g_phase_max, n * 8) != cudaSuccess ||
        cudaMemcpyFromSymbol(cnt.data(), g_phase_cnt, kPhaseKernels * 8) != cudaSuccess)
        return 0;
    for (size_t i = 0; i < n; ++i) {
        out[2 * i] = sum[i];
        out[2 * i + 1] = mx[i];
    }
    for (int k = 0; k < kPhaseKernels; ++k) out[2 * n + k] = cnt[k];
    std::fill(sum.begin(), sum.end(), 0ull);
    cudaMemcpyToSymbol(g_phase_sum, sum.data(), n * 8);
    cudaMemcpyToSymbol(g_phase_max, sum.data(), n * 8);
    cudaMemcpyToSymbol(g_phase_cnt, sum.data(), kPhaseKernels * 8);
    return 1;
#else
    (void)out;
    return 0;
#endif
}

const char *graphkv_status_string(graphkv_status status)
{
    switch (status) {
        case GRAPHKV_OK: return "ok";
        case GRAPHKV_ERR_INVALID_ARG: return "invalid argument";
        case GRAPHKV_ERR_UNSUPPORTED: return "unsupported configuration";
        case GRAPHKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GRAPHKV_ERR_CUDA: return "CUDA error";
        case GRAPHKV_ERR_TIMEOUT: return "device-side wait timed out";
        case GRAPHKV_ERR_BUILTIN_SCRATCH:
            return "problem needs more scratch than the built-in array of graphkv_score_noalloc holds";
    }
    return "unknown status";
}

}  // extern "C"
