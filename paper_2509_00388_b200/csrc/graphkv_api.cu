// C ABI of the GraphKV library: argument validation, workspace layout and kernel launches.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "gather.cuh"
#include "propagate_simt.cuh"
#include "score_simt.cuh"
#include "score_tc.cuh"
#include "select.cuh"

using namespace graphkv;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Workspace carve-up; every region starts 256-byte aligned.
struct Layout {
    size_t status;      // int status word (256 bytes reserved)
    size_t part;        // softmax row statistics per key chunk
    size_t a;           // attention mass before pooling [units][N]
    size_t s;           // scores when the caller gives no array [units][N]
    size_t src;         // source nodes [units][K_src]
    size_t sims;        // edges of the sources [units][K_src][N]
    size_t nbr_idx;     // neighbourhoods [units][K_src][m]
    size_t nbr_e;
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
    if (p->pool_mode != GRAPHKV_POOL_MAX) return GRAPHKV_ERR_UNSUPPORTED;
    if (p->head_dim != kHeadDim) return GRAPHKV_ERR_UNSUPPORTED;
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
    if (p->q_stride[2] < kHeadDim || p->k_stride[2] < kHeadDim || p->v_stride[2] < kHeadDim)
        return GRAPHKV_ERR_INVALID_ARG;
    d->batch = p->batch; d->hq = p->n_q_heads; d->hkv = p->n_kv_heads; d->G = G;
    d->W = p->window; d->L = p->seq_len; d->N = N; d->GW = G * p->window;
    d->B = p->budget; d->kp = p->pool_kernel; d->K_src = p->topk_nodes;
    d->m = graphkv_resolve_neighbors(N, p->neighbors);
    d->T = p->rounds; d->lambda = p->decay; d->units = p->batch * p->n_kv_heads;
    for (int i = 0; i < 3; ++i) {
        d->qs[i] = p->q_stride[i]; d->ks[i] = p->k_stride[i]; d->vs[i] = p->v_stride[i];
    }
    return GRAPHKV_OK;
}

Layout layout_of(const Dims &d)
{
    Layout l;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    l.n_stat_chunks = ceil_div(d.L, kStatsChunk);
    l.max_parts = l.n_stat_chunks > 2 * 148 ? l.n_stat_chunks : 2 * 148;
    l.status = take(kAlign);
    l.part = take((size_t)d.units * l.max_parts * d.GW * 2 * sizeof(float));
    l.a = take((size_t)d.units * d.N * sizeof(float));
    l.s = take((size_t)d.units * d.N * sizeof(float));
    l.src = take((size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * sizeof(int));
    const size_t pairs = (size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * (d.m > 0 ? d.m : 1);
    l.sims = take((size_t)d.units * (d.K_src > 0 ? d.K_src : 1) * d.N * sizeof(float));
    l.nbr_idx = take(pairs * sizeof(int));
    l.nbr_e = take(pairs * sizeof(float));
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

// ---- step (I) ------------------------------------------------------------------------------
template <typename T>
graphkv_status run_score(const Dims &d, const Layout &l, const T *Q, const T *K, float *scores,
                         void *ws, cudaStream_t st)
{
    float *part = at<float>(ws, l.part);
    float *a = d.kp > 1 ? at<float>(ws, l.a) : scores;
    const int threads = ceil_div(d.GW, 32) * 32;
    GKV_LAUNCH("score_stats_simt", st,
               (score_stats_simt<T><<<dim3(l.n_stat_chunks, d.units), threads, 0, st>>>(
                   d, Q, K, part, l.n_stat_chunks, at<int>(ws, l.status))));
    const size_t smem = ((size_t)d.GW * kHeadDim + 2 * d.GW) * sizeof(float);
    static bool attr_set[2] = {false, false};
    if (!attr_set[sizeof(T) == 2]) {
        if (cudaFuncSetAttribute(score_emit_simt<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(((size_t)kMaxRows * kHeadDim + 2 * kMaxRows) * sizeof(float))) !=
            cudaSuccess)
            return GRAPHKV_ERR_CUDA;
        attr_set[sizeof(T) == 2] = true;
    }
    GKV_LAUNCH("score_emit_simt", st,
               (score_emit_simt<T><<<dim3(ceil_div(d.N, kEmitChunk), d.units), kEmitThreads, smem,
                                     st>>>(d, Q, K, part, l.n_stat_chunks, a)));
    if (d.kp > 1)
        GKV_LAUNCH("pool_max", st,
                   (pool_max_kernel<<<dim3(ceil_div(d.N, 256), d.units), 256, 0, st>>>(d.N, d.kp, a,
                                                                                      scores)));
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
bool make_k_tensormap(CUtensorMap *tm, const void *K, const Dims &d, int rows)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t row_b = (cuuint64_t)d.ks[2] * 2;
    cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows, (cuuint64_t)d.hkv, (cuuint64_t)d.batch};
    cuuint64_t head_b = (cuuint64_t)d.ks[1] * 2, batch_b = (cuuint64_t)d.ks[0] * 2;
    if (d.hkv == 1 || head_b == 0) head_b = row_b * (cuuint64_t)rows;
    if (d.batch == 1 || batch_b == 0) batch_b = head_b * (cuuint64_t)d.hkv;
    cuuint64_t strides[3] = {row_b, head_b, batch_b};
    cuuint32_t box[4] = {64, (cuuint32_t)tc::kTileKeys, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(K), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int env_int(const char *name, int dflt)
{
    const char *v = getenv(name);
    return v ? atoi(v) : dflt;
}

// Units per launch group: the group's keys should stay in L2 between the two sweeps.
int units_per_group(const Dims &d)
{
    const double mb = (double)d.L * kHeadDim * 2 / 1.0e6;
    int n = (int)(env_int("GRAPHKV_L2_GROUP_MB", 72) / mb);
    if (n < 1) n = 1;
    if (n > d.units) n = d.units;
    return n;
}

template <typename Kern> bool set_smem(Kern k, size_t bytes)
{
    return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

graphkv_status run_score_tc(const Dims &d, const Layout &l, const __nv_bfloat16 *Q,
                            const __nv_bfloat16 *K, float *scores, void *ws, cudaStream_t st)
{
    CUtensorMap tmK;
    if (!make_k_tensormap(&tmK, K, d, d.L)) return GRAPHKV_ERR_CUDA;
    const int row_tiles = d.GW <= 128 ? 1 : 2;
    const int rows_pad = 128 * row_tiles;
    const int stages = row_tiles == 1 ? 5 : 4;
    const size_t smem = tc::score_smem_bytes(rows_pad, stages);
    static bool attr = false;
    if (!attr) {
        const size_t mx = tc::score_smem_bytes(256, 4) > tc::score_smem_bytes(128, 5)
                              ? tc::score_smem_bytes(256, 4) : tc::score_smem_bytes(128, 5);
        if (!set_smem(tc::score_stats_tc<1>, mx) || !set_smem(tc::score_stats_tc<2>, mx) ||
            !set_smem(tc::score_emit_tc<1>, mx) || !set_smem(tc::score_emit_tc<2>, mx))
            return GRAPHKV_ERR_CUDA;
        attr = true;
    }
    float *a = d.kp > 1 ? at<float>(ws, l.a) : scores;
    const int n_sms = 148;
    const int tiles_stats = ceil_div(d.L, tc::kTileKeys), tiles_emit = ceil_div(d.N, tc::kTileKeys);
    const int group = units_per_group(d);
    for (int u0 = 0; u0 < d.units; u0 += group) {
        const int nu = std::min(group, d.units - u0);
        int chunks_s = std::max(1, std::min(n_sms / nu, tiles_stats));
        chunks_s = std::min(chunks_s, l.max_parts / 2);
        const int chunks_e = std::max(1, std::min(n_sms / nu, tiles_emit));
        tc::ScoreTcArgs sa{d, Q, at<float>(ws, l.part), a, at<int>(ws, l.status), u0, chunks_s,
                           tiles_stats, 2 * chunks_s, stages};
        tc::ScoreTcArgs ea = sa;
        ea.chunks = chunks_e;
        ea.n_tiles = tiles_emit;
        if (row_tiles == 1) {
            GKV_LAUNCH("score_stats_tc", st,
                       (tc::score_stats_tc<1><<<dim3(chunks_s, nu), tc::kScoreThreads, smem, st>>>(tmK, sa)));
            GKV_LAUNCH("score_emit_tc", st,
                       (tc::score_emit_tc<1><<<dim3(chunks_e, nu), tc::kScoreThreads, smem, st>>>(tmK, ea)));
        } else {
            GKV_LAUNCH("score_stats_tc", st,
                       (tc::score_stats_tc<2><<<dim3(chunks_s, nu), tc::kScoreThreads, smem, st>>>(tmK, sa)));
            GKV_LAUNCH("score_emit_tc", st,
                       (tc::score_emit_tc<2><<<dim3(chunks_e, nu), tc::kScoreThreads, smem, st>>>(tmK, ea)));
        }
    }
    if (d.kp > 1)
        GKV_LAUNCH("pool_max", st,
                   (pool_max_kernel<<<dim3(ceil_div(d.N, 256), d.units), 256, 0, st>>>(d.N, d.kp, a,
                                                                                      scores)));
    return launch_status();
}

inline graphkv_status run_score_any(const Dims &d, const Layout &l, const __nv_bfloat16 *Q,
                                    const __nv_bfloat16 *K, float *scores, void *ws, cudaStream_t st)
{
    if (env_int("GRAPHKV_FORCE_SIMT", 0)) return run_score(d, l, Q, K, scores, ws, st);
    return run_score_tc(d, l, Q, K, scores, ws, st);
}

// ---- steps (II)+(III) ------------------------------------------------------------------------
template <typename T>
graphkv_status run_propagate(const Dims &d, const Layout &l, const T *K, float *scores,
                             int *src_out, void *ws, cudaStream_t st)
{
    if (d.K_src == 0) return GRAPHKV_OK;
    int *src = src_out ? src_out : at<int>(ws, l.src);
    SelectArgs sa{scores, d.N, d.N, d.K_src, nullptr, src, nullptr};
    GKV_LAUNCH("select_sources", st, (topk_select_kernel<<<d.units, kSelectThreads, 0, st>>>(sa)));
    if (d.T == 0 || d.m == 0) return launch_status();
    float *sims = at<float>(ws, l.sims);
    GKV_LAUNCH("similarity_simt", st,
               (similarity_simt<T><<<dim3(ceil_div(d.N, kSimChunk), d.units), kSimThreads, 0, st>>>(
                   d, K, src, sims)));
    SelectArgs na{sims, d.N, d.N, d.m, src, at<int>(ws, l.nbr_idx), at<float>(ws, l.nbr_e)};
    GKV_LAUNCH("select_neighbors", st,
               (topk_select_kernel<<<d.units * d.K_src, kSelectThreads, 0, st>>>(na)));
    GKV_LAUNCH("decay_rounds", st,
               (decay_rounds_kernel<<<d.units, 256, 0, st>>>(d, at<int>(ws, l.nbr_idx),
                                                             at<float>(ws, l.nbr_e), scores)));
    return launch_status();
}

// ---- step (IV) ---------------------------------------------------------------------------------
graphkv_status run_select_gather(const Dims &d, int elem_bytes, const float *scores, const void *K,
                                 const void *V, void *K_out, void *V_out, int *idx_out,
                                 cudaStream_t st)
{
    SelectArgs sa{scores, d.N, d.N, d.B, nullptr, idx_out, nullptr};
    GKV_LAUNCH("select_budget", st, (topk_select_kernel<<<d.units, kSelectThreads, 0, st>>>(sa)));
    if (K || V) {
        const long long total = (long long)d.units * (d.B + d.W) * (kHeadDim * elem_bytes / 16);
        const int blocks = (int)std::min<long long>((total + kGatherThreads - 1) / kGatherThreads,
                                                    148LL * 16);
        GKV_LAUNCH("gather_rows", st,
                   (gather_rows_kernel<<<blocks, kGatherThreads, 0, st>>>(
                       d, elem_bytes, static_cast<const unsigned char *>(K),
                       static_cast<const unsigned char *>(V), idx_out,
                       static_cast<unsigned char *>(K_out), static_cast<unsigned char *>(V_out))));
    }
    return launch_status();
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
    if (!Qw || !K || !scores || !aligned16(Qw) || !aligned16(K)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->dtype == GRAPHKV_BF16)
        return run_score_any(d, l, static_cast<const __nv_bfloat16 *>(Qw),
                             static_cast<const __nv_bfloat16 *>(K), scores, workspace, st);
    return run_score(d, l, static_cast<const float *>(Qw), static_cast<const float *>(K), scores,
                     workspace, st);
}

graphkv_status graphkv_propagate(const graphkv_params *params, const void *K, float *scores,
                                 int32_t *src_idx_out, void *workspace, size_t workspace_bytes,
                                 void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    if (!K || !scores || !aligned16(K)) return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->dtype == GRAPHKV_BF16)
        return run_propagate(d, l, static_cast<const __nv_bfloat16 *>(K), scores, src_idx_out,
                             workspace, st);
    return run_propagate(d, l, static_cast<const float *>(K), scores, src_idx_out, workspace, st);
}

graphkv_status graphkv_select_gather(const graphkv_params *params, const float *scores,
                                     const void *K, const void *V, void *K_out, void *V_out,
                                     int32_t *idx_out, void *workspace, size_t workspace_bytes,
                                     void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    if (!scores || !idx_out) return GRAPHKV_ERR_INVALID_ARG;
    if ((K == nullptr) != (K_out == nullptr) || (V == nullptr) != (V_out == nullptr))
        return GRAPHKV_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    const int elem = params->dtype == GRAPHKV_BF16 ? 2 : 4;
    return run_select_gather(d, elem, scores, K, V, K_out, V_out, idx_out,
                             static_cast<cudaStream_t>(stream));
}

graphkv_status graphkv_compress(const graphkv_params *params, const void *Qw, const void *K,
                                const void *V, void *K_out, void *V_out, int32_t *idx_out,
                                float *scores_out, void *workspace, size_t workspace_bytes,
                                void *stream)
{
    Dims d;
    graphkv_status rc = resolve(params, &d);
    if (rc != GRAPHKV_OK) return rc;
    if (!Qw || !K || !V || !K_out || !V_out || !idx_out) return GRAPHKV_ERR_INVALID_ARG;
    if (!aligned16(Qw) || !aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return GRAPHKV_ERR_INVALID_ARG;
    const Layout l = layout_of(d);
    if ((rc = check_ws(l, workspace, workspace_bytes)) != GRAPHKV_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *s = scores_out ? scores_out : at<float>(workspace, l.s);
    const int elem = params->dtype == GRAPHKV_BF16 ? 2 : 4;
    if (params->dtype == GRAPHKV_BF16) {
        rc = run_score_any(d, l, static_cast<const __nv_bfloat16 *>(Qw),
                           static_cast<const __nv_bfloat16 *>(K), s, workspace, st);
        if (rc == GRAPHKV_OK)
            rc = run_propagate(d, l, static_cast<const __nv_bfloat16 *>(K), s, nullptr, workspace, st);
    } else {
        rc = run_score(d, l, static_cast<const float *>(Qw), static_cast<const float *>(K), s,
                       workspace, st);
        if (rc == GRAPHKV_OK)
            rc = run_propagate(d, l, static_cast<const float *>(K), s, nullptr, workspace, st);
    }
    if (rc != GRAPHKV_OK) return rc;
    return run_select_gather(d, elem, s, K, V, K_out, V_out, idx_out, st);
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

const char *graphkv_status_string(graphkv_status status)
{
    switch (status) {
        case GRAPHKV_OK: return "ok";
        case GRAPHKV_ERR_INVALID_ARG: return "invalid argument";
        case GRAPHKV_ERR_UNSUPPORTED: return "unsupported configuration";
        case GRAPHKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GRAPHKV_ERR_CUDA: return "CUDA error";
        case GRAPHKV_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
