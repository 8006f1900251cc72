/*
 * graphkv.h -- C ABI of the GraphKV prefill KV-cache compression library (CUDA, sm_100a).
 *
 * GraphKV (paper, Methodology) treats the n prompt tokens of one attention head as graph nodes
 * o_j with importance scores s_j, takes the top-k nodes as sources (Eq. 2), links each source
 * to every node by the cosine similarity of their keys (Eq. 1, Algorithm 1), decays the scores
 * of each source's m most similar neighbours for T rounds (Eq. 3-5, Algorithm 2) and keeps the
 * k_l highest-scoring tokens' K/V (Problem Formulation: K_s^l, V_s^l).  This library runs that
 * path at prefill time for all KV heads of a layer on one GPU, with SnapKV-style
 * observation-window attention as the initial score.
 *
 * Conventions common to every call
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library allocates and
 *     frees nothing; scratch comes from a caller-supplied workspace of at least
 *     graphkv_workspace_bytes(params) bytes, 256-byte aligned.
 *     V, K_out, V_out and idx_out may instead be page-locked host memory that the device can
 *     address (unified addressing: the same pointer): V is read only row by row for the B+W
 *     tokens that are kept, so a cache that lives in host memory needs only Qw and K copied.
 *   - Calls validate their arguments on the host, enqueue kernels on `stream` (a cudaStream_t
 *     passed as void*; NULL = the legacy default stream) and return without synchronising.
 *     The return value reports host-side validation and launch errors only.
 *   - Layout: Qw [batch][n_q_heads][W][D], K and V [batch][n_kv_heads][L][D] with element
 *     strides given in the params (D contiguous, every row 16-byte aligned); L = N + W, rows
 *     [0,N) are the prefix tokens (the graph's nodes), rows [N,L) the observation window.
 *     KV head h serves query heads [h*G, (h+1)*G), G = n_q_heads / n_kv_heads.
 *     Outputs are dense: scores [batch][n_kv_heads][N] fp32, idx [batch][n_kv_heads][B] int32,
 *     K_out / V_out [batch][n_kv_heads][B+W][D] in the input dtype.
 *   - Every top-k keeps exactly k items; equal values are ordered lower index first, so results
 *     are deterministic.
 *   - One workspace serves one call at a time: calls sharing a workspace must be ordered on
 *     one stream.  graphkv_score and graphkv_compress set up every word of it they rely on
 *     (the status word at its head included), whatever it held before; a workspace whose first
 *     use is another call (graphkv_propagate after graphkv_score_knorm, graphkv_select_gather
 *     alone) must be zero-filled once by its owner for graphkv_read_status to mean anything.
 */
#ifndef GRAPHKV_H_
#define GRAPHKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GRAPHKV_OK = 0,
    GRAPHKV_ERR_INVALID_ARG = 1,   /* NULL pointer, size or stride out of range, misalignment   */
    GRAPHKV_ERR_UNSUPPORTED = 2,   /* valid but not implemented (head_dim not 128 or 64, G*W > 256, ...) */
    GRAPHKV_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small                 */
    GRAPHKV_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                          */
    GRAPHKV_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out (read_status only)      */
    GRAPHKV_ERR_BUILTIN_SCRATCH = 6 /* graphkv_score_noalloc: the problem needs more scratch than
                                      the library's built-in array holds                         */
} graphkv_status;

typedef enum { GRAPHKV_BF16 = 0, GRAPHKV_F32 = 1 } graphkv_dtype;
typedef enum { GRAPHKV_POOL_MAX = 0, GRAPHKV_POOL_AVG = 1 } graphkv_pool;
/* What a source node sends to its neighbours (Discussion, "Diversity of Graph Signal"): the decay
 * signal of Eq. 4-5, an enhanced signal (factor 1 + lambda*e), or an evicted signal (the
 * neighbour's score becomes -inf). */
typedef enum { GRAPHKV_SIGNAL_DECAY = 0, GRAPHKV_SIGNAL_ENHANCE = 1, GRAPHKV_SIGNAL_EVICT = 2 } graphkv_signal;
/* Which vectors an edge compares (Discussion, "Exploration of similarity for Graph Edge"). */
typedef enum { GRAPHKV_TENSOR_K = 0, GRAPHKV_TENSOR_V = 1 } graphkv_tensor;

typedef struct {
    int32_t batch;        /* independent sequences (or any independent units sharing the shape)  */
    int32_t n_q_heads;
    int32_t n_kv_heads;   /* must divide n_q_heads                                               */
    int32_t head_dim;     /* D: 128, or 64 (served by the general kernels, not the tensor cores) */
    int32_t seq_len;      /* L = N + W rows present in K and V                                   */
    int32_t window;       /* W >= 1 observation-window rows: queried from, always kept           */
    int32_t budget;       /* B = k_l: prefix tokens kept, 1 <= B <= N; outputs hold B + W rows   */
    int32_t pool_kernel;  /* odd >= 1 (1 = no pooling); 1-D pooling of the initial score         */
    int32_t pool_mode;    /* graphkv_pool: maximum, or mean over pool_kernel positions with zeros
                             outside the row                                                     */
    int32_t topk_nodes;   /* k of Eq. 2: number of source nodes, 0 <= k <= N (0: no propagation) */
    int32_t neighbors;    /* m of Eq. 3; 0 = adaptive: clamp(floor(N/1000), 1, 32), at most N-1  */
    int32_t rounds;       /* T of Eq. 5, >= 0; 0 = the base method's plain top-B                 */
    float   decay;        /* lambda in [0,1], the strength in Eq. 4: factor (1 - lambda*e_ij)    */
    int32_t dtype;        /* graphkv_dtype of Qw, K, V, K_out, V_out                             */
    int64_t q_stride[3];  /* element strides of Qw: batch, head, row                             */
    int64_t k_stride[3];  /* element strides of K: batch, head, token                            */
    int64_t v_stride[3];  /* element strides of V: batch, head, token                            */
    int32_t signal;       /* graphkv_signal; 0 = the decay signal of Eq. 4-5                     */
    int32_t reselect;     /* 0: the graph is built once and reused by all T rounds (Algorithm 2);
                             1: every round re-picks the sources from the current scores and
                             rebuilds their neighbourhoods (1 + T sweeps of the keys)            */
} graphkv_params;

/* Bytes of scratch any of the calls below needs for these params; 0 if the params are invalid
 * or unsupported.  Pure host function. */
size_t graphkv_workspace_bytes(const graphkv_params *params);

/* The neighbour count m the library uses for a prefix of n_prefix tokens when
 * params.neighbors = `neighbors` (the paper's "Effect of Adjacent Nodes": the smaller of a
 * preset value and a length-derived one; the length rule is input length x 1e-3). */
int32_t graphkv_resolve_neighbors(int32_t n_prefix, int32_t neighbors);

/* Step (I) of the pipeline figure, "Initiate Importance Score", with the SnapKV-style score the
 * paper's Sparse Graph Building section names as one admissible initialisation:
 *   logits q.k/sqrt(D) of the G*W window rows of each KV head against the prefix keys and the
 *   causally visible window keys; row softmax; sum over rows and grouped heads of the prefix
 *   columns; max pooling with pool_kernel.
 * Reads Qw, K.  Writes scores [batch][n_kv_heads][N] fp32.  Uses topk/decay fields: none. */
graphkv_status graphkv_score(const graphkv_params *params, const void *Qw, const void *K,
                             float *scores, void *workspace, size_t workspace_bytes,
                             void *stream);

/* graphkv_score for callers that cannot provide a workspace.  (The paper has no counterpart: this
 * entry point exists for the way some programs embed the library.)
 *
 * Who needs it: code that runs where device memory may not be allocated -- inside a region that
 * a framework has closed to cudaMalloc (its caching allocator is being recorded or is locked),
 * in a hook or callback invoked from such a region, or in a process whose memory budget was
 * handed out in full at start-up.  Such callers still own Qw, K and the `scores` output, but
 * have nowhere to get the scratch that graphkv_score takes as `workspace`.
 *
 * What it does: the same kernels as graphkv_score, with the scratch (status word, per-chunk
 * softmax statistics, row constants, the attention mass before pooling) placed in an array that
 * is part of the library image: GRAPHKV_BUILTIN_SCRATCH_BYTES bytes of device memory that every
 * GPU loading the library holds until the process exits.  It calls no cudaMalloc, cudaFree or
 * allocating library routine.  Results are bit-identical to graphkv_score.
 *
 * Limits and rules:
 *   - graphkv_builtin_scratch_needed(params) must not exceed GRAPHKV_BUILTIN_SCRATCH_BYTES;
 *     otherwise nothing is launched and GRAPHKV_ERR_BUILTIN_SCRATCH is returned (for bf16
 *     inputs with pooling the need is about 4 * batch * n_kv_heads * N bytes plus 1.5 MB).
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps what the last call left: the call
 *     clears the words that must start at zero itself, but two calls whose kernels overlap on
 *     the GPU (different streams, no ordering between them) race on it.  Order them.
 *   - The device-side status word lives in the array too: graphkv_read_status_noalloc(stream)
 *     reads it.  */
#define GRAPHKV_BUILTIN_SCRATCH_BYTES (16u << 20)
size_t graphkv_builtin_scratch_needed(const graphkv_params *params);
graphkv_status graphkv_score_noalloc(const graphkv_params *params, const void *Qw, const void *K,
                                     float *scores, void *stream);
graphkv_status graphkv_read_status_noalloc(void *stream);

/* Another initial score for step (I): KNorm (Experimental Setup, baseline methods: the L2 norm of
 * the keys; the cited method keeps the keys of lowest norm).  Writes s_j = 1 / max(||k_j||, 1e-12)
 * for the prefix keys, scores [batch][n_kv_heads][N] fp32: the ranking of ascending norm, as
 * positive scores (which the multiplicative decay needs).  One pass over K; no workspace.  Feed
 * the result to graphkv_propagate and graphkv_select_gather like any other initial score. */
graphkv_status graphkv_score_knorm(const graphkv_params *params, const void *K, float *scores,
                                   void *stream);

/* Steps (II)+(III), "Build Graph" and "Decay Signal Propagation" (Eq. 1-5, Algorithms 1-2):
 * sources = top-k of `scores`; e_ij = cosine(k_i, k_j) for each source i and every prefix j != i;
 * N(o_i) = the m largest e_ij; then T times s_j <- s_j * prod_{i: j in N(o_i)} (1 - lambda*max(e_ij,0)).
 * The graph is built once from the incoming scores and reused by all rounds.
 * `scores` is updated in place.  src_idx_out (optional, [batch][n_kv_heads][k] int32) receives
 * the source nodes in ascending position.  With topk_nodes = 0, rounds = 0 or N = 1 the scores
 * are left unchanged. */
graphkv_status graphkv_propagate(const graphkv_params *params, const void *K, float *scores,
                                 int32_t *src_idx_out, void *workspace, size_t workspace_bytes,
                                 void *stream);

/* graphkv_propagate with other edges (Discussion, "Exploration of similarity for Graph Edge"):
 * e_ij = cosine(x_i, y_j) with x the source node's row of tensor `src_tensor` and y the rows of
 * tensor `all_tensor` (graphkv_tensor: K or V, with the strides the params give for it).  K/K is
 * Eq. 1 and what graphkv_propagate computes; V/V and K/V are the value-to-value and key-to-value
 * variants.  The two arguments are operands only: a caller that still holds the query vectors of
 * every token (one vector per KV head and token, laid out like V: e.g. the mean over the head's
 * query group) passes them as `V` to get query-to-key or query-to-query edges.  A tensor that is
 * not used may be NULL. */
graphkv_status graphkv_propagate_edges(const graphkv_params *params, const void *K, const void *V,
                                       int32_t src_tensor, int32_t all_tensor, float *scores,
                                       int32_t *src_idx_out, void *workspace,
                                       size_t workspace_bytes, void *stream);

/* Step (IV), "Select Important Tokens": per head the B highest scores (ties: lower index),
 * written to idx_out in ascending position, and the compact cache
 *   K_out[b][h][0:B] = K[b][h][idx], K_out[b][h][B:B+W] = K[b][h][N:L]   (same for V),
 * copied bit for bit.  K/K_out or V/V_out may be NULL together to skip that tensor;
 * idx_out is required. */
graphkv_status graphkv_select_gather(const graphkv_params *params, const float *scores,
                                     const void *K, const void *V, void *K_out, void *V_out,
                                     int32_t *idx_out, void *workspace, size_t workspace_bytes,
                                     void *stream);

/* The whole path (I)-(IV) in one call.  scores_out (optional, [batch][n_kv_heads][N] fp32)
 * receives the final scores s^(T). */
graphkv_status graphkv_compress(const graphkv_params *params, const void *Qw, const void *K,
                                const void *V, void *K_out, void *V_out, int32_t *idx_out,
                                float *scores_out, void *workspace, size_t workspace_bytes,
                                void *stream);

/* graphkv_compress for several layers (or sequences) of one shape with a budget each: the
 * layer-specific k_l of the Problem Formulation, e.g. PyramidKV's budgets that shrink with depth.
 * The batch dimension of the params enumerates the layers: layer i's Qw, K and V start i batch
 * strides after the base pointers (a cache kept as one [layers][heads][L][D] allocation), and
 * budgets[i] (a HOST array of params.batch entries, 1 <= budgets[i] <= params.budget) is its
 * budget.  params.budget is the row capacity of the outputs: K_out / V_out are
 * [batch][n_kv_heads][budget + W][D] and idx_out [batch][n_kv_heads][budget]; layer i fills its
 * first budgets[i] (+ W) rows and leaves the rest untouched.  All layers run in one set of
 * launches.  At most 64 layers per call (GRAPHKV_ERR_UNSUPPORTED beyond). */
graphkv_status graphkv_compress_layers(const graphkv_params *params, const int32_t *budgets,
                                       const void *Qw, const void *K, const void *V, void *K_out,
                                       void *V_out, int32_t *idx_out, float *scores_out,
                                       void *workspace, size_t workspace_bytes, void *stream);

/* Decode-side micro-benchmark support (Efficiency Analysis: the paper's latency table is decoding
 * latency; this is the attention of one decoding step over a cache, full or compact):
 *   out[b][hq][:] = sum_j softmax_j(q[b][hq] . K[b][h][j] / sqrt(D)) * V[b][h][j],  h = hq / G,
 * over params->seq_len rows of K and V per KV head (no mask: every cached row is visible to the
 * new token).  q [batch][n_q_heads][D] with q_stride[0], q_stride[1]; K, V with k_stride,
 * v_stride; out [batch][n_q_heads][D] fp32, dense.  Of the params only batch, n_q_heads,
 * n_kv_heads, head_dim (128), seq_len, dtype and the strides are read; G <= 8.  The cache is read
 * once.  Scratch: graphkv_decode_workspace_bytes(params) bytes. */
size_t graphkv_decode_workspace_bytes(const graphkv_params *params);
graphkv_status graphkv_decode_attention(const graphkv_params *params, const void *q, const void *K,
                                        const void *V, float *out, void *workspace,
                                        size_t workspace_bytes, void *stream);

/* Synchronises `stream` and returns the status word kernels keep at the head of the workspace
 * (GRAPHKV_OK unless a bounded device-side wait ran out or a CUDA error surfaced).  The only
 * call that blocks the host. */
graphkv_status graphkv_read_status(const void *workspace, void *stream);

const char *graphkv_status_string(graphkv_status status);

/* ---- diagnostics (the paper has no counterpart: inspection support of this library) -----------
 * graphkv_read_neighbors: copies the neighbourhoods N(o_i) of Eq. 3 that the last graphkv_propagate
 * or graphkv_compress on this workspace built, as they were applied by the decay rounds:
 *   nbr_idx_out [batch][n_kv_heads][k][m] int32  positions of each source's m neighbours
 *   nbr_e_out   [batch][n_kv_heads][k][m] fp32   their cosines e_ij
 * (device pointers; either may be NULL), row i of a head belonging to the i-th source in the
 * order graphkv_propagate reports the sources (ascending position); the order within a row
 * carries no meaning.  m = graphkv_resolve_neighbors(N, params.neighbors).
 * The copies are enqueued on `stream` after that call; `params` must be the ones it was given.
 * Returns GRAPHKV_ERR_INVALID_ARG when those params build no graph (topk_nodes, rounds or m zero). */
graphkv_status graphkv_read_neighbors(const graphkv_params *params, const void *workspace,
                                      size_t workspace_bytes, int32_t *nbr_idx_out,
                                      float *nbr_e_out, void *stream);

/* ---- tracing (the paper has no counterpart: measurement support of this library) -------------
 * graphkv_launch_count: kernels this process has launched through the library so far.
 * graphkv_trace_enable(1): from now on every kernel launch is bracketed by a pair of CUDA events
 * recorded on the launch's stream (host-side objects; no device memory).  Off by default.
 * graphkv_trace_read: waits for the recorded events, writes up to `capacity` records (kernel
 * name, device milliseconds) in launch order, forgets all records and returns how many were
 * written.  Not to be called while a traced stream is being captured into a CUDA graph. */
typedef struct {
    char name[40];
    float ms;
} graphkv_trace_record;
int64_t graphkv_launch_count(void);
void graphkv_trace_enable(int32_t enable);
int32_t graphkv_trace_read(graphkv_trace_record *out, int32_t capacity);

/* graphkv_phase_timing_read: only a library built with -DGRAPHKV_PHASE_TIMING keeps, per kernel, the
 * time its CTAs spent between the phase marks in its source (one thread per CTA reads the global
 * timer).  Synchronises the device, copies out and clears the tables:
 *   out[(k * 24 + i) * 2]     nanoseconds summed over CTAs, kernel k, phase i (i = 0: whole CTA)
 *   out[(k * 24 + i) * 2 + 1] the largest single value
 *   out[8 * 24 * 2 + k]       CTAs counted for kernel k
 * `out` is a HOST array of 8 * 24 * 2 + 8 words.  Returns 1, or 0 (nothing written) when the
 * library was built without the option. */
int32_t graphkv_phase_timing_read(uint64_t *out);

#ifdef __cplusplus
}
#endif
#endif /* GRAPHKV_H_ */
