/*
 * GraphKV prefill KV-cache compression -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, fp64 restatement of what the path computes, one (sequence, KV head) unit
 * at a time, taking the steps in the paper's order.  Only tests, the smoke check and the
 * benchmark's cpu-baseline leg may call it.  It shares no code with the CUDA path.
 *
 * Notation (paper, Methodology): n tokens are nodes o_j with scores s_j; keys k_j;
 * e_ij = cosine similarity of keys (Eq. 1); O_source = top-k nodes by score (Eq. 2);
 * N(o_i) = top-m edges of source i, j != i (Eq. 3); decay (Eq. 4-5, Algorithm 2);
 * keep the k_l highest s^(T) (end of "Decay Signal Propagation").
 * Here: N = prefix tokens (the nodes), W = observation window (always kept, never a node),
 * L = N + W key rows, G = query heads per KV head, D = head dim, K_src = k of Eq. 2,
 * m of Eq. 3, T rounds, lambda = decay strength, B = k_l, kp = pooling kernel.
 *
 * Readings where the paper is silent or garbled (kept identical in the CUDA path):
 *   - initial score = SnapKV-style window attention: logits q.k/sqrt(D); row softmax over the
 *     prefix and the causally visible window keys (window key N+r' visible to window row r
 *     iff r' <= r); summed over the W rows and the G grouped heads; prefix columns only;
 *     then 1-D max pooling, stride 1, same length, positions outside [0,N) ignored.
 *   - the coefficient in Eq. 4 / Algorithm 2 line 7 is a scalar lambda: factor (1 - lambda*e_ij);
 *     lambda = 1 gives Eq. 5 as printed.  Negative cosines are clamped to 0.
 *   - the graph is built once (Algorithm 1) and reused by all T rounds (Algorithm 2).
 *   - decays from several sources multiply (Eq. 5), sources may decay each other (only j = i
 *     is excluded by Eq. 3).
 *   - every top-k (sources, neighbours, final budget) keeps exactly k items; equal values are
 *     ordered by lower index first.  Ranking decisions compare fp32 values (the precision the
 *     library's score arrays have); all arithmetic is fp64.
 *   - zero-norm keys: norms are floored at 1e-12, so e = 0.  A computed cosine is clipped to
 *     [-1, 1] (its mathematical range), so with lambda <= 1 a factor is never negative.
 *   - kept prefix rows are emitted in ascending position, followed by the W window rows.
 *
 * Parity pins (tests marked "not gpu"): brute-force numpy softmax attention, the closed form
 * for all-zero queries, pooling of single spikes, numpy normalised matmul for edges,
 * T = 0 / lambda = 0 identities, the s * f^T closed form, argsort brute force for selection.
 * Parity unpinned: the numeric defaults (lambda = 1, the adaptive m rule and its cap 32,
 * K_src) -- the paper prints no value and no worked example for them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim;
    int32_t seq_len;     /* L = N + W */
    int32_t window;      /* W */
    int32_t budget;      /* B */
    int32_t pool_kernel; /* kp, odd */
    int32_t topk_nodes;  /* K_src */
    int32_t neighbors;   /* m; 0 = adaptive */
    int32_t rounds;      /* T */
    double  decay;       /* lambda */
    int32_t pool_mode;   /* 0 = max pooling, 1 = mean over kp positions, zeros outside the row */
    int32_t signal;      /* 0 = decay (Eq. 4-5), 1 = enhanced (1 + lambda e), 2 = evicted (-inf) */
    int32_t reselect;    /* 1 = sources and neighbourhoods rebuilt before every round */
} okv_params;

/* ---- adaptive neighbour count: "input length x 1e-3", floored, kept within [1, 32] ---- */
int32_t okv_resolve_neighbors(int32_t n_prefix, int32_t neighbors)
{
    if (neighbors > 0) return neighbors;
    int32_t m = n_prefix / 1000;
    if (m < 1) m = 1;
    if (m > 32) m = 32;
    if (m > n_prefix - 1) m = n_prefix - 1;
    return m;
}

/* ---- exact top-k with the lower index winning ties -------------------------------------
 * Returns the k indices of x[0..n) with the largest values (index `skip` is not a candidate
 * when skip >= 0), ordered by (value descending, index ascending). */
typedef struct { float v; int32_t i; } okv_item;

static int okv_item_cmp(const void *pa, const void *pb)
{
    const okv_item *a = (const okv_item *)pa, *b = (const okv_item *)pb;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->i > b->i) - (a->i < b->i);
}

void okv_topk(const float *x, int32_t n, int32_t k, int32_t skip, int32_t *idx_out)
{
    okv_item *it = (okv_item *)malloc((size_t)(n > 0 ? n : 1) * sizeof(okv_item));
    int32_t c = 0;
    for (int32_t j = 0; j < n; ++j) {
        if (j == skip) continue;
        it[c].v = x[j];
        it[c].i = j;
        ++c;
    }
    qsort(it, (size_t)c, sizeof(okv_item), okv_item_cmp);
    for (int32_t t = 0; t < k && t < c; ++t) idx_out[t] = it[t].i;
    free(it);
}

/* ---- step (I): SnapKV-style window-attention score of one KV head -----------------------
 * Qg [G][W][D], Kh [L][D] (exact input values widened to fp32).
 * a_out (optional) [N] fp64: attention mass before pooling.  s_out [N] fp32: pooled score. */
void okv_score_unit(const float *Qg, const float *Kh, int32_t G, int32_t W, int32_t D,
                    int32_t N, int32_t kp, int32_t pool_mode, double *a_out, float *s_out)
{
    const int32_t L = N + W;
    double *a = (double *)calloc((size_t)N, sizeof(double));
    double *l = (double *)malloc((size_t)L * sizeof(double));
    const double inv_sqrt_d = 1.0 / sqrt((double)D);
    for (int32_t g = 0; g < G; ++g) {
        for (int32_t r = 0; r < W; ++r) {
            const float *q = Qg + ((size_t)g * W + r) * D;
            const int32_t visible = N + r + 1;          /* keys 0 .. N+r */
            double mx = -INFINITY;
            for (int32_t j = 0; j < visible; ++j) {
                const float *k = Kh + (size_t)j * D;
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d) acc += (double)q[d] * (double)k[d];
                l[j] = acc * inv_sqrt_d;
                if (l[j] > mx) mx = l[j];
            }
            double z = 0.0;
            for (int32_t j = 0; j < visible; ++j) {
                l[j] = exp(l[j] - mx);
                z += l[j];
            }
            for (int32_t j = 0; j < N; ++j) a[j] += l[j] / z;   /* prefix columns only */
        }
    }
    const int32_t half = (kp - 1) / 2;
    for (int32_t j = 0; j < N; ++j) {
        int32_t lo = j - half < 0 ? 0 : j - half;
        int32_t hi = j + half > N - 1 ? N - 1 : j + half;
        double best = a[lo];
        if (pool_mode == 1) {
            /* mean pooling as the common SnapKV implementations do it: zeros outside the row,
             * divided by the kernel size */
            for (int32_t t = lo + 1; t <= hi; ++t) best += a[t];
            best /= (double)kp;
        } else {
            for (int32_t t = lo + 1; t <= hi; ++t)
                if (a[t] > best) best = a[t];
        }
        s_out[j] = (float)best;
    }
    if (a_out) memcpy(a_out, a, (size_t)N * sizeof(double));
    free(a);
    free(l);
}

/* ---- another initial score: KNorm (Experimental Setup, baselines: "applies L2 norm of keys") ----
 * The cited method keeps the keys of LOWEST L2 norm; the paper gives no formula.  Reading used
 * here: s_j = 1 / max(||k_j||_2, 1e-12), which ranks like ascending norm and is positive, as the
 * multiplicative decay of Eq. 5 needs (a negative score would gain rank under a factor in [0,1]).
 * Kh [L][D]; s_out [N] fp32. */
void okv_score_knorm_unit(const float *Kh, int32_t N, int32_t D, float *s_out)
{
    for (int32_t j = 0; j < N; ++j) {
        const float *k = Kh + (size_t)j * D;
        double n2 = 0.0;
        for (int32_t d = 0; d < D; ++d) n2 += (double)k[d] * (double)k[d];
        double n = sqrt(n2);
        if (n < 1e-12) n = 1e-12;
        s_out[j] = (float)(1.0 / n);
    }
}

/* ---- Eq. 1: edges of one source node to every prefix node ------------------------------
 * e_ij = cosine(S[i], A[j]): S = A = the keys for Eq. 1; keys and values, or values and values,
 * for the other edge kinds of the Discussion. */
void okv_edges2_unit(const float *Sh, const float *Kh, int32_t N, int32_t D, int32_t i, double *e_out)
{
    const float *ki = Sh + (size_t)i * D;
    double ni = 0.0;
    for (int32_t d = 0; d < D; ++d) ni += (double)ki[d] * (double)ki[d];
    ni = sqrt(ni);
    if (ni < 1e-12) ni = 1e-12;
    for (int32_t j = 0; j < N; ++j) {
        const float *kj = Kh + (size_t)j * D;
        double dot = 0.0, nj = 0.0;
        for (int32_t d = 0; d < D; ++d) {
            dot += (double)ki[d] * (double)kj[d];
            nj += (double)kj[d] * (double)kj[d];
        }
        nj = sqrt(nj);
        if (nj < 1e-12) nj = 1e-12;
        double e = dot / (ni * nj);
        if (e > 1.0) e = 1.0;        /* Cauchy-Schwarz: rounding must not push a cosine past 1 */
        if (e < -1.0) e = -1.0;
        e_out[j] = e;
    }
}

void okv_edges_unit(const float *Kh, int32_t N, int32_t D, int32_t i, double *e_out)
{
    okv_edges2_unit(Kh, Kh, N, D, i, e_out);
}

/* ---- steps (II)+(III): sparse graph + T rounds of decay on one KV head ------------------
 * s [N] fp32, updated in place.  forced_src (optional, [K_src]) replaces the top-K_src pick;
 * forced_nbr (optional, [K_src][m]) replaces the top-m pick of each source.
 * Outputs (each optional): src_out [K_src], nbr_out [K_src][m], nbr_e_out [K_src][m] fp64. */
void okv_propagate2_unit(const float *Sh, const float *Kh, int32_t N, int32_t D, float *s, int32_t K_src,
                         int32_t m, int32_t T, double lambda, int32_t signal, const int32_t *forced_src,
                         const int32_t *forced_nbr, int32_t *src_out, int32_t *nbr_out,
                         double *nbr_e_out)
{
    if (K_src <= 0 || m <= 0) return;
    int32_t *src = (int32_t *)malloc((size_t)K_src * sizeof(int32_t));
    int32_t *nbr = (int32_t *)malloc((size_t)K_src * m * sizeof(int32_t));
    double *nbr_e = (double *)malloc((size_t)K_src * m * sizeof(double));
    double *e = (double *)malloc((size_t)N * sizeof(double));
    float *e32 = (float *)malloc((size_t)N * sizeof(float));

    /* Eq. 2 / Algorithm 1: the source nodes, from the scores before any decay */
    if (forced_src) memcpy(src, forced_src, (size_t)K_src * sizeof(int32_t));
    else okv_topk(s, N, K_src, -1, src);

    /* Eq. 1 + Eq. 3: edges of each source, and its top-m neighbourhood (j != i) */
    for (int32_t a = 0; a < K_src; ++a) {
        const int32_t i = src[a];
        okv_edges2_unit(Sh, Kh, N, D, i, e);
        if (forced_nbr) memcpy(nbr + (size_t)a * m, forced_nbr + (size_t)a * m,
                               (size_t)m * sizeof(int32_t));
        else {
            for (int32_t j = 0; j < N; ++j) e32[j] = (float)e[j];
            okv_topk(e32, N, m, i, nbr + (size_t)a * m);
        }
        for (int32_t t = 0; t < m; ++t) nbr_e[(size_t)a * m + t] = e[nbr[(size_t)a * m + t]];
    }

    /* Eq. 5 / Algorithm 2: T rounds over the fixed graph */
    double *cur = (double *)malloc((size_t)N * sizeof(double));
    for (int32_t j = 0; j < N; ++j) cur[j] = (double)s[j];
    for (int32_t t = 0; t < T; ++t) {
        for (int32_t a = 0; a < K_src; ++a) {
            for (int32_t u = 0; u < m; ++u) {
                const int32_t j = nbr[(size_t)a * m + u];
                double eij = nbr_e[(size_t)a * m + u];
                if (eij < 0.0) eij = 0.0;
                if (signal == 2) cur[j] = -INFINITY;                        /* evicted */
                else if (signal == 1) cur[j] = cur[j] * (1.0 + lambda * eij); /* enhanced */
                else cur[j] = cur[j] * (1.0 - lambda * eij);                /* decay, Eq. 5 */
            }
        }
    }
    for (int32_t j = 0; j < N; ++j) s[j] = (float)cur[j];

    if (src_out) memcpy(src_out, src, (size_t)K_src * sizeof(int32_t));
    if (nbr_out) memcpy(nbr_out, nbr, (size_t)K_src * m * sizeof(int32_t));
    if (nbr_e_out) memcpy(nbr_e_out, nbr_e, (size_t)K_src * m * sizeof(double));
    free(cur); free(e32); free(e); free(nbr_e); free(nbr); free(src);
}

void okv_propagate_unit(const float *Kh, int32_t N, int32_t D, float *s, int32_t K_src,
                        int32_t m, int32_t T, double lambda, const int32_t *forced_src,
                        const int32_t *forced_nbr, int32_t *src_out, int32_t *nbr_out,
                        double *nbr_e_out)
{
    okv_propagate2_unit(Kh, Kh, N, D, s, K_src, m, T, lambda, 0, forced_src, forced_nbr, src_out,
                        nbr_out, nbr_e_out);
}

/* The other reading of "dynamically updated ... one or multiple times": every round re-picks the
 * sources from the scores the round before left (as fp32, the precision the score arrays have)
 * and rebuilds their neighbourhoods: T passes of Algorithm 1 + one round of Algorithm 2. */
void okv_propagate_reselect_unit(const float *Sh, const float *Kh, int32_t N, int32_t D, float *s,
                                 int32_t K_src, int32_t m, int32_t T, double lambda, int32_t signal,
                                 int32_t *src_out)
{
    for (int32_t t = 0; t < T; ++t)
        okv_propagate2_unit(Sh, Kh, N, D, s, K_src, m, 1, lambda, signal, NULL, NULL, src_out, NULL, NULL);
}

/* ---- step (IV): keep the B highest scores, ascending position --------------------------- */
static int okv_int_cmp(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

void okv_select_unit(const float *s, int32_t N, int32_t B, int32_t *idx_out)
{
    okv_topk(s, N, B, -1, idx_out);
    qsort(idx_out, (size_t)B, sizeof(int32_t), okv_int_cmp);
}

/* ---- compact cache of one head: kept prefix rows, then the window rows (byte copies) ---- */
void okv_gather_unit(const unsigned char *Xh, int32_t N, int32_t W, size_t row_bytes,
                     const int32_t *idx, int32_t B, unsigned char *out)
{
    for (int32_t t = 0; t < B; ++t)
        memcpy(out + (size_t)t * row_bytes, Xh + (size_t)idx[t] * row_bytes, row_bytes);
    for (int32_t r = 0; r < W; ++r)
        memcpy(out + (size_t)(B + r) * row_bytes, Xh + (size_t)(N + r) * row_bytes, row_bytes);
}

/* ---- decode-side use of a cache: one new token's attention over `rows` cached rows ----------
 * out[g][:] = sum_j softmax_j(q[g].K[j] / sqrt(D)) V[j] for the G query heads of one KV head
 * (no mask: every cached row is visible).  q [G][D], Kh, Vh [rows][D]; out [G][D] fp64. */
void okv_decode_attention_unit(const float *q, const float *Kh, const float *Vh, int32_t G,
                               int32_t rows, int32_t D, double *out)
{
    double *l = (double *)malloc((size_t)rows * sizeof(double));
    const double inv_sqrt_d = 1.0 / sqrt((double)D);
    for (int32_t g = 0; g < G; ++g) {
        double mx = -INFINITY;
        for (int32_t j = 0; j < rows; ++j) {
            double acc = 0.0;
            for (int32_t d = 0; d < D; ++d) acc += (double)q[(size_t)g * D + d] * (double)Kh[(size_t)j * D + d];
            l[j] = acc * inv_sqrt_d;
            if (l[j] > mx) mx = l[j];
        }
        double z = 0.0;
        for (int32_t j = 0; j < rows; ++j) {
            l[j] = exp(l[j] - mx);
            z += l[j];
        }
        for (int32_t d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int32_t j = 0; j < rows; ++j) acc += l[j] * (double)Vh[(size_t)j * D + d];
            out[(size_t)g * D + d] = acc / z;
        }
    }
    free(l);
}

/* ---- whole-layer drivers over contiguous [batch][heads][rows][D] arrays ------------------
 * Units are independent; OpenMP (when compiled in) only spreads units over cores. */
int32_t okv_num_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}

void okv_score(const okv_params *p, const float *Qw, const float *K, float *scores)
{
    const int32_t G = p->n_q_heads / p->n_kv_heads, W = p->window, D = p->head_dim;
    const int32_t L = p->seq_len, N = L - W;
    const int32_t units = p->batch * p->n_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t u = 0; u < units; ++u) {
        const int32_t b = u / p->n_kv_heads, h = u % p->n_kv_heads;
        const float *Qg = Qw + (((size_t)b * p->n_q_heads + (size_t)h * G) * W) * D;
        const float *Kh = K + ((size_t)u * L) * D;
        okv_score_unit(Qg, Kh, G, W, D, N, p->pool_kernel, p->pool_mode, NULL, scores + (size_t)u * N);
    }
}

void okv_propagate(const okv_params *p, const float *K, float *scores, int32_t *src_out)
{
    const int32_t W = p->window, D = p->head_dim, L = p->seq_len, N = L - W;
    const int32_t units = p->batch * p->n_kv_heads;
    const int32_t m = okv_resolve_neighbors(N, p->neighbors);
    if (p->rounds <= 0 || p->topk_nodes <= 0) {
        /* no propagation; still report the sources Eq. 2 would pick */
        if (src_out && p->topk_nodes > 0)
            for (int32_t u = 0; u < units; ++u)
                okv_topk(scores + (size_t)u * N, N, p->topk_nodes, -1,
                         src_out + (size_t)u * p->topk_nodes);
        return;
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t u = 0; u < units; ++u) {
        const float *Kh = K + ((size_t)u * L) * D;
        int32_t *so = src_out ? src_out + (size_t)u * p->topk_nodes : NULL;
        if (p->reselect)
            okv_propagate_reselect_unit(Kh, Kh, N, D, scores + (size_t)u * N, p->topk_nodes, m, p->rounds,
                                        p->decay, p->signal, so);
        else
            okv_propagate2_unit(Kh, Kh, N, D, scores + (size_t)u * N, p->topk_nodes, m, p->rounds,
                                p->decay, p->signal, NULL, NULL, so, NULL, NULL);
    }
}

void okv_select_gather(const okv_params *p, const float *scores, const unsigned char *K,
                       const unsigned char *V, size_t elem_bytes, unsigned char *K_out,
                       unsigned char *V_out, int32_t *idx_out)
{
    const int32_t W = p->window, D = p->head_dim, L = p->seq_len, N = L - W, B = p->budget;
    const int32_t units = p->batch * p->n_kv_heads;
    const size_t row = (size_t)D * elem_bytes;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t u = 0; u < units; ++u) {
        int32_t *idx = idx_out + (size_t)u * B;
        okv_select_unit(scores + (size_t)u * N, N, B, idx);
        if (K && K_out)
            okv_gather_unit(K + (size_t)u * L * row, N, W, row, idx, B,
                            K_out + (size_t)u * (B + W) * row);
        if (V && V_out)
            okv_gather_unit(V + (size_t)u * L * row, N, W, row, idx, B,
                            V_out + (size_t)u * (B + W) * row);
    }
}

/* Whole path.  Qw/K as fp32 copies of the exact input values drive the arithmetic;
 * K_raw/V_raw are the original bytes (bf16 or fp32) for the bit-exact gather. */
void okv_compress(const okv_params *p, const float *Qw, const float *K,
                  const unsigned char *K_raw, const unsigned char *V_raw, size_t elem_bytes,
                  unsigned char *K_out, unsigned char *V_out, int32_t *idx_out,
                  float *scores_out)
{
    const int32_t N = p->seq_len - p->window;
    const size_t total = (size_t)p->batch * p->n_kv_heads * N;
    float *s = scores_out ? scores_out : (float *)malloc(total * sizeof(float));
    okv_score(p, Qw, K, s);
    okv_propagate(p, K, s, NULL);
    okv_select_gather(p, s, K_raw, V_raw, elem_bytes, K_out, V_out, idx_out);
    if (!scores_out) free(s);
}
