/*
 * slonn_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, CPU-only statement of the SLO-NN inference path of
 * "Dynamic Network Adaptation at Inference" (arxiv 2204.08400): Node-Activator
 * training (Algorithm 1 with the variance-proportional FreeHash sampling of
 * Sec. 3.4) and the SLO-aware forward pass (Fig. 2 steps 1,3,4; Sec. 3.3),
 * plus the two budget rules that feed it (LCAO, Eq. 3; ACLO, Eq. 2 with the
 * Confidence tables of Sec. 3.2).
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call it.  It shares no code with the CUDA library and includes none of its
 * headers.
 *
 * The method is a heuristic (it computes a cheaper function than the dense
 * MLP), so this file follows the algorithm's steps in the paper's order.  No
 * blocking, fusion or re-ordering is applied beyond the summation contract
 * stated below.
 *
 * Two arithmetic modes:
 *   REF64    every dot product is a plain left-to-right fp64 sum.
 *   CANON32  the fp32 summation contract that both this file and the GPU
 *            library promise, so that hash bits (signs of sums) and therefore
 *            active sets can agree bit for bit:
 *              32 fp32 partial sums, all +0;
 *              element j (j = 0..n-1 in order) goes to partial (j / V) mod 32
 *              with acc = fmaf(w[j], x[j], acc);
 *              then a fixed tree: for off = 16,8,4,2,1: acc[p] += acc[p+off]
 *              for p < off;  z = acc[0] + bias.
 *            V = 4 when weights are stored as fp32, 8 when stored as bf16
 *            (dense operand: j is the input index), V = 1 for the
 *            sparse-operand form (j is the position in the id-ascending list
 *            of nonzeros).
 *
 * Pins (tests, CPU only): REF64 against a float64 matrix product; CANON32
 * against hand-worked orderings and exact small-integer sums; the selection
 * against its closed form and brute force; Algorithm 1 against a
 * dict-of-lists restatement on tiny layers; the budget rounding against hand
 * computed counts; sampling against frequencies; the free-hash-node variant
 * against list filtering and the closed-form selection; the confidence measure
 * against scipy's entropy kernels and closed forms, the Confidence tables and
 * the ACLO rule against brute force.  Parity unpinned: nothing in
 * this file; the paper's accuracy and speed-up claims are not reproduced here
 * at all (they need its datasets and trained weights).
 *
 * Weights are passed widened to fp32 (bf16 -> fp32 is exact); V tells which
 * storage width the summation contract refers to.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_LAYERS 16
#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_BUDGET (-2)
#define ORC_ERR_NOMEM (-3)

enum { ORC_CANON32 = 0, ORC_REF64 = 1 };

/* ------------------------------------------------------------------ */
/* Dot products                                                        */
/* ------------------------------------------------------------------ */

/* CANON32 (see header).  w and x are the operand lists in contract order. */
float orc_dot_canon32(const float *w, const float *x, uint64_t n, uint32_t V, float bias)
{
    float acc[32];
    for (int p = 0; p < 32; ++p) acc[p] = 0.0f;
    for (uint64_t j = 0; j < n; ++j) {
        uint32_t p = (uint32_t)((j / V) % 32u);
        acc[p] = fmaf(w[j], x[j], acc[p]);
    }
    for (int off = 16; off >= 1; off >>= 1)
        for (int p = 0; p < off; ++p) acc[p] = acc[p] + acc[p + off];
    return acc[0] + bias;
}

/* REF64: the plain definition  z = sum_j w_j x_j + b  in fp64, j ascending. */
double orc_dot_ref64(const float *w, const double *x, uint64_t n, float bias)
{
    double s = 0.0;
    for (uint64_t j = 0; j < n; ++j) s += (double)w[j] * x[j];
    return s + (double)bias;
}

/* k% -> node count: nearest whole node, never fewer than one
 * (Sec. 3.2, latency-profile paragraph).  bp = budget in basis points. */
uint32_t orc_budget_nodes(uint32_t bp, uint32_t N)
{
    uint64_t b = ((uint64_t)bp * N + 5000u) / 10000u;
    if (b < 1) b = 1;
    if (b > N) b = N;
    return (uint32_t)b;
}

/* SplitMix64 (Steele, Lea, Flood 2014): state advances by the golden gamma,
 * output is the finalising mix of the new state. */
static uint64_t splitmix64_next(uint64_t *state)
{
    uint64_t z = (*state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
uint64_t orc_splitmix64(uint64_t *state) { return splitmix64_next(state); }

/* ------------------------------------------------------------------ */
/* Model                                                               */
/* ------------------------------------------------------------------ */

typedef struct orc_model {
    uint32_t n_layers;
    uint32_t dims[ORC_MAX_LAYERS + 1]; /* D0, N1, ..., N_out */
    uint8_t has_act[ORC_MAX_LAYERS];
    uint32_t V;            /* 4: fp32 storage, 8: bf16 storage */
    uint32_t K, L;         /* key bits per table, number of tables */
    uint32_t list_cap;     /* 0 => full permutation */
    int first_sparse;      /* layer 0 takes a sparse operand (id-ascending list) */
    int free_hash_nodes;   /* variant of Sec. 3.4: the K*L hash nodes of a layer are always part of
                            * its active set (their pre-activations are computed for the keys anyway)
                            * and never appear in its ranked lists; the budget counts list nodes only */
    const float *W[ORC_MAX_LAYERS];    /* row-major [N_l][D_l], referenced */
    const float *bias[ORC_MAX_LAYERS]; /* [N_l], referenced */
    uint32_t *hash_nodes[ORC_MAX_LAYERS]; /* [L*K]; draw b*K+j = function j of table b */
    uint32_t *rank[ORC_MAX_LAYERS];       /* [L][2^K][cap_l] node ids, most important first */
    uint32_t cap[ORC_MAX_LAYERS];
    double *var[ORC_MAX_LAYERS];          /* [N_l] activation variance (kept for tests) */
    double *score[ORC_MAX_LAYERS];        /* [L][2^K][N_l] NodeScore, kept only if asked */
    uint32_t *bucket_count[ORC_MAX_LAYERS]; /* [L][2^K] calibration samples per bucket */
    int keep_scores;
} orc_model;

orc_model *orc_model_new(uint32_t n_layers, const uint32_t *dims, const uint8_t *has_act,
                         uint32_t V, uint32_t K, uint32_t L, uint32_t list_cap, int first_sparse)
{
    if (n_layers < 1 || n_layers > ORC_MAX_LAYERS) return NULL;
    if (K < 1 || K > 16 || L < 1 || L > 8) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    if (!m) return NULL;
    m->n_layers = n_layers;
    for (uint32_t i = 0; i <= n_layers; ++i) m->dims[i] = dims[i];
    for (uint32_t i = 0; i < n_layers; ++i) m->has_act[i] = has_act[i];
    m->V = V; m->K = K; m->L = L; m->list_cap = list_cap; m->first_sparse = first_sparse;
    return m;
}

void orc_model_set_layer(orc_model *m, uint32_t l, const float *W, const float *bias)
{
    m->W[l] = W; m->bias[l] = bias;
}

void orc_model_keep_scores(orc_model *m, int keep) { m->keep_scores = keep; }
void orc_model_set_free_hash_nodes(orc_model *m, int on) { m->free_hash_nodes = on; }

/* Nodes computed in a layer of N nodes at budget bp: the budget's node count, and in the
 * free-hash-node variant that many list nodes (at most the N - K*L non-hash nodes) plus the
 * K*L hash nodes. */
uint32_t orc_layer_nodes(const orc_model *m, uint32_t bp, uint32_t N)
{
    const uint32_t B = orc_budget_nodes(bp, N);
    if (!m->free_hash_nodes) return B;
    const uint32_t H = m->K * m->L;
    const uint32_t rest = N - H;
    return (B < rest ? B : rest) + H;
}

void orc_model_free(orc_model *m)
{
    if (!m) return;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        free(m->hash_nodes[l]); free(m->rank[l]); free(m->var[l]);
        free(m->score[l]); free(m->bucket_count[l]);
    }
    free(m);
}

const uint32_t *orc_model_hash_nodes(const orc_model *m, uint32_t l) { return m->hash_nodes[l]; }
const uint32_t *orc_model_rank(const orc_model *m, uint32_t l) { return m->rank[l]; }
uint32_t orc_model_cap(const orc_model *m, uint32_t l) { return m->cap[l]; }
const double *orc_model_var(const orc_model *m, uint32_t l) { return m->var[l]; }
const double *orc_model_score(const orc_model *m, uint32_t l) { return m->score[l]; }
const uint32_t *orc_model_bucket_count(const orc_model *m, uint32_t l) { return m->bucket_count[l]; }

/* Install hash nodes and tables made elsewhere (tests that hand-build a model). */
int orc_model_set_tables(orc_model *m, uint32_t l, const uint32_t *hash_nodes,
                         const uint32_t *rank, uint32_t cap)
{
    uint32_t H = m->K * m->L;
    uint64_t nent = (uint64_t)m->L * ((uint64_t)1 << m->K) * cap;
    free(m->hash_nodes[l]); free(m->rank[l]);
    m->hash_nodes[l] = (uint32_t *)malloc(sizeof(uint32_t) * H);
    m->rank[l] = (uint32_t *)malloc(sizeof(uint32_t) * nent);
    if (!m->hash_nodes[l] || !m->rank[l]) return ORC_ERR_NOMEM;
    memcpy(m->hash_nodes[l], hash_nodes, sizeof(uint32_t) * H);
    memcpy(m->rank[l], rank, sizeof(uint32_t) * nent);
    m->cap[l] = cap;
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* One layer, one node, one query                                      */
/* ------------------------------------------------------------------ */

static inline int is_last(const orc_model *m, uint32_t l) { return l + 1 == m->n_layers; }

/* Hidden layers use ReLU (never returns -0); the last layer is the identity. */
static inline float act32(const orc_model *m, uint32_t l, float z)
{
    if (is_last(m, l)) return z;
    return z > 0.0f ? z : 0.0f;
}
static inline double act64(const orc_model *m, uint32_t l, double z)
{
    if (is_last(m, l)) return z;
    return z > 0.0 ? z : 0.0;
}

/* Pre-activation of node n of layer l for a dense input vector (CANON32). */
static float node_z32_dense(const orc_model *m, uint32_t l, uint32_t n, const float *in)
{
    uint32_t D = m->dims[l];
    return orc_dot_canon32(m->W[l] + (uint64_t)n * D, in, D, m->V, m->bias[l][n]);
}
static double node_z64_dense(const orc_model *m, uint32_t l, uint32_t n, const double *in)
{
    uint32_t D = m->dims[l];
    return orc_dot_ref64(m->W[l] + (uint64_t)n * D, in, D, m->bias[l][n]);
}

/* Sparse operand (layer 0 only): the operand lists are the nonzeros in
 * id-ascending order, V = 1. */
static float node_z32_sparse(const orc_model *m, uint32_t n, const uint32_t *ids,
                             const float *vals, uint32_t nnz, float *wtmp)
{
    uint32_t D = m->dims[0];
    for (uint32_t j = 0; j < nnz; ++j) wtmp[j] = m->W[0][(uint64_t)n * D + ids[j]];
    return orc_dot_canon32(wtmp, vals, nnz, 1, m->bias[0][n]);
}
static double node_z64_sparse(const orc_model *m, uint32_t n, const uint32_t *ids,
                              const float *vals, uint32_t nnz)
{
    uint32_t D = m->dims[0];
    double s = 0.0;
    for (uint32_t j = 0; j < nnz; ++j)
        s += (double)m->W[0][(uint64_t)n * D + ids[j]] * (double)vals[j];
    return s + (double)m->bias[0][n];
}

/* ------------------------------------------------------------------ */
/* BUILD: Algorithm 1 + FreeHash sampling (Sec. 3.4)                   */
/* ------------------------------------------------------------------ */

typedef struct { const double *score; } sort_ctx;

/* "highest to lowest" activation sum; equal sums: lower node id first. */
static int cmp_rank(const void *pa, const void *pb, void *vctx)
{
    const sort_ctx *c = (const sort_ctx *)vctx;
    uint32_t a = *(const uint32_t *)pa, b = *(const uint32_t *)pb;
    double sa = c->score[a], sb = c->score[b];
    if (sa > sb) return -1;
    if (sa < sb) return 1;
    return (a < b) ? -1 : (a > b) ? 1 : 0;
}

/* Draw H distinct nodes with probability proportional to var (Sec. 3.4):
 * sequentially, without replacement, by inverse CDF over the remaining
 * weights in id order.  When no positive weight remains the draw is uniform
 * over the remaining nodes. */
void orc_sample_hash_nodes(const double *var, uint32_t N, uint32_t H, uint64_t seed,
                           uint32_t layer, uint32_t *out)
{
    uint8_t *taken = (uint8_t *)calloc(N, 1);
    uint64_t state = seed ^ (0xD6E8FEB86659FD93ull * (uint64_t)(layer + 1));
    for (uint32_t d = 0; d < H; ++d) {
        double u = (double)(splitmix64_next(&state) >> 11) * (1.0 / 9007199254740992.0);
        double total = 0.0;
        uint32_t remaining = 0;
        for (uint32_t i = 0; i < N; ++i)
            if (!taken[i]) { total += var[i]; ++remaining; }
        uint32_t pick = N;
        if (total > 0.0) {
            double t = u * total, c = 0.0;
            uint32_t last_pos = N;
            for (uint32_t i = 0; i < N; ++i) {
                if (taken[i] || !(var[i] > 0.0)) continue;
                c += var[i];
                last_pos = i;
                if (c > t) { pick = i; break; }
            }
            if (pick == N) pick = last_pos; /* rounding left c <= t at the end */
        } else {
            uint32_t idx = (uint32_t)(u * (double)remaining);
            if (idx >= remaining) idx = remaining - 1;
            for (uint32_t i = 0; i < N; ++i) {
                if (taken[i]) continue;
                if (idx == 0) { pick = i; break; }
                --idx;
            }
        }
        taken[pick] = 1;
        out[d] = pick;
    }
    free(taken);
}

/* Train the Node-Importance tables of layer l from the full activations
 * A [n_cal][N] of that layer on the calibration set. */
static int train_layer_tables(orc_model *m, uint32_t l, const float *A, uint32_t n_cal,
                              uint64_t seed, const uint32_t *hash_override)
{
    const uint32_t N = m->dims[l + 1], K = m->K, L = m->L, H = K * L;
    const uint32_t nb = 1u << K;
    if (H > N) return ORC_ERR_ARG;
    /* lists hold every node, or in the free-hash-node variant every node that is not a hash node */
    const uint32_t listable = m->free_hash_nodes ? N - H : N;
    const uint32_t cap = (m->list_cap == 0 || m->list_cap > listable) ? listable : m->list_cap;

    /* variance of each node's activation over the calibration set (population,
     * two-pass, fp64, sample order) */
    double *mean = (double *)calloc(N, sizeof(double));
    double *var = (double *)calloc(N, sizeof(double));
    if (!mean || !var) return ORC_ERR_NOMEM;
    for (uint32_t x = 0; x < n_cal; ++x)
        for (uint32_t i = 0; i < N; ++i) mean[i] += (double)A[(uint64_t)x * N + i];
    for (uint32_t i = 0; i < N; ++i) mean[i] = mean[i] / (double)n_cal;
    for (uint32_t x = 0; x < n_cal; ++x)
        for (uint32_t i = 0; i < N; ++i) {
            double d = (double)A[(uint64_t)x * N + i] - mean[i];
            var[i] += d * d;
        }
    for (uint32_t i = 0; i < N; ++i) var[i] = var[i] / (double)n_cal;
    free(mean);
    free(m->var[l]); m->var[l] = var;

    /* h := GenerateHashFamily(K, L) */
    free(m->hash_nodes[l]);
    m->hash_nodes[l] = (uint32_t *)malloc(sizeof(uint32_t) * H);
    if (!m->hash_nodes[l]) return ORC_ERR_NOMEM;
    if (hash_override) memcpy(m->hash_nodes[l], hash_override, sizeof(uint32_t) * H);
    else orc_sample_hash_nodes(var, N, H, seed, l, m->hash_nodes[l]);
    const uint32_t *hn = m->hash_nodes[l];

    /* NodeScore[b][key] += Activation, for every sample and table */
    double *score = (double *)calloc((uint64_t)L * nb * N, sizeof(double));
    double *global = (double *)calloc(N, sizeof(double));
    uint32_t *count = (uint32_t *)calloc((uint64_t)L * nb, sizeof(uint32_t));
    if (!score || !global || !count) return ORC_ERR_NOMEM;
    for (uint32_t x = 0; x < n_cal; ++x) {
        const float *a = A + (uint64_t)x * N;
        for (uint32_t b = 0; b < L; ++b) {
            /* key = (h^b_1(x), ..., h^b_K(x)); a FreeHash bit is [z > 0]; for
             * ReLU layers z > 0 <=> a > 0 and for the identity layer a = z. */
            uint32_t key = 0;
            for (uint32_t j = 0; j < K; ++j)
                if (a[hn[b * K + j]] > 0.0f) key |= (1u << j);
            double *s = score + ((uint64_t)b * nb + key) * N;
            for (uint32_t i = 0; i < N; ++i) s[i] += (double)a[i];
            count[b * nb + key] += 1;
        }
        for (uint32_t i = 0; i < N; ++i) global[i] += (double)a[i];
    }

    /* Rank[b][key] := argsort(NodeScore[b][key]), highest first; a bucket no
     * sample reached gets the ranking of the sums over all samples. */
    free(m->rank[l]);
    m->rank[l] = (uint32_t *)malloc(sizeof(uint32_t) * (uint64_t)L * nb * cap);
    uint32_t *glist = (uint32_t *)malloc(sizeof(uint32_t) * N);
    if (!m->rank[l] || !glist) return ORC_ERR_NOMEM;
    uint8_t *is_hash = (uint8_t *)calloc(N, 1);
    if (!is_hash) return ORC_ERR_NOMEM;
    if (m->free_hash_nodes) for (uint32_t h = 0; h < H; ++h) is_hash[hn[h]] = 1;
    for (uint32_t i = 0; i < N; ++i) glist[i] = i;
    { sort_ctx c = { global }; qsort_r(glist, N, sizeof(uint32_t), cmp_rank, &c); }
    int err = ORC_OK;
#pragma omp parallel for schedule(dynamic)
    for (uint32_t bk = 0; bk < L * nb; ++bk) {
        uint32_t *dst = m->rank[l] + (uint64_t)bk * cap;
        const uint32_t *src = glist;
        uint32_t *perm = NULL;
        if (count[bk] != 0) {
            perm = (uint32_t *)malloc(sizeof(uint32_t) * N);
            if (!perm) { err = ORC_ERR_NOMEM; continue; }
            for (uint32_t i = 0; i < N; ++i) perm[i] = i;
            sort_ctx c = { score + (uint64_t)bk * N };
            qsort_r(perm, N, sizeof(uint32_t), cmp_rank, &c);
            src = perm;
        }
        /* the first cap listable nodes of the ranking, in ranking order */
        uint32_t o = 0;
        for (uint32_t i = 0; i < N && o < cap; ++i)
            if (!is_hash[src[i]]) dst[o++] = src[i];
        free(perm);
    }
    free(is_hash);
    free(glist); free(global);
    m->cap[l] = cap;
    free(m->bucket_count[l]); m->bucket_count[l] = count;
    free(m->score[l]); m->score[l] = NULL;
    if (m->keep_scores) m->score[l] = score; else free(score);
    return err;
}

/* Build every activator of the model.  The calibration set plays the role of
 * the paper's LSH training set; Input_l is the complete (100 %) activation of
 * layer l-1 on it.  Calibration is dense [n_cal][D0], or CSR when layer 0
 * takes a sparse operand.  hash_override[l] (nullable) fixes the L*K hash
 * nodes of layer l instead of sampling them. */
int orc_build(orc_model *m, const float *calib_dense, const uint64_t *c_indptr,
              const uint32_t *c_ids, const float *c_vals, uint32_t n_cal, uint64_t seed,
              const uint32_t *const *hash_override)
{
    if (n_cal == 0) return ORC_ERR_ARG;
    if (m->first_sparse ? (!c_indptr || !c_ids || !c_vals) : !calib_dense) return ORC_ERR_ARG;
    uint32_t last_needed = 0;
    int any = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l) if (m->has_act[l]) { last_needed = l; any = 1; }
    if (!any) return ORC_OK;

    float *cur = NULL; /* Input_l, dense [n_cal][D_l]; NULL while it is the caller's array */
    for (uint32_t l = 0; l <= last_needed; ++l) {
        const uint32_t D = m->dims[l], N = m->dims[l + 1];
        float *A = (float *)malloc(sizeof(float) * (uint64_t)n_cal * N);
        if (!A) { free(cur); return ORC_ERR_NOMEM; }
        /* Activation = ForwardProp_l(x), all N nodes */
#pragma omp parallel for schedule(static)
        for (uint32_t x = 0; x < n_cal; ++x) {
            if (l == 0 && m->first_sparse) {
                uint32_t nnz = (uint32_t)(c_indptr[x + 1] - c_indptr[x]);
                float *wtmp = (float *)malloc(sizeof(float) * (nnz ? nnz : 1));
                for (uint32_t n = 0; n < N; ++n)
                    A[(uint64_t)x * N + n] = act32(m, l, node_z32_sparse(m, n, c_ids + c_indptr[x],
                                                   c_vals + c_indptr[x], nnz, wtmp));
                free(wtmp);
            } else {
                const float *in = (l == 0 ? calib_dense : cur) + (uint64_t)x * D;
                for (uint32_t n = 0; n < N; ++n)
                    A[(uint64_t)x * N + n] = act32(m, l, node_z32_dense(m, l, n, in));
            }
        }
        if (m->has_act[l]) {
            int rc = train_layer_tables(m, l, A, n_cal, seed, hash_override ? hash_override[l] : NULL);
            if (rc != ORC_OK) { free(A); free(cur); return rc; }
        }
        free(cur);
        cur = A;
    }
    free(cur);
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* RUN: SLO-aware forward pass (Fig. 2 steps 1, 3, 4; Sec. 3.3)        */
/* ------------------------------------------------------------------ */

/* Active set of one layer for one query: the first B distinct node ids met
 * when the L bucket lists are read rank by rank (rank 0 of table 0, rank 0 of
 * table 1, ..., rank 1 of table 0, ...), then sorted ascending.  B == N means
 * every node.  Returns B, or a negative error. */
static int select_active(const orc_model *m, uint32_t l, const uint32_t *keys, uint32_t B,
                         uint32_t *out_ids, uint8_t *seen /* [N] scratch */)
{
    const uint32_t N = m->dims[l + 1], L = m->L, nb = 1u << m->K, cap = m->cap[l];
    memset(seen, 0, N);
    if (B == N) {
        for (uint32_t i = 0; i < N; ++i) out_ids[i] = i;
        return (int)B;
    }
    if (B > cap) return ORC_ERR_BUDGET;
    uint32_t got = 0;
    for (uint32_t r = 0; r < cap && got < B; ++r)
        for (uint32_t b = 0; b < L && got < B; ++b) {
            uint32_t id = m->rank[l][((uint64_t)b * nb + keys[b]) * cap + r];
            if (!seen[id]) { seen[id] = 1; ++got; }
        }
    if (got < B) return ORC_ERR_BUDGET;
    uint32_t o = 0;
    for (uint32_t i = 0; i < N; ++i) if (seen[i]) out_ids[o++] = i;
    return (int)B;
}

/* The same in the free-hash-node variant: the layer's K*L hash nodes, plus the first
 * min(B, N - K*L) distinct ids of the rank-interleaved lists (which hold no hash node), ascending.
 * Returns the number of ids, or a negative error. */
static int select_active_free(const orc_model *m, uint32_t l, const uint32_t *keys, uint32_t B,
                              uint32_t *out_ids, uint8_t *seen /* [N] scratch */)
{
    const uint32_t N = m->dims[l + 1], L = m->L, nb = 1u << m->K, cap = m->cap[l], H = m->K * m->L;
    const uint32_t want = B < N - H ? B : N - H;
    memset(seen, 0, N);
    for (uint32_t h = 0; h < H; ++h) seen[m->hash_nodes[l][h]] = 1;
    if (want == N - H) {
        for (uint32_t i = 0; i < N; ++i) out_ids[i] = i;
        return (int)N;
    }
    if (want > cap) return ORC_ERR_BUDGET;
    uint32_t got = 0;
    for (uint32_t r = 0; r < cap && got < want; ++r)
        for (uint32_t b = 0; b < L && got < want; ++b) {
            uint32_t id = m->rank[l][((uint64_t)b * nb + keys[b]) * cap + r];
            if (!seen[id]) { seen[id] = 1; ++got; }
        }
    if (got < want) return ORC_ERR_BUDGET;
    uint32_t o = 0;
    for (uint32_t i = 0; i < N; ++i) if (seen[i]) out_ids[o++] = i;
    return (int)o;
}

typedef struct {
    /* inputs */
    uint32_t n_queries;
    const float *x_dense;       /* [n][D0] or NULL */
    const uint64_t *x_indptr;   /* CSR when layer 0 takes a sparse operand */
    const uint32_t *x_ids;
    const float *x_vals;
    const uint16_t *budget_bp;  /* [n] basis points 1..10000 */
    int mode;                   /* ORC_CANON32 | ORC_REF64 */
    uint32_t logit_stride;      /* N_out, or >= max B when the last layer is budgeted */
    /* outputs (each nullable) */
    float *logits32;            /* CANON32: [n][logit_stride] */
    double *logits64;           /* REF64:   [n][logit_stride] */
    uint32_t *logit_ids;        /* [n][logit_stride] when the last layer is budgeted */
    uint32_t *pred;             /* [n] argmax node id, lowest id on ties */
    uint16_t *codes;            /* [n][n_act][L] */
    uint64_t *active_indptr;    /* [n*n_act + 1], filled here */
    uint32_t *active_ids;       /* CSR payload, ids ascending */
    float *active_vals32;       /* CSR payload (CANON32 activations) */
    double *active_vals64;      /* CSR payload (REF64 activations) */
} orc_batch;

static uint32_t count_act_layers(const orc_model *m)
{
    uint32_t c = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l) c += m->has_act[l] ? 1 : 0;
    return c;
}

/* One query through all layers.  The layer input is kept as a dense vector in
 * which every node that was not computed holds exactly 0. */
static int run_query(const orc_model *m, const orc_batch *bt, uint32_t q)
{
    const uint32_t n_act = count_act_layers(m);
    const int ref = (bt->mode == ORC_REF64);
    uint32_t maxw = 0;
    for (uint32_t i = 0; i <= m->n_layers; ++i) if (m->dims[i] > maxw) maxw = m->dims[i];
    float *in32 = (float *)calloc(maxw, sizeof(float)), *out32 = (float *)calloc(maxw, sizeof(float));
    double *in64 = (double *)calloc(maxw, sizeof(double)), *out64 = (double *)calloc(maxw, sizeof(double));
    uint32_t *ids = (uint32_t *)malloc(sizeof(uint32_t) * maxw);
    uint8_t *seen = (uint8_t *)malloc(maxw);
    float *wtmp = NULL;
    uint32_t keys[8];
    int rc = ORC_OK;
    if (!in32 || !out32 || !in64 || !out64 || !ids || !seen) { rc = ORC_ERR_NOMEM; goto done; }

    const uint32_t bp = bt->budget_bp[q];
    if (bp < 1 || bp > 10000) { rc = ORC_ERR_BUDGET; goto done; }

    /* input := x */
    const uint32_t *sp_ids = NULL; const float *sp_vals = NULL; uint32_t nnz = 0;
    if (m->first_sparse) {
        sp_ids = bt->x_ids + bt->x_indptr[q]; sp_vals = bt->x_vals + bt->x_indptr[q];
        nnz = (uint32_t)(bt->x_indptr[q + 1] - bt->x_indptr[q]);
        wtmp = (float *)malloc(sizeof(float) * (nnz ? nnz : 1));
        if (!wtmp) { rc = ORC_ERR_NOMEM; goto done; }
    } else {
        for (uint32_t j = 0; j < m->dims[0]; ++j) {
            in32[j] = bt->x_dense[(uint64_t)q * m->dims[0] + j];
            in64[j] = (double)in32[j];
        }
    }

    uint32_t a = 0; /* index among activator layers */
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const uint32_t N = m->dims[l + 1];
        const int sparse_op = (l == 0 && m->first_sparse);
        uint32_t B = N;
        if (m->has_act[l]) {
            /* (1) FreeHash: bit = [w_h . input + b_h > 0]; key_b = sum_j bit_{b,j} 2^j */
            for (uint32_t b = 0; b < m->L; ++b) {
                uint32_t key = 0;
                for (uint32_t j = 0; j < m->K; ++j) {
                    uint32_t h = m->hash_nodes[l][b * m->K + j];
                    int bit;
                    if (ref) bit = (sparse_op ? node_z64_sparse(m, h, sp_ids, sp_vals, nnz)
                                              : node_z64_dense(m, l, h, in64)) > 0.0;
                    else bit = (sparse_op ? node_z32_sparse(m, h, sp_ids, sp_vals, nnz, wtmp)
                                          : node_z32_dense(m, l, h, in32)) > 0.0f;
                    if (bit) key |= (1u << j);
                }
                keys[b] = key;
                if (bt->codes) bt->codes[((uint64_t)q * n_act + a) * m->L + b] = (uint16_t)key;
            }
            /* (3) ranked lists -> top-k% */
            B = orc_budget_nodes(bp, N);
            int s = m->free_hash_nodes ? select_active_free(m, l, keys, B, ids, seen)
                                       : select_active(m, l, keys, B, ids, seen);
            if (s < 0) { rc = s; goto done; }
            B = (uint32_t)s; /* nodes to compute */
        } else {
            for (uint32_t i = 0; i < N; ++i) ids[i] = i;
        }
        /* (4) compute the selected nodes; everything else is exactly 0 */
        for (uint32_t i = 0; i < N; ++i) { out32[i] = 0.0f; out64[i] = 0.0; }
        for (uint32_t r = 0; r < B; ++r) {
            uint32_t n = ids[r];
            if (ref) out64[n] = act64(m, l, sparse_op ? node_z64_sparse(m, n, sp_ids, sp_vals, nnz)
                                                      : node_z64_dense(m, l, n, in64));
            else out32[n] = act32(m, l, sparse_op ? node_z32_sparse(m, n, sp_ids, sp_vals, nnz, wtmp)
                                                  : node_z32_dense(m, l, n, in32));
        }
        if (m->has_act[l]) {
            uint64_t off = bt->active_indptr ? bt->active_indptr[(uint64_t)q * n_act + a] : 0;
            for (uint32_t r = 0; r < B; ++r) {
                if (bt->active_ids) bt->active_ids[off + r] = ids[r];
                if (bt->active_vals32 && !ref) bt->active_vals32[off + r] = out32[ids[r]];
                if (bt->active_vals64 && ref) bt->active_vals64[off + r] = out64[ids[r]];
            }
            ++a;
        }
        if (is_last(m, l)) {
            /* logits and prediction (argmax, lowest id on ties, over computed nodes) */
            const uint64_t base = (uint64_t)q * bt->logit_stride;
            uint32_t best = ids[0];
            for (uint32_t r = 0; r < B; ++r) {
                uint32_t n = ids[r];
                if (ref ? (out64[n] > out64[best]) : (out32[n] > out32[best])) best = n;
                if (m->has_act[l]) {
                    if (bt->logit_ids) bt->logit_ids[base + r] = n;
                    if (bt->logits32 && !ref) bt->logits32[base + r] = out32[n];
                    if (bt->logits64 && ref) bt->logits64[base + r] = out64[n];
                } else {
                    if (bt->logits32 && !ref) bt->logits32[base + n] = out32[n];
                    if (bt->logits64 && ref) bt->logits64[base + n] = out64[n];
                }
            }
            if (bt->pred) bt->pred[q] = best;
        }
        /* input := Activation */
        float *t32 = in32; in32 = out32; out32 = t32;
        double *t64 = in64; in64 = out64; out64 = t64;
    }
done:
    free(in32); free(out32); free(in64); free(out64); free(ids); free(seen); free(wtmp);
    return rc;
}

/* Run a batch.  Queries are independent; they are spread over the host's
 * threads, which changes no query's arithmetic. */
int orc_run(const orc_model *m, const orc_batch *bt)
{
    const uint32_t n_act = count_act_layers(m);
    if (m->first_sparse ? (!bt->x_indptr || !bt->x_ids || !bt->x_vals) : !bt->x_dense) return ORC_ERR_ARG;
    if (!bt->budget_bp) return ORC_ERR_ARG;
    if (bt->active_indptr) {
        uint64_t off = 0;
        for (uint32_t q = 0; q < bt->n_queries; ++q) {
            uint32_t a = 0;
            for (uint32_t l = 0; l < m->n_layers; ++l) {
                if (!m->has_act[l]) continue;
                bt->active_indptr[(uint64_t)q * n_act + a] = off;
                off += orc_layer_nodes(m, bt->budget_bp[q], m->dims[l + 1]);
                ++a;
            }
        }
        bt->active_indptr[(uint64_t)bt->n_queries * n_act] = off;
    }
    int err = ORC_OK;
#pragma omp parallel for schedule(dynamic, 16)
    for (uint32_t q = 0; q < bt->n_queries; ++q) {
        int rc = run_query(m, bt, q);
        if (rc != ORC_OK) {
#pragma omp critical
            err = rc;
        }
    }
    return err;
}

/* Thread count the batch loop will use (for the benchmark's report). */
#ifdef _OPENMP
#include <omp.h>
int orc_threads(void) { return omp_get_max_threads(); }
#else
int orc_threads(void) { return 1; }
#endif

/* ------------------------------------------------------------------ */
/* LCAO budget choice (Sec. 2.3, Eq. 3)                                */
/* ------------------------------------------------------------------ */

/* Latency-Constrained Accuracy-Optimized: the largest profiled k whose predicted total time
 * t0 + T(k, beta) still meets the latency target tau.  profile_bp / profile_ms: the latency
 * profile T(k, beta) of one co-location scenario at n_k settings of k.  When no setting meets
 * the target the query cannot be served within its SLO (Def. 1): feasible = 0 and the smallest
 * profiled k is returned. */
void orc_lcao_budgets(const uint16_t *profile_bp, const float *profile_ms, uint32_t n_k, const float *t0,
                      const float *tau, uint32_t n, uint16_t *budget_bp, uint8_t *feasible)
{
    for (uint32_t q = 0; q < n; ++q) {
        int found = 0;
        uint16_t best = 0, smallest = profile_bp[0];
        for (uint32_t i = 0; i < n_k; ++i) {
            if (profile_bp[i] < smallest) smallest = profile_bp[i];
            if (t0[q] + profile_ms[i] <= tau[q] && (!found || profile_bp[i] > best)) {
                best = profile_bp[i];
                found = 1;
            }
        }
        budget_bp[q] = found ? best : smallest;
        feasible[q] = (uint8_t)found;
    }
}

/* ------------------------------------------------------------------ */
/* Confidence (Sec. 2.1, Eq. 1), Confidence LSH tables (Sec. 3.2,      */
/* Eq. 4) and the ACLO budget choice (Sec. 2.2, Eq. 2)                 */
/* ------------------------------------------------------------------ */

/* c(k, x) = -distance(y, y_k) with the cross-entropy as distance (the paper's choice for
 * classification): y = softmax of the full network's logits is the target distribution,
 * y_k = softmax of the logits with the top k% of nodes computed.
 *   c = sum_j y_j * log y_k,j        (fp64; both softmaxes shifted by their maximum) */
double orc_confidence(const float *z_full, const float *z_k, uint32_t n)
{
    double mf = (double)z_full[0], mk = (double)z_k[0];
    for (uint32_t j = 1; j < n; ++j) {
        if ((double)z_full[j] > mf) mf = (double)z_full[j];
        if ((double)z_k[j] > mk) mk = (double)z_k[j];
    }
    double sf = 0.0, sk = 0.0;
    for (uint32_t j = 0; j < n; ++j) {
        sf += exp((double)z_full[j] - mf);
        sk += exp((double)z_k[j] - mk);
    }
    const double lse_k = mk + log(sk);
    double c = 0.0;
    for (uint32_t j = 0; j < n; ++j) {
        const double y = exp((double)z_full[j] - mf) / sf;
        c += y * ((double)z_k[j] - lse_k);
    }
    return c;
}

/* Confidence LSH tables: one set of L tables for the whole network, keyed by the hash functions
 * of the first layer's Node Activator.  For every profiled k_i and every training row x':
 * c(k_i, x') from a k_i% run and a 100 % run (CANON32 logits); the row's value is added to the
 * bucket it hashes to in each table.
 *   sum   [L][2^K][n_k]  fp64, rows added in row order
 *   count [L][2^K]       rows per bucket
 * Needs: layer 0 carries an activator and takes a dense input; the last layer carries none (the
 * distance is taken over the complete logit vector). */
int orc_confidence_build(const orc_model *m, const float *calib_dense, uint32_t n_cal,
                         const uint16_t *profile_bp, uint32_t n_k, double *sum, uint32_t *count)
{
    if (!m->has_act[0] || m->first_sparse || m->has_act[m->n_layers - 1] || n_cal == 0 || n_k == 0)
        return ORC_ERR_ARG;
    const uint32_t n_out = m->dims[m->n_layers], L = m->L, nb = 1u << m->K;
    const uint32_t n_act = count_act_layers(m);
    float *zf = (float *)malloc(sizeof(float) * (uint64_t)n_cal * n_out);
    float *zk = (float *)malloc(sizeof(float) * (uint64_t)n_cal * n_out);
    uint16_t *codes = (uint16_t *)malloc(sizeof(uint16_t) * (uint64_t)n_cal * n_act * L);
    uint16_t *bp = (uint16_t *)malloc(sizeof(uint16_t) * n_cal);
    if (!zf || !zk || !codes || !bp) return ORC_ERR_NOMEM;
    orc_batch bt;
    memset(&bt, 0, sizeof(bt));
    bt.n_queries = n_cal; bt.x_dense = calib_dense; bt.budget_bp = bp; bt.mode = ORC_CANON32;
    bt.logit_stride = n_out;
    for (uint32_t x = 0; x < n_cal; ++x) bp[x] = 10000;
    bt.logits32 = zf; bt.codes = codes;
    int rc = orc_run(m, &bt);
    memset(sum, 0, sizeof(double) * (uint64_t)L * nb * n_k);
    memset(count, 0, sizeof(uint32_t) * (uint64_t)L * nb);
    for (uint32_t x = 0; x < n_cal && rc == ORC_OK; ++x)
        for (uint32_t b = 0; b < L; ++b) count[b * nb + codes[((uint64_t)x * n_act + 0) * L + b]] += 1;
    bt.logits32 = zk; bt.codes = NULL;
    for (uint32_t i = 0; i < n_k && rc == ORC_OK; ++i) {
        for (uint32_t x = 0; x < n_cal; ++x) bp[x] = profile_bp[i];
        rc = orc_run(m, &bt);
        if (rc != ORC_OK) break;
        for (uint32_t x = 0; x < n_cal; ++x) {
            const double c = orc_confidence(zf + (uint64_t)x * n_out, zk + (uint64_t)x * n_out, n_out);
            for (uint32_t b = 0; b < L; ++b) {
                const uint32_t key = codes[((uint64_t)x * n_act + 0) * L + b];
                sum[((uint64_t)b * nb + key) * n_k + i] += c;
            }
        }
    }
    free(zf); free(zk); free(codes); free(bp);
    return rc;
}

/* Accuracy-Constrained Latency-Optimized (Eq. 2): the smallest profiled k whose estimated
 * confidence reaches the threshold that the accuracy target maps to.
 *   estimate (Eq. 4, aggregation = arithmetic mean): over the training rows that share a bucket
 *   with x in any of the L tables (a row counted once per table it shares):
 *       c^(k_i, x) = sum_b sum[b][key_b(x)][i] / sum_b count[b][key_b(x)]
 *   keys: the first layer's FreeHash keys of x (CANON32);
 *   threshold [n_targets][n_k]: t_i of each accuracy target (found on held-out data by the
 *   caller), target[q] picks the row;
 *   profile_bp ascending.  No training row in any of x's buckets, or no k_i reaching its
 *   threshold: the full network (10000 bp), met = 0. */
int orc_aclo_budgets(const orc_model *m, const double *sum, const uint32_t *count,
                     const uint16_t *profile_bp, uint32_t n_k, const float *x_dense, uint32_t n,
                     const float *threshold, const uint32_t *target, uint16_t *budget_bp,
                     uint8_t *met, double *estimate /* [n][n_k], nullable */)
{
    if (!m->has_act[0] || m->first_sparse) return ORC_ERR_ARG;
    const uint32_t D = m->dims[0], L = m->L, K = m->K, nb = 1u << K;
    for (uint32_t q = 0; q < n; ++q) {
        const float *in = x_dense + (uint64_t)q * D;
        uint32_t keys[8];
        for (uint32_t b = 0; b < L; ++b) {
            uint32_t key = 0;
            for (uint32_t j = 0; j < K; ++j)
                if (node_z32_dense(m, 0, m->hash_nodes[0][b * K + j], in) > 0.0f) key |= (1u << j);
            keys[b] = key;
        }
        uint64_t rows = 0;
        for (uint32_t b = 0; b < L; ++b) rows += count[b * nb + keys[b]];
        const float *thr = threshold + (uint64_t)(target ? target[q] : 0) * n_k;
        uint16_t pick = 10000;
        uint8_t ok = 0;
        for (uint32_t i = 0; i < n_k; ++i) {
            double s = 0.0;
            for (uint32_t b = 0; b < L; ++b) s += sum[((uint64_t)b * nb + keys[b]) * n_k + i];
            const double est = rows ? s / (double)rows : 0.0;
            if (estimate) estimate[(uint64_t)q * n_k + i] = est;
            if (!ok && rows && est >= (double)thr[i]) { pick = profile_bp[i]; ok = 1; }
        }
        budget_bp[q] = pick;
        if (met) met[q] = ok;
    }
    return ORC_OK;
}
