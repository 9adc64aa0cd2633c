/*
 * slonn.h -- C ABI of the SLO-NN inference library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-query inference path of an SLO-Aware Neural
 * Network ("Dynamic Network Adaptation at Inference", arxiv 2204.08400):
 *   build : Node-Activator training -- Algorithm 1 with FreeHash hash functions
 *           (Def. 2, Eq. 5) sampled in proportion to activation variance (Sec. 3.4);
 *   run   : the SLO-aware forward pass (Fig. 2 steps 1, 3, 4; Sec. 3.3): hash the
 *           layer input, fetch one ranked node list per table, keep the top k% of
 *           the lists, compute only those nodes, pass the sparse activation on.
 * The percentage k arrives as a per-query budget; the paper's two rules for
 * choosing it (LCAO, ACLO) are provided as separate calls that write such budgets.
 *
 * Conventions
 *   - Every function returns SLONN_OK (0) or a negative SLONN_ERR_* code.  Nothing
 *     throws, aborts or traps; device-side problems are reported through the
 *     batch's status words.
 *   - Pointers are DEVICE pointers unless the comment says "host".
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Ownership: the caller owns every buffer it passes in.  Weights and biases
 *     given to slonn_build are referenced, not copied: they must stay valid and
 *     unchanged until slonn_free.  The library owns what it allocates inside
 *     slonn_model (tables, hash-node ids, transposed copies of a CSR-fed first
 *     layer and of every layer that follows an activator layer -- a snapshot of
 *     those weights taken at build time).
 *   - A model is read-only after slonn_build; slonn_run may be called
 *     concurrently on different streams with different workspaces.
 *   - Arithmetic: every dot product is summed in fp32 in one fixed order (32
 *     partial sums; input element j goes to partial (j / V) mod 32 by fused
 *     multiply-add in ascending j, V = 16 bytes / weight element size; a fixed
 *     pairwise tree with strides 16, 8, 4, 2, 1; bias added last).  For a
 *     first layer fed by CSR input, j is the position in the row's id-ascending
 *     nonzero list and V = 1.  An input that is exactly 0 leaves its partial
 *     sum unchanged and may be skipped (weights must be finite).  Hash bits are
 *     signs of such sums, so the order is part of the interface: it does not
 *     depend on batch size, budget or launch shape.  bf16 weights are widened
 *     exactly; activations and biases are fp32.
 */
#ifndef SLONN_H
#define SLONN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLONN_VERSION 1

/* weight storage types */
#define SLONN_F32 0
#define SLONN_BF16 1

/* error codes */
#define SLONN_OK 0
#define SLONN_ERR_ARG (-1)       /* null pointer, bad handle, bad flag combination        */
#define SLONN_ERR_DIM (-2)       /* a width is 0 / too large, K*L exceeds a layer's width   */
#define SLONN_ERR_DTYPE (-3)     /* unknown weight type                                    */
#define SLONN_ERR_ALIGN (-4)     /* a weight row or buffer is not 16-byte aligned          */
#define SLONN_ERR_BUDGET (-5)    /* budget outside 1..10000 bp, above the batch's stated   */
                                 /* maximum, or above list_cap without being 100 %         */
#define SLONN_ERR_NOMEM (-6)     /* host or device allocation failed (build only)          */
#define SLONN_ERR_CUDA (-7)      /* a CUDA runtime call failed                             */
#define SLONN_ERR_TIMEOUT (-8)   /* a bounded device-side wait ran out                     */
#define SLONN_ERR_WORKSPACE (-9) /* workspace missing, misaligned or too small             */

#define SLONN_MAX_LAYERS 16
/* Widest input of a layer that is not fed by CSR rows: a query's layer input is staged in shared memory as fp32
 * (225 KB).  On a layer with a Node Activator the bitmap of its nodes shares that space: 4 * D + N / 8 bytes
 * must fit as well.  slonn_build and slonn_deserialize answer SLONN_ERR_DIM otherwise. */
#define SLONN_MAX_INPUT_WIDTH 57600u

typedef struct slonn_model slonn_model;

int slonn_version(void);
/* Static, NUL-terminated description of an error code. */
const char *slonn_strerror(int code);

/* ---------------------------------------------------------------------------
 * Build (Algorithm 1; hash-function sampling of Sec. 3.4)
 * ------------------------------------------------------------------------- */
typedef struct {
    uint32_t n_layers;             /* weight layers (hidden + output), 1..SLONN_MAX_LAYERS   */
    const uint32_t *dims;          /* host: n_layers+1 widths D0, N1, ..., N_out             */
    const uint8_t *has_activator;  /* host: per layer, 1 = the layer carries a Node Activator */
    int32_t dtype;                 /* SLONN_F32 | SLONN_BF16: storage type of every W         */
    uint32_t K, L;                 /* key bits per table (1..16), tables (1..8); paper: 10, 2 */
    uint32_t list_cap;             /* entries kept per bucket list; 0 = the whole layer       */
    uint64_t seed;                 /* seed of the hash-node sampling                          */
    uint32_t first_layer_sparse;   /* 1: layer 0 is fed CSR rows (sparse operand); it must    */
                                   /*    then carry no activator; calibration is CSR as well  */
    const uint32_t *const *hash_nodes_override; /* host, nullable; per layer nullable: L*K    */
                                   /* distinct node ids to use instead of sampling            */
    uint32_t free_hash_nodes;      /* 1: the variant of Sec. 3.4 in which a hash function's   */
                                   /*    dot product doubles as its node's output: a layer's  */
                                   /*    K*L hash nodes are always in its active set and are  */
                                   /*    left out of its ranked lists; the budget then counts */
                                   /*    list nodes only, so a layer computes                 */
                                   /*    min(B, N - K*L) + K*L nodes.  Needs K*L < N_l.       */
} slonn_build_desc;

typedef struct {
    uint32_t n_rows;
    const float *dense;            /* [n_rows][D0] fp32 row-major, or NULL when CSR           */
    const uint64_t *indptr;        /* CSR: [n_rows+1]                                         */
    const uint32_t *ids;           /* CSR: column ids, ascending and distinct within a row    */
    const float *vals;             /* CSR: values                                             */
} slonn_rows;

/*
 * Trains the Node-Importance tables of every activator layer on the calibration
 * rows (the paper's LSH training set): complete forward pass of the calibration
 * rows, per-node activation variance, K*L hash nodes per layer drawn with
 * probability proportional to variance, per table and bucket the sum of the
 * activations of the rows that hash there, and the node ids sorted by that sum
 * (highest first, equal sums by lower id).  A bucket no row reached holds the
 * ranking of the sums over all rows.
 *   W[l]    : row-major [N_l][D_l], rows 16-byte aligned (D_l * element size
 *             must be a multiple of 16), fp32 or bf16 bit patterns per desc->dtype
 *   bias[l] : [N_l] fp32
 * W and bias are host arrays of device pointers.  Hidden layers use ReLU, the
 * last layer the identity.  Synchronises `stream` before returning (the build
 * allocates, reads variances back and samples on the host).  *out is set only
 * on success.
 */
int slonn_build(const slonn_build_desc *desc, const void *const *W, const float *const *bias,
                const slonn_rows *calib, void *stream, slonn_model **out);

/*
 * Layer facts for parity checks.  hash_nodes: host buffer of L*K ids (nullable);
 * the other outputs are nullable too.  tables_dev points at the layer's lists,
 * laid out [L][2^K][cap] with ids of id_bytes (2 when N_l <= 65536, else 4).
 * Layers without activator report cap 0 and a NULL table.
 */
int slonn_model_info(const slonn_model *m, uint32_t layer, uint32_t *hash_nodes,
                     const void **tables_dev, uint64_t *table_bytes, uint32_t *id_bytes,
                     uint32_t *cap);

/*
 * Copies a layer's tables ([L][2^K][cap] ids of id_bytes each) into a HOST
 * buffer of at least table_bytes; synchronous.  For parity checks and for
 * persisting a trained activator.
 */
int slonn_model_tables_to_host(const slonn_model *m, uint32_t layer, void *dst_host, uint64_t dst_bytes);

/*
 * Persisting a trained Node Activator (the paper trains it "pre- or post-deployment",
 * Sec. 3.2: the tables outlive the process that made them).  slonn_serialize writes the
 * model's configuration, hash nodes and tables into a HOST buffer of at least
 * slonn_serialized_bytes(); slonn_deserialize rebuilds a model from such a blob without any
 * calibration pass.  Weights and biases are not stored: pass the same device arrays again
 * (same rules as slonn_build: referenced, must outlive the model).  A blob that is truncated,
 * damaged (checksum) or inconsistent with itself is refused with SLONN_ERR_ARG before
 * anything is allocated.  Both calls are synchronous.
 */
int slonn_serialized_bytes(const slonn_model *m, uint64_t *bytes);
int slonn_serialize(const slonn_model *m, void *dst_host, uint64_t dst_bytes);
int slonn_deserialize(const void *src_host, uint64_t src_bytes, const void *const *W,
                      const float *const *bias, void *stream, slonn_model **out);

/* Frees the model and everything it owns.  NULL is accepted. */
void slonn_free(slonn_model *m);

/* ---------------------------------------------------------------------------
 * Run (Fig. 2 steps 1, 3, 4; Sec. 3.3)
 * ------------------------------------------------------------------------- */
typedef struct {
    uint32_t n_queries;
    /* inputs */
    const float *x_dense;          /* [n][D0], or NULL when the model takes CSR rows          */
    const uint64_t *x_indptr;      /* CSR alternative (first_layer_sparse models)            */
    const uint32_t *x_ids;
    const float *x_vals;
    const uint16_t *budget_bp;     /* [n] per-query budget k in basis points, 1..10000;       */
                                   /* node count per activator layer B = max(1, round half up */
                                   /* of bp * N_l / 10000); free_hash_nodes models compute    */
                                   /* min(B, N_l - K*L) listed nodes plus the K*L hash nodes  */
    uint32_t max_budget_bp;        /* HOST value: upper bound of budget_bp[] (0 = 10000);     */
                                   /* sizes the launch grids, the workspace and logit_stride  */
    /* outputs (nullable unless stated) */
    float *logits;                 /* required. [n][logit_stride]: the last layer's           */
                                   /* pre-activations.  logit_stride = N_out, or, when the    */
                                   /* last layer is budgeted, the node count of max_budget_bp */
                                   /* (entries past a query's own count are left untouched)   */
    uint32_t *logit_ids;           /* [n][logit_stride] node id of each logit; required when  */
                                   /* the last layer is budgeted, ignored otherwise           */
    uint32_t *pred;                /* [n] argmax node id over the computed logits, lowest id  */
                                   /* on ties                                                 */
    uint16_t *codes;               /* [n][n_act_layers][L] hash keys                          */
    uint64_t *active_indptr;       /* [n*n_act_layers + 1] offsets into active_ids/vals,      */
                                   /* entry q*n_act_layers + a                                */
    uint32_t *active_ids;          /* active node ids, ascending within (query, layer);       */
                                   /* capacity = slonn_active_capacity()                      */
    float *active_vals;            /* their activations (zeros kept), same layout             */
    uint32_t *status;              /* required. [4] words: [0] first error code seen on the   */
                                   /* device (0 = ok, else -SLONN_ERR_*), [1] query index,    */
                                   /* [2] layer index, [3] reserved.  Cleared by slonn_run    */
    uint32_t flags;                /* HOST value: 0 or SLONN_FLAG_* below                     */
    uint32_t kernel_path;          /* HOST value: SLONN_PATH_AUTO, or force one of the        */
                                   /* kernel families (results are identical; for testing and */
                                   /* tuning).  _FUSED on a network it cannot take returns    */
                                   /* SLONN_ERR_DIM                                           */
} slonn_batch;

/*
 * SLONN_FLAG_DENSE_TC: queries whose budget is 10000 bp compute every node of every layer, i.e.
 * the plain dense network (Sec. 3.4).  With this flag they are taken out of the per-query
 * kernels, compacted, and run layer by layer as bf16 matrix products on the tensor cores
 * (activations rounded to bf16 between layers, fp32 accumulation).  Their active sets are still
 * "all nodes" and their logits stay within the bf16-weight tolerance (2e-2 of the largest
 * logit), but nothing about them is bit-compatible with the fixed-order kernels: values differ
 * in the last bits, and a hash code or an argmax decided by a near-tie can differ.  Other
 * queries are unaffected.  Honoured when weights are bf16, the first layer is dense, the last
 * layer has no activator and max_budget_bp is 10000 (or 0); otherwise ignored.
 */
#define SLONN_FLAG_DENSE_TC 1u
/*
 * A layer whose input is the sparse output of an activator layer (Sec. 3.3) can be evaluated in two
 * ways with identical results: row kernels read each selected weight row whole; input-stationary
 * kernels walk the query's nonzero inputs and read single weights from a transposed copy the model
 * keeps of such layers.  By default the library picks per query by budget: up to SLONN_COLS_MAX_BP
 * the input list is sparse enough for the input-stationary kernels to win (batches of tens of queries
 * only when no budget exceeds 1500 bp and only for layers at least 2048 inputs wide; a handful of queries keep
 * the row kernels).  These two flags force one kind for the whole batch, for testing and
 * tuning; setting both is an error.  They apply to the per-stage kernels and to the
 * one-warp-per-query kernel; the one-cluster-per-query kernel has row form only.
 */
#define SLONN_COLS_MAX_BP 3500u /* default split: budgets up to this take the input-stationary kernels */
#define SLONN_FLAG_ROW_KERNELS 2u
#define SLONN_FLAG_COLUMN_KERNELS 4u
/*
 * The row kernels take the queries of a large batch four per block, so that a weight row most of the four
 * selected is loaded once for all of them (the batch formulation of Sec. 7).  This flag keeps every query in
 * a block of its own (results are identical; for testing and tuning).
 */
#define SLONN_FLAG_UNGROUPED_ROWS 8u
#define SLONN_FLAG_ALL 15u

#define SLONN_PATH_AUTO 0    /* library chooses                                               */
#define SLONN_PATH_STAGED 1  /* one block per query and stage: any model, any batch size      */
#define SLONN_PATH_CLUSTER 3 /* one thread-block cluster per query through all layers, for a      */
                             /* handful of queries (latency): widths and layers <= 8192, dense  */
                             /* first layer, no SLONN_FLAG_DENSE_TC                             */
#define SLONN_PATH_FUSED 2   /* one warp per query through all layers: widths <= 1024 inputs, */
                             /* <= 4096 nodes per layer, dense first layer                    */
#define SLONN_PATH_BLOCK 4   /* one block of four warps per query through all layers: the same */
                             /* networks as _FUSED; chosen by itself for batches of at most 512 */
                             /* queries whose layers compute at most 64 rows per query; no      */
                             /* SLONN_FLAG_DENSE_TC                                             */

/*
 * Latency-Constrained Accuracy-Optimized budgets (Sec. 2.3, Eq. 3): for each query the largest
 * profiled k whose predicted total time t0 + T(k, beta) meets the query's latency target tau.
 *   profile_bp, profile_ms : [n_k] the latency profile T(k, beta) of the current co-location
 *                            scenario: budgets in basis points and the measured latency of a
 *                            batch at that budget (n_k <= 4096, any order)
 *   t0, tau                : [n] time already spent on the query outside inference, and its
 *                            latency target (same unit as profile_ms)
 *   budget_bp              : [n] out: ready to be used as slonn_batch.budget_bp
 *   feasible               : [n] out, nullable: 0 where no profiled k meets the target (Def. 1:
 *                            the SLO cannot be fulfilled); such queries get the smallest profiled k
 * All pointers are device pointers; asynchronous on `stream`.
 */
int slonn_lcao_budgets(const uint16_t *profile_bp, const float *profile_ms, uint32_t n_k,
                       const float *t0, const float *tau, uint32_t n, uint16_t *budget_bp,
                       uint8_t *feasible, void *stream);

/*
 * Confidence LSH tables (Sec. 3.2, Eq. 4) for the Accuracy-Constrained Latency-Optimized policy.
 * The confidence of the network on input x at budget k is c(k, x) = -distance(y, y_k) (Sec. 2.1,
 * Eq. 1) with the cross-entropy as distance: y = softmax of the complete network's logits (the
 * target distribution), y_k = softmax of the logits at budget k, c = sum_j y_j log y_k,j (fp64).
 * The tables are one set of L tables for the whole network, keyed by the first layer's FreeHash
 * keys.  Training needs no labels: every row is run at 100 % and at each profiled k; its c(k, x)
 * is added to the bucket it hashes to in each table (fp64, rows in order), and the rows per
 * bucket are counted.
 *   rows       : dense training rows (device), as for slonn_build
 *   profile_bp : HOST, [n_k] budgets in basis points, strictly ascending, n_k <= 64
 * Needs a model whose layer 0 carries an activator and takes dense input and whose last layer
 * carries none (the distance is taken over the complete logit vector); otherwise SLONN_ERR_ARG.
 * Allocates, runs 1 + n_k forward passes over the rows and synchronises `stream`.
 */
typedef struct slonn_confidence slonn_confidence;
int slonn_confidence_build(const slonn_model *m, const slonn_rows *rows, const uint16_t *profile_bp,
                           uint32_t n_k, void *stream, slonn_confidence **out);
/* Copies the tables to HOST arrays: sum [L][2^K][n_k] (fp64), count [L][2^K]; synchronous. */
int slonn_confidence_to_host(const slonn_confidence *c, double *sum_host, uint64_t sum_entries,
                             uint32_t *count_host, uint64_t count_entries);
/* Frees the tables.  NULL is accepted. */
void slonn_confidence_free(slonn_confidence *c);

/*
 * ACLO budgets (Sec. 2.2, Eq. 2): for each query the smallest profiled k whose estimated
 * confidence reaches the threshold its accuracy target maps to.  The estimate (Eq. 4 with the
 * arithmetic mean) pools the training rows that share a bucket with x in any of the L tables:
 *     c^(k_i, x) = sum_b sum[b][key_b(x)][i] / sum_b count[b][key_b(x)]
 *   x_dense    : [n][D0] the queries (16-byte aligned); their keys are computed here with the
 *                same fixed-order dot products as in slonn_run
 *   threshold  : [n_targets][n_k] confidence threshold t_i of each accuracy target at each
 *                profiled k (the caller finds them on held-out data, Sec. 3.2)
 *   target     : [n] row of `threshold` per query; NULL = row 0 for every query
 *   budget_bp  : [n] out, ready to be used as slonn_batch.budget_bp
 *   met        : [n] out, nullable: 0 where no training row shares a bucket with x or no
 *                profiled k reaches its threshold; such queries get 10000 bp (the full network)
 *   estimate   : [n][n_k] out, nullable: the estimates (0 where no row shares a bucket)
 *   status     : [4] nullable, as in slonn_batch: a target index out of range is reported there
 *                (the query then uses row 0); not cleared by this call
 * All pointers are device pointers; asynchronous on `stream`; no allocation.
 */
int slonn_aclo_budgets(const slonn_model *m, const slonn_confidence *c, const float *x_dense,
                       uint32_t n, const float *threshold, uint32_t n_targets, const uint32_t *target,
                       uint16_t *budget_bp, uint8_t *met, double *estimate, uint32_t *status,
                       void *stream);

/* Number of entries active_ids / active_vals need for n queries at max_budget_bp. */
int slonn_active_capacity(const slonn_model *m, uint32_t n_queries, uint32_t max_budget_bp,
                          uint64_t *entries);
/* logit_stride for this model at max_budget_bp (see slonn_batch.logits). */
int slonn_logit_stride(const slonn_model *m, uint32_t max_budget_bp, uint32_t *stride);
/* Bytes of device workspace slonn_run needs (256-byte aligned buffer) for a batch with these
 * n_queries, max_budget_bp and flags. */
int slonn_workspace_bytes(const slonn_model *m, uint32_t n_queries, uint32_t max_budget_bp,
                          uint32_t flags, uint64_t *bytes);

/*
 * Runs the batch on `stream`: asynchronous, no allocation, no host
 * synchronisation.  The caller synchronises the stream and reads status[0].
 * A query whose budget is invalid gets a clamped, in-range active set and the
 * error is recorded in status; other queries are unaffected.
 */
int slonn_run(const slonn_model *m, const slonn_batch *batch, void *workspace,
              uint64_t workspace_bytes, void *stream);

/*
 * One dense layer on the tensor cores: out = act(X * W^T + bias), the case in which every
 * node of a layer is computed (Sec. 3.4: with all nodes computed an SLO-NN does exactly the
 * work of the full network).  bf16 operands, fp32 accumulation in tensor memory.
 *   x_bf16  : [M][D] bf16 bit patterns, row-major      w_bf16 : [N][D] bf16, row-major
 *   bias    : [N] fp32, nullable                       relu   : 1 = max(., 0), 0 = identity
 *   out_f32 : [M][N] fp32, nullable                    out_bf16 : [M][N] bf16 (rounded to
 *             nearest even), nullable; at least one of the two
 *   status  : [4] device words, nullable; cleared, then [0] = -SLONN_ERR_TIMEOUT if a bounded
 *             on-chip wait ran out
 * D * 2 bytes must be a multiple of 16 and both matrices 16-byte aligned.  Asynchronous on
 * `stream`.  The accumulation order of the tensor core is unspecified, so results agree with
 * the fixed-order kernels to rounding (about 1e-6 relative per sum), not bit for bit.
 */
int slonn_dense_layer(const void *x_bf16, const void *w_bf16, const float *bias, uint32_t M,
                      uint32_t N, uint32_t D, uint32_t relu, float *out_f32, void *out_bf16,
                      uint32_t *status, void *stream);

/*
 * Testing aid for the give-up path of the tensor-core kernel (no passage of the paper: the library's own
 * failure reporting).  Every on-chip wait of that kernel is bounded; when one runs out the block stops issuing
 * work, lets copies in flight land, frees its tensor memory and writes -SLONN_ERR_TIMEOUT to status[0].  With
 * polls != 0 every later slonn_dense_layer / SLONN_FLAG_DENSE_TC launch of this process makes its loader wait,
 * for at most `polls` polls, on a barrier that nothing signals -- before it has issued any copy or product -- so
 * the launch ends through that path and computes nothing.  0 restores normal operation.  Process-wide; not for
 * production use.
 */
int slonn_test_tc_wait_limit(uint32_t polls);

/*
 * slonn_run without a caller-provided workspace.  (The paper has no counterpart;
 * this exists for deployment.)
 *
 * Who needs it: code that has to serve queries but is not allowed to obtain
 * device memory -- a request handler in a serving process whose device memory
 * was partitioned at start-up and where later cudaMalloc calls are forbidden or
 * would stall every stream; a plug-in inside a host program whose own allocator
 * owns the GPU; a C caller with no allocator at hand at all.  Such a caller still
 * passes its input and output buffers in `batch`, exactly as for slonn_run, but
 * the intermediate lists and activations go to a fixed scratch area of
 * SLONN_STATIC_WORKSPACE_BYTES that is compiled into the library as a device
 * array (each GPU that loads the library holds those bytes until the process
 * ends).  The call performs no cudaMalloc / cudaFree and uses no allocating
 * library routine.
 *
 *   - The batch must fit: if slonn_workspace_bytes(m, n_queries, max_budget_bp, flags)
 *     exceeds SLONN_STATIC_WORKSPACE_BYTES the call returns SLONN_ERR_WORKSPACE
 *     and launches nothing.  Use smaller batches or slonn_run.
 *   - The model's device must be the current device (else SLONN_ERR_ARG).
 *   - The first call on each device looks up the scratch area's device address
 *     (a one-time set-up step under a lock).  Make that first call during
 *     start-up, before any stream capture begins.
 *   - All calls on a device share the one scratch area and it keeps whatever the
 *     previous call left there.  Nothing in it needs to start at zero (every
 *     entry is written before it is read within a call), but two calls whose
 *     kernels overlap on the GPU -- different streams, or different host threads
 *     -- race on it: serialise them on one stream.
 * Results are identical to slonn_run's.
 */
#define SLONN_STATIC_WORKSPACE_BYTES (16u << 20)
int slonn_run_static(const slonn_model *m, const slonn_batch *batch, void *stream);

/*
 * slonn_run with a CUDA event pair around every kernel launch, for measurement
 * (the per-stage breakdown of Fig. 3 of the paper: time in the LSH part, which
 * includes the hash functions, against time in the forward computation).
 * Synchronises `stream`, then adds each launch's device time to
 * stage_ms[stage] and counts it in stage_launches[stage] (both HOST arrays of
 * SLONN_N_STAGES entries).  Creates and destroys events, so unlike slonn_run it
 * is not allocation-free.
 */
#define SLONN_STAGE_PLAN 0          /* budgets -> list offsets                      */
#define SLONN_STAGE_HASH_SELECT 1   /* FreeHash bits, keys, bucket lists, top-k% cut */
#define SLONN_STAGE_GATHER_DOT 2    /* selected rows' dot products                   */
#define SLONN_STAGE_SPARSE_FIRST 3  /* first layer fed by CSR rows                   */
#define SLONN_STAGE_ARGMAX 4        /* prediction                                    */
#define SLONN_STAGE_FUSED 5         /* all of 1, 2, 4 in the one-warp-per-query kernel */
#define SLONN_STAGE_DENSE_TC 6      /* 100 % budget queries on the tensor cores        */
#define SLONN_STAGE_CLUSTER 7       /* all of 1, 2, 4 in the one-cluster-per-query kernel */
#define SLONN_STAGE_GATHER_COLS 8   /* selected nodes' dot products, input-stationary kernel */
#define SLONN_STAGE_LAYER_COLS 9    /* all of 1 and 8 for a list-fed activator layer in one launch */
#define SLONN_STAGE_FULL_ROWS 10    /* every layer of the 100 % budget queries, four queries per block */
#define SLONN_STAGE_GROUP_ROWS 11   /* selected rows' dot products, four queries per block   */
#define SLONN_N_STAGES 12
int slonn_run_timed(const slonn_model *m, const slonn_batch *batch, void *workspace,
                    uint64_t workspace_bytes, void *stream, float *stage_ms,
                    uint32_t *stage_launches);

/*
 * The same measurement launch by launch: which stage, which layer, which queries (by budget range) and, for
 * the whole-network kernels, which form the list-fed layers took -- enough for a caller that knows the
 * budgets to count the weight bytes each launch had to touch (Sec. 3.3: hashed rows, bucket lists, selected
 * nodes times input entries) without repeating the library's kernel choice.  `records` is a HOST array of
 * `capacity` entries (SLONN_MAX_RECORDS always suffices); *n_records (host) receives how many were written,
 * in launch order.  Synchronises `stream`; creates and destroys events.
 */
#define SLONN_ALL_LAYERS 0xffffffffu
#define SLONN_MAX_RECORDS (10 * SLONN_MAX_LAYERS)
typedef struct {
    uint32_t stage;      /* SLONN_STAGE_*                                                             */
    uint32_t layer;      /* the layer the launch works on, or SLONN_ALL_LAYERS                        */
    uint32_t bp_lo, bp_hi; /* it serves the queries whose budget lies in [bp_lo, bp_hi] ...           */
    uint32_t skips_full; /* ... 1: except those at 10000 bp, which another launch serves              */
    uint32_t cols_bp;    /* whole-network launches: queries with budgets up to this evaluated their   */
                         /* list-fed activator layers input-stationary (0 = every layer row-wise)     */
    float ms;            /* device time between the event pair around the launch                      */
} slonn_launch_record;
int slonn_run_traced(const slonn_model *m, const slonn_batch *batch, void *workspace,
                     uint64_t workspace_bytes, void *stream, slonn_launch_record *records,
                     uint32_t capacity, uint32_t *n_records);

/*
 * Same computation for callers that keep queries and results in HOST memory:
 * every pointer of `host_batch` (inputs, outputs, status) is a host pointer,
 * pinned memory recommended.  Copies the inputs to the device, runs, copies
 * every non-NULL output back and synchronises `stream` before returning.
 * `workspace` is device memory of at least slonn_host_workspace_bytes().
 * h2d_bytes / d2h_bytes (host, nullable) receive the bytes copied each way.
 */
int slonn_host_workspace_bytes(const slonn_model *m, uint32_t n_queries, uint32_t max_budget_bp,
                               uint32_t flags, uint64_t x_nnz, uint64_t *bytes);
int slonn_run_host(const slonn_model *m, const slonn_batch *host_batch, void *workspace,
                   uint64_t workspace_bytes, void *stream, uint64_t *h2d_bytes,
                   uint64_t *d2h_bytes);

#ifdef __cplusplus
}
#endif
#endif /* SLONN_H */
