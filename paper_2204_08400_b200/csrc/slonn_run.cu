// Host side of slonn_run: validates the batch, carves the workspace and
// enqueues the per-layer kernels on the caller's stream.  No allocation, no
// host synchronisation.
#include <algorithm>
#include <cstring>
#include <mutex>

#include "slonn_dense_tc.cuh"
#include "slonn_fused_kernel.cuh"
#include "slonn_run_kernels.cuh"
#include "slonn_cluster_kernel.cuh"

namespace {

// Optional per-launch timing: an event pair around every launch, with what the launch covers.
struct stage_timer {
    struct span { int stage; uint32_t layer, bp_lo, bp_hi, skips_full, cols_bp; cudaEvent_t a, b; };
    span spans[10 * SLONN_MAX_LAYERS];
    int n = 0;
    bool failed = false;
    cudaStream_t st = nullptr;
    uint32_t layer = SLONN_ALL_LAYERS; // layer the next launches work on
    void tic(int stage, const uint16_t *range_bp = nullptr, uint32_t lo = 0, uint32_t hi = 0xffffu, const uint16_t *skip_bp = nullptr,
             uint32_t cols_bp = 0)
    {
        if (n >= (int)(sizeof(spans) / sizeof(spans[0]))) { failed = true; return; }
        span &s = spans[n];
        s.stage = stage; s.layer = layer;
        s.bp_lo = range_bp ? lo : 0u; s.bp_hi = range_bp ? std::min(hi, 10000u) : 10000u;
        s.skips_full = skip_bp ? 1u : 0u; s.cols_bp = cols_bp;
        if (cudaEventCreate(&s.a) != cudaSuccess || cudaEventCreate(&s.b) != cudaSuccess) { failed = true; return; }
        cudaEventRecord(s.a, st);
        ++n;
    }
    void toc() { if (n > 0 && !failed) cudaEventRecord(spans[n - 1].b, st); }
};
#define TIC(...) do { if (tm) tm->tic(__VA_ARGS__); } while (0)
#define TOC() do { if (tm) tm->toc(); } while (0)
#define AT_LAYER(l) do { if (tm) tm->layer = (l); } while (0)

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

inline bool model_ok(const slonn_model *m) { return m && m->magic == SLONN_MAGIC; }

inline uint32_t eff_max_bp(uint32_t max_bp) { return (max_bp == 0 || max_bp > 10000u) ? 10000u : max_bp; }

// entries of the active CSR payload for n queries at max_bp
uint64_t active_entries(const slonn_model *m, uint32_t n, uint32_t max_bp)
{
    uint64_t per = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l)
        if (m->layer[l].has_act) per += slonn_layer_nodes(max_bp, m->layer[l].N, slonn_model_pre(m));
    return per * n;
}

// widest dense intermediate a non-activator hidden layer writes
uint32_t dense_width(const slonn_model *m)
{
    uint32_t w = 0;
    for (uint32_t l = 0; l + 1 < m->n_layers; ++l)
        if (!m->layer[l].has_act) w = std::max(w, m->layer[l].N);
    return w;
}

struct ws_layout {
    uint64_t indptr, plan_sums, ids, vals, dense0, dense1, tc_list, tc_count, tc_a0, tc_a1, total;
};

// widest bf16 activation matrix row the tensor-core route needs
uint32_t tc_width(const slonn_model *m)
{
    uint32_t w = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l) w = std::max(w, m->layer[l].D);
    return w;
}

// whether the batch's 100 % budget queries take the tensor-core route
bool tc_route(const slonn_model *m, uint32_t max_bp, uint32_t flags)
{
    return (flags & SLONN_FLAG_DENSE_TC) && max_bp == 10000u && m->dtype == SLONN_BF16 && !m->first_sparse &&
           !m->layer[m->n_layers - 1].has_act;
}

// whether a batch with this largest budget may hold 100 % queries that the grouped full-network kernel can take
bool full_route_possible(const slonn_model *m, uint32_t max_bp)
{
    return max_bp == 10000u && !m->first_sparse;
}

ws_layout carve(const slonn_model *m, uint32_t n, uint32_t max_bp, uint32_t flags)
{
    ws_layout w;
    const uint64_t ent = active_entries(m, n, max_bp);
    uint64_t o = 0;
    w.indptr = o; o = align_up(o + ((uint64_t)n * m->n_act + 1) * sizeof(uint64_t), 256);
    const uint64_t tiles = ((uint64_t)n * m->n_act + SLONN_PLAN_TILE - 1) / SLONN_PLAN_TILE;
    w.plan_sums = o; o = align_up(o + (tiles + 1) * sizeof(uint64_t), 256);
    w.ids = o; o = align_up(o + ent * sizeof(uint32_t), 256);
    w.vals = o; o = align_up(o + ent * sizeof(float), 256);
    const uint64_t db = align_up((uint64_t)n * dense_width(m) * sizeof(float), 256);
    w.dense0 = o; o += db;
    w.dense1 = o; o += db;
    w.tc_list = w.tc_count = w.tc_a0 = w.tc_a1 = 0;
    // a compacted list of queries: the batch's 100 % queries, or the queries a grouped launch serves
    w.tc_list = o; o = align_up(o + (uint64_t)n * sizeof(uint32_t), 256);
    w.tc_count = o; o += 256;
    if (tc_route(m, max_bp, flags)) {
        const uint64_t ab = align_up((uint64_t)n * tc_width(m) * sizeof(uint16_t), 256);
        w.tc_a0 = o; o += ab;
        w.tc_a1 = o; o += ab;
    }
    w.total = std::max<uint64_t>(o, 256);
    return w;
}

template <typename K>
int set_smem(K kernel, size_t bytes)
{
#ifdef SLONN_CARVEOUT
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, SLONN_CARVEOUT);
#endif
    return slonn_allow_smem(reinterpret_cast<const void *>(kernel), bytes);
}

template <bool BF16, typename IDT, bool LAT>
int launch_select_t(const slonn_select_params &P, uint32_t n, uint32_t threads, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(hash_select_kernel<BF16, IDT, LAT>, smem);
    if (rc) return rc;
    hash_select_kernel<BF16, IDT, LAT><<<n, threads, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

// Fewer queries than SMs: latency variant, one warp per hash row (at least 8, at most 32 warps).
// Very long lists (tens of thousands of positions to walk per query): the same variant with 1024 threads,
// so that a selection step covers 1024 list positions.
int launch_select(const slonn_model *m, const slonn_select_params &P, uint32_t n, uint32_t max_rows, cudaStream_t st)
{
    const size_t smem = (size_t)P.D * 4 + (size_t)((P.N + 31) / 32) * 4;
    const bool bf = m->dtype == SLONN_BF16;
    const bool id16 = m->layer[P.layer].id_bytes == 2;
    const bool few = n <= 148, long_lists = (uint64_t)max_rows * m->L >= 32768;
    const bool lat = few || long_lists;
    const uint32_t threads = long_lists ? (n > 148u ? 512u : 1024u) : few ? 32u * std::min(32u, std::max(8u, m->H)) : (uint32_t)SLONN_THREADS;
    if (lat) {
        if (bf && id16) return launch_select_t<true, uint16_t, true>(P, n, threads, smem, st);
        if (bf) return launch_select_t<true, uint32_t, true>(P, n, threads, smem, st);
        if (id16) return launch_select_t<false, uint16_t, true>(P, n, threads, smem, st);
        return launch_select_t<false, uint32_t, true>(P, n, threads, smem, st);
    }
    if (bf && id16) return launch_select_t<true, uint16_t, false>(P, n, threads, smem, st);
    if (bf) return launch_select_t<true, uint32_t, false>(P, n, threads, smem, st);
    if (id16) return launch_select_t<false, uint16_t, false>(P, n, threads, smem, st);
    return launch_select_t<false, uint32_t, false>(P, n, threads, smem, st);
}

// Rows per block: whole queries per block once the batch alone fills the GPU,
// smaller row chunks for small batches so that every SM gets work.
void gather_shape(uint32_t n, uint32_t max_rows, uint32_t rows_per_pass, uint32_t *rows_per_cta, uint32_t *ctas_per_query)
{
    const uint32_t unit = (SLONN_THREADS / 32) * rows_per_pass; // rows one block pass covers
    const uint64_t want_ctas = 148ull * 16;                     // a few waves of resident blocks
    uint64_t total_rows = (uint64_t)n * max_rows;
    uint64_t rpc = (total_rows + want_ctas - 1) / want_ctas;
    rpc = std::max<uint64_t>(unit, (rpc + unit - 1) / unit * unit);
    if (rpc > max_rows) rpc = (max_rows + unit - 1) / unit * unit;
    *rows_per_cta = (uint32_t)rpc;
    *ctas_per_query = (uint32_t)((max_rows + rpc - 1) / rpc);
}

template <bool BF16, bool LAT, int R>
int launch_gather_t(const slonn_gather_params &P, uint64_t grid, uint32_t threads, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(gather_dot_kernel<BF16, LAT, R>, smem);
    if (rc) return rc;
    gather_dot_kernel<BF16, LAT, R><<<(uint32_t)grid, threads, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

template <bool BF16>
int launch_gather_short_t(const slonn_gather_params &P, uint64_t grid, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(gather_short_kernel<BF16>, smem);
    if (rc) return rc;
    gather_short_kernel<BF16><<<(uint32_t)grid, SLONN_THREADS, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

#ifndef SLONN_GATHER_R
#define SLONN_GATHER_R 4 // rows per warp pass of the row kernel for rows longer than one 512-byte round (4 or 8)
#endif
int launch_gather(const slonn_model *m, slonn_gather_params &P, uint32_t n, uint32_t max_rows, cudaStream_t st)
{
    // so few rows that the GPU cannot be filled: latency variant, 4 warps per block, one row per warp
    const bool lat = (uint64_t)n * max_rows <= 148ull * 64;
    const bool short_rows = P.nchunks <= 32; // a row is one 512-byte round: 8 rows per warp pass
    uint32_t threads = SLONN_THREADS;
    if (lat) {
        threads = 128;
        P.rows_per_cta = 4;
        P.ctas_per_query = (max_rows + 3) / 4;
    } else {
        gather_shape(n, max_rows, short_rows ? 32u : (uint32_t)SLONN_GATHER_R, &P.rows_per_cta, &P.ctas_per_query);
    }
    const size_t smem = (size_t)P.D * 4;
    const uint64_t grid = (uint64_t)n * P.ctas_per_query;
    if (grid == 0 || grid > 0x7fffffffull) return SLONN_ERR_DIM;
    const bool bf = m->dtype == SLONN_BF16;
    if (lat) return bf ? launch_gather_t<true, true, 4>(P, grid, threads, smem, st) : launch_gather_t<false, true, 4>(P, grid, threads, smem, st);
    if (short_rows) return bf ? launch_gather_short_t<true>(P, grid, smem, st) : launch_gather_short_t<false>(P, grid, smem, st);
    return bf ? launch_gather_t<true, false, SLONN_GATHER_R>(P, grid, threads, smem, st)
              : launch_gather_t<false, false, SLONN_GATHER_R>(P, grid, threads, smem, st);
}

// ---- selected rows, four queries per block --------------------------------------

struct group_ws { uint32_t *list, *count; }; // workspace for the compacted list of the queries a launch serves

template <bool BF16>
int launch_group_rows_t(const slonn_group_params &Q, uint64_t grid, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(group_rows_kernel<BF16>, smem);
    if (rc) return rc;
    group_rows_kernel<BF16><<<(uint32_t)grid, SLONN_THREADS, smem, st>>>(Q);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

size_t group_rows_smem(const slonn_gather_params &P, uint32_t max_rows, uint32_t *shared_cap)
{
    const uint32_t nwords = (P.N + 31u) / 32u;
    *shared_cap = std::min<uint64_t>(P.N, (uint64_t)4 * max_rows / 3 + 1);
    return (size_t)SLONN_GROUP * P.D * 4 + (size_t)(2 * SLONN_GROUP + 1) * nwords * 4 + (size_t)((*shared_cap + 7u) & ~7u) * 2 +
           (size_t)SLONN_GROUP * ((max_rows + 7u) & ~7u) * 2;
}

// The selected rows of a list-selecting layer for the queries in P's budget range.  In a large batch the queries
// whose budget exceeds SLONN_GROUP_MIN_BP are taken four per block (rows that most of the four selected are loaded
// once for all of them): at such budgets any four queries share most of their rows.  Below that, and for small
// batches, layers of more than 65,535 nodes, rows of a single 512-byte round and shapes whose staging does not
// fit two blocks per SM, every query has a block (or several) of its own.  Same values either way.
// Measured on a 4096-wide layer with 4096 queries: 50 % budget 3.5 -> 2.8 ms per layer, 25 % 1.77 -> 1.68 ms,
// 10 % 0.72 -> 0.79 ms (hence the limit).
#ifndef SLONN_GROUP_MIN_BP
#define SLONN_GROUP_MIN_BP 2000u
#endif
int launch_rows(const slonn_model *m, slonn_gather_params &P, const slonn_batch *b, uint32_t n, uint32_t max_bp,
                uint32_t max_rows, const group_ws &gw, cudaStream_t st, stage_timer *tm)
{
    uint32_t shared_cap = 0;
    const size_t smem = group_rows_smem(P, max_rows, &shared_cap);
    const uint32_t lo = P.range_bp ? P.bp_lo : 0u, hi = std::min(P.range_bp ? P.bp_hi : 0xffffu, max_bp);
    const uint32_t split = std::max(lo, SLONN_GROUP_MIN_BP + 1u); // budgets from here on are grouped
    const bool grouped = P.use_list && n >= 256 && P.N <= 65535u && P.nchunks > 32 && gw.list && smem <= 110 * 1024 &&
                         !(b->flags & SLONN_FLAG_UNGROUPED_ROWS) && hi >= split;
    int rc;
    if (!grouped) {
        TIC(SLONN_STAGE_GATHER_DOT, P.range_bp, P.bp_lo, P.bp_hi, P.skip_bp);
        rc = launch_gather(m, P, n, max_rows, st);
        TOC();
        return rc;
    }
    if (lo < split) { // the low budgets of this launch: one query per block
        slonn_gather_params A = P;
        A.range_bp = b->budget_bp; A.bp_lo = lo; A.bp_hi = split - 1u;
        TIC(SLONN_STAGE_GATHER_DOT, A.range_bp, A.bp_lo, A.bp_hi, A.skip_bp);
        rc = launch_gather(m, A, n, std::min(max_rows, slonn_layer_nodes(split - 1u, P.N, slonn_model_pre(m))), st);
        TOC();
        if (rc) return rc;
    }
    // the others, compacted in two budget classes so that the queries of a group select about as many rows
    if (cudaMemsetAsync(gw.count, 0, sizeof(uint32_t), st) != cudaSuccess) return SLONN_ERR_CUDA;
    const uint32_t mid = 3750u;
    if (split <= mid)
        range_compact_kernel<<<(n + 255) / 256, 256, 0, st>>>(b->budget_bp, P.skip_bp, n, split, std::min(mid, hi), gw.list, gw.count);
    if (hi > mid)
        range_compact_kernel<<<(n + 255) / 256, 256, 0, st>>>(b->budget_bp, P.skip_bp, n, std::max(split, mid + 1u), hi, gw.list, gw.count);
    if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
    slonn_group_params Q;
    memset(&Q, 0, sizeof(Q));
    Q.G = P; Q.list = gw.list; Q.count = gw.count; Q.rows_cap = max_rows; Q.shared_cap = shared_cap;
    const uint32_t groups = (n + SLONN_GROUP - 1) / SLONN_GROUP;
    // enough blocks for a few waves of two per SM, but no block with fewer than 32 rows of each kind
    Q.ctas_per_group = std::max(1u, std::min(std::min(8u, (148u * 8u + groups - 1) / groups), max_rows / 32u));
    TIC(SLONN_STAGE_GROUP_ROWS, b->budget_bp, split, hi, P.skip_bp);
    rc = m->dtype == SLONN_BF16 ? launch_group_rows_t<true>(Q, (uint64_t)groups * Q.ctas_per_group, smem, st)
                                : launch_group_rows_t<false>(Q, (uint64_t)groups * Q.ctas_per_group, smem, st);
    TOC();
    return rc;
}

// Input-stationary gather for a layer fed by (id, value) lists: 32 * R nodes per warp pass, the passes of
// a block spread evenly over at most 8 warps, a few blocks per SM.
#ifndef SLONN_COLS_R
#define SLONN_COLS_R 2
#endif
// few-queries variants: warps per block, four segments of the input list each (4, 16 and 32 warps measured
// slower on a 4096-wide nine-layer network with 64 queries: 0.237 / 0.248 / 0.372 ms against 0.195 ms for its
// seven hidden layers)
#define SLONN_SPLIT_WARPS 8u
template <bool BF16, int R, bool SPLIT, bool VEC = false>
int launch_gather_cols_t(const slonn_gather_params &P, uint64_t grid, uint32_t threads, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(gather_cols_kernel<BF16, R, SPLIT, VEC>, smem);
    if (rc) return rc;
    gather_cols_kernel<BF16, R, SPLIT, VEC><<<(uint32_t)grid, threads, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

int launch_gather_cols(const slonn_model *m, slonn_gather_params &P, uint32_t n, uint32_t max_rows, cudaStream_t st)
{
    const bool bf = m->dtype == SLONN_BF16;
    const uint32_t R = SLONN_COLS_R;
    const uint64_t want_ctas = 148ull * 8;
    // too few warp passes to fill the GPU: one block per pass, its warps sharing the walk over the input list
    const bool split = (uint64_t)n * ((max_rows + 32u * R - 1u) / (32u * R)) < want_ctas;
    // a layer that computes every node, its width a multiple of the nodes one 16-byte load holds: a lane takes that
    // many neighbouring columns (1000-node output layer of a 4096-wide network: 0.36 -> 0.26 ms per 4096 queries)
    const uint32_t nv = bf ? 8u : 4u;
    const bool vec = !split && !P.use_list && P.N % nv == 0u;
    const uint32_t unit = vec ? 32u * nv : 32u * R; // nodes per warp pass
    const uint32_t passes = (max_rows + unit - 1u) / unit;
    uint64_t ppc = ((uint64_t)n * passes + want_ctas - 1) / want_ctas; // passes per block
    ppc = std::min<uint64_t>(std::max<uint64_t>(ppc, 1), passes);
    const uint32_t rounds = (uint32_t)((ppc + 7) / 8);
    const uint32_t warps = split ? SLONN_SPLIT_WARPS : std::max(vec ? 1u : 4u, (uint32_t)((ppc + rounds - 1) / rounds));
    P.rows_per_cta = (uint32_t)ppc * unit;
    P.ctas_per_query = (max_rows + P.rows_per_cta - 1) / P.rows_per_cta;
    P.rows_cap = max_rows;
    size_t scratch = cols_image_bytes(P.D, bf ? 8u : 4u);
    if (P.use_list && P.colpos) scratch = std::max(scratch, ((size_t)2 * ((P.N + 31u) / 32u) + (size_t)3 * max_rows) * 4);
    scratch = (scratch + 15) & ~(size_t)15;
    P.scratch_bytes = (uint32_t)scratch;
    const size_t smem = scratch + (size_t)cols_ent_cap(P.D, P.in_cap) * 8 + (split ? (size_t)32 * R * 32 * 4 : 0);
    if (smem > 200 * 1024) return SLONN_ERR_DIM; // caller falls back to the row kernel
    const uint64_t grid = (uint64_t)n * P.ctas_per_query;
    if (grid == 0 || grid > 0x7fffffffull) return SLONN_ERR_DIM;
    if (split)
        return bf ? launch_gather_cols_t<true, SLONN_COLS_R, true>(P, grid, warps * 32u, smem, st)
                  : launch_gather_cols_t<false, SLONN_COLS_R, true>(P, grid, warps * 32u, smem, st);
    if (vec)
        return bf ? launch_gather_cols_t<true, SLONN_COLS_R, false, true>(P, grid, warps * 32u, smem, st)
                  : launch_gather_cols_t<false, SLONN_COLS_R, false, true>(P, grid, warps * 32u, smem, st);
    return bf ? launch_gather_cols_t<true, SLONN_COLS_R, false>(P, grid, warps * 32u, smem, st)
              : launch_gather_cols_t<false, SLONN_COLS_R, false>(P, grid, warps * 32u, smem, st);
}

template <bool BF16, typename IDT, bool SPLIT, bool TIGHT>
int launch_layer_cols_t(const slonn_layer_cols_params &Q, uint64_t grid, uint32_t threads, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(layer_cols_kernel<BF16, IDT, SPLIT, TIGHT>, smem);
    if (rc) return rc;
    layer_cols_kernel<BF16, IDT, SPLIT, TIGHT><<<(uint32_t)grid, threads, smem, st>>>(Q);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

template <bool BF16, typename IDT>
int launch_layer_cols_s(const slonn_layer_cols_params &Q, bool split, uint64_t grid, uint32_t threads, size_t smem, cudaStream_t st)
{
    if (split) return launch_layer_cols_t<BF16, IDT, true, false>(Q, grid, threads, smem, st);
    // blocks of at most seven warps: the 40-register instantiation, seven of them per SM
    return threads <= 224u ? launch_layer_cols_t<BF16, IDT, false, true>(Q, grid, threads, smem, st)
                           : launch_layer_cols_t<BF16, IDT, false, false>(Q, grid, threads, smem, st);
}

// Hash, selection and input-stationary gather of a list-fed activator layer in one launch: one block per
// query, or, for batches of tens of queries, one block per (query, 64 nodes) with the selection repeated in
// every block of a query.  SLONN_ERR_DIM: not applicable here (no side-by-side hash rows, or the staging
// does not fit) -- the caller takes the separate kernels.
int launch_layer_cols(const slonn_model *m, const slonn_layer &ly, uint32_t layer, slonn_gather_params G,
                      const slonn_batch *b, uint32_t n, uint32_t max_rows, cudaStream_t st)
{
    if (!ly.WH || !ly.WT || !ly.colpos || !G.use_list) return SLONN_ERR_DIM;
    const uint32_t passes = (max_rows + 63u) / 64u;
    const bool split = (uint64_t)n * passes < 148ull * 8; // whole queries per block would leave SMs idle
    const uint32_t rounds = (passes + 7) / 8;
    const uint32_t warps = split ? SLONN_SPLIT_WARPS : std::max(4u, (passes + rounds - 1) / rounds);
    const bool bf = m->dtype == SLONN_BF16;
    G.rows_cap = max_rows;
    G.rows_per_cta = split ? 64u : passes * 64u;
    G.ctas_per_query = split ? passes : 1u;
    size_t scratch = cols_image_bytes(G.D, bf ? 8u : 4u);
    scratch = std::max(scratch, ((size_t)2 * ((G.N + 31u) / 32u) + (size_t)3 * max_rows) * 4);
    scratch = std::max(scratch, (size_t)32 * 32 * 4); // the hash functions' partial sums pass through it
    scratch = (scratch + 15) & ~(size_t)15;
    G.scratch_bytes = (uint32_t)scratch;
    const size_t smem = scratch + (size_t)cols_ent_cap(G.D, G.in_cap) * 8 + (size_t)((G.N + 31u) / 32u) * 4 +
                        (split ? (size_t)32 * 2 * 32 * 4 + (size_t)max_rows * 4 : 0);
    if (smem > 200 * 1024) return SLONN_ERR_DIM;
    const uint64_t grid = (uint64_t)n * G.ctas_per_query;
    if (grid == 0 || grid > 0x7fffffffull) return SLONN_ERR_DIM;
    slonn_layer_cols_params Q;
    memset(&Q, 0, sizeof(Q));
    Q.G = G; Q.WH = ly.WH; Q.hash_nodes = ly.hash_nodes; Q.tables = ly.tables; Q.cap = ly.cap;
    Q.K = m->K; Q.L = m->L; Q.pre = slonn_model_pre(m); Q.layer = layer; Q.codes = b->codes; Q.status = b->status;
    const bool id16 = ly.id_bytes == 2;
    if (bf) return id16 ? launch_layer_cols_s<true, uint16_t>(Q, split, grid, warps * 32u, smem, st) : launch_layer_cols_s<true, uint32_t>(Q, split, grid, warps * 32u, smem, st);
    return id16 ? launch_layer_cols_s<false, uint16_t>(Q, split, grid, warps * 32u, smem, st) : launch_layer_cols_s<false, uint32_t>(Q, split, grid, warps * 32u, smem, st);
}

// Budgets 1..limit take the input-stationary kernels in this layer (0: none do).
uint32_t cols_budget_limit(const slonn_layer &ly, const slonn_gather_params &P, const slonn_batch *b, uint32_t n, uint32_t max_rows,
                           uint32_t max_bp)
{
    if (!ly.WT || P.in.kind != SLONN_IN_LIST || (b->flags & SLONN_FLAG_ROW_KERNELS)) return 0;
    if (b->flags & SLONN_FLAG_COLUMN_KERNELS) return (uint64_t)n * max_rows > 148ull * 64 ? 10000u : 0u;
    if ((uint64_t)n * max_rows >= 148ull * 1024) return SLONN_COLS_MAX_BP;
    // tens of queries: the one-block-per-64-nodes variant pays only for long weight rows and very sparse lists
    // (4096-wide nine-layer network, 64 queries: 0.36 -> 0.30 ms per step at 10 %, but 0.57 -> 0.92 ms at 25 %)
    // and only when no query of the batch needs the row kernels (a second launch of idle blocks costs such a batch 6 %)
    return ((uint64_t)n * max_rows > 148ull * 64 && ly.D >= 2048u && max_bp <= 1500u) ? 1500u : 0u;
}

// Rows of one layer for a batch whose layer input is `P.in`: the input-stationary kernel for the queries
// whose input list is sparse (by budget), the row kernel for the others.  Results do not depend on the split.
// rows_done: the queries above the input-stationary limit were served by another launch already.
int launch_layer_rows(const slonn_model *m, const slonn_layer &ly, slonn_gather_params &P, const slonn_batch *b,
                      uint32_t n, uint32_t max_bp, uint32_t max_rows, uint32_t in_cap, const group_ws &gw, cudaStream_t st,
                      stage_timer *tm, bool rows_done = false)
{
    const uint32_t cols_bp = cols_budget_limit(ly, P, b, n, max_rows, max_bp);
    int rc;
    if (!cols_bp && rows_done) return SLONN_OK;
    if (cols_bp) {
        const bool both = max_bp > cols_bp;
        slonn_gather_params C = P;
        C.WT = ly.WT; C.colpos = ly.colpos;
        if (both) { C.range_bp = b->budget_bp; C.bp_lo = 0; C.bp_hi = cols_bp; }
        // the blocks of a launch are sized for the largest budget it serves
        const uint32_t pre = slonn_model_pre(m);
        const uint32_t cols_rows = (both && P.use_list) ? std::min(max_rows, slonn_layer_nodes(cols_bp, ly.N, pre)) : max_rows;
        C.in_cap = both ? std::min(in_cap, slonn_layer_nodes(cols_bp, ly.D, pre)) : in_cap;
        TIC(SLONN_STAGE_GATHER_COLS, C.range_bp, C.bp_lo, C.bp_hi, C.skip_bp);
        rc = launch_gather_cols(m, C, n, cols_rows, st);
        TOC();
        if (rc != SLONN_ERR_DIM) { // SLONN_ERR_DIM: the staging does not fit shared memory, rows for everyone
            if (rc || !both || rows_done) return rc;
            P.range_bp = b->budget_bp; P.bp_lo = cols_bp + 1; P.bp_hi = 0xffffu;
        } else if (rows_done) { // only the low budgets are still open
            P.range_bp = b->budget_bp; P.bp_lo = 0; P.bp_hi = cols_bp;
        }
    }
    return launch_rows(m, P, b, n, max_bp, max_rows, gw, st, tm);
}

// An activator layer: FreeHash, selection and the selected nodes.  A list-fed layer with the copies for it
// runs as ONE input-stationary launch for the queries whose budget leaves the list sparse; the others (and
// every query where that launch does not apply) take the selection kernel followed by the row or
// input-stationary gather.
int launch_act_layer(const slonn_model *m, const slonn_layer &ly, uint32_t l, slonn_select_params &sp, slonn_gather_params &gp,
                     const slonn_batch *b, uint32_t n, uint32_t max_bp, uint32_t max_rows, uint32_t in_cap, const group_ws &gw,
                     cudaStream_t st, stage_timer *tm)
{
    int rc;
    const uint32_t cols_bp = cols_budget_limit(ly, gp, b, n, max_rows, max_bp);
    if (cols_bp && ly.WH) {
        const bool both = max_bp > cols_bp;
        const uint32_t pre = slonn_model_pre(m);
        slonn_gather_params C = gp;
        C.WT = ly.WT; C.colpos = ly.colpos;
        if (both) { C.range_bp = b->budget_bp; C.bp_lo = 0; C.bp_hi = cols_bp; }
        const uint32_t cols_rows = both ? std::min(max_rows, slonn_layer_nodes(cols_bp, ly.N, pre)) : max_rows;
        C.in_cap = both ? std::min(in_cap, slonn_layer_nodes(cols_bp, ly.D, pre)) : in_cap;
        TIC(SLONN_STAGE_LAYER_COLS, C.range_bp, C.bp_lo, C.bp_hi, C.skip_bp);
        rc = launch_layer_cols(m, ly, l, C, b, n, cols_rows, st);
        TOC();
        if (rc == SLONN_OK) {
            if (!both) return SLONN_OK;
            sp.range_bp = b->budget_bp; sp.bp_lo = cols_bp + 1; sp.bp_hi = 0xffffu;
            TIC(SLONN_STAGE_HASH_SELECT, sp.range_bp, sp.bp_lo, sp.bp_hi, sp.skip_bp);
            rc = launch_select(m, sp, n, max_rows, st);
            TOC();
            if (rc) return rc;
            gp.range_bp = b->budget_bp; gp.bp_lo = cols_bp + 1; gp.bp_hi = 0xffffu;
            return launch_rows(m, gp, b, n, max_bp, max_rows, gw, st, tm);
        }
        if (rc != SLONN_ERR_DIM) return rc;
    }
    TIC(SLONN_STAGE_HASH_SELECT, sp.range_bp, sp.bp_lo, sp.bp_hi, sp.skip_bp);
    rc = launch_select(m, sp, n, max_rows, st);
    TOC();
    if (rc) return rc;
    return launch_layer_rows(m, ly, gp, b, n, max_bp, max_rows, in_cap, gw, st, tm);
}

// ---- 100 % queries, four per block ---------------------------------------------

template <bool BF16>
int launch_full_rows_t(const slonn_full_params &P, uint64_t grid, size_t smem, cudaStream_t st)
{
    const int rc = set_smem(full_rows_kernel<BF16, SLONN_FULL_R>, smem);
    if (rc) return rc;
    full_rows_kernel<BF16, SLONN_FULL_R><<<(uint32_t)grid, SLONN_THREADS, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

// SLONN_ERR_DIM: four staged inputs do not fit shared memory (the caller leaves these queries to the other kernels,
// which it can only decide before the first layer: see full_route_fits)
int launch_full_rows(const slonn_model *m, slonn_full_params &P, uint32_t n, cudaStream_t st)
{
    const uint32_t groups = (n + SLONN_FULL_GROUP - 1) / SLONN_FULL_GROUP;
    P.rows_per_cta = std::min((P.N + 31u) / 32u * 32u, 1024u);
    P.ctas_per_group = (P.N + P.rows_per_cta - 1) / P.rows_per_cta;
    const size_t smem = (size_t)SLONN_FULL_GROUP * P.D * 4;
    const uint64_t grid = (uint64_t)groups * P.ctas_per_group;
    if (grid == 0 || grid > 0x7fffffffull || smem > 200 * 1024) return SLONN_ERR_DIM;
    return m->dtype == SLONN_BF16 ? launch_full_rows_t<true>(P, grid, smem, st) : launch_full_rows_t<false>(P, grid, smem, st);
}

bool full_route_fits(const slonn_model *m)
{
    for (uint32_t l = 0; l < m->n_layers; ++l)
        if ((size_t)SLONN_FULL_GROUP * m->layer[l].D * 4 > 200 * 1024) return false;
    return true;
}

// ---- whole-network kernel for narrow layers -----------------------------------

#ifndef SLONN_FUSED_COLS_MAX_BP
#define SLONN_FUSED_COLS_MAX_BP 1250u // batches whose largest budget is at most this take the input-stationary form
#endif

bool fused_eligible(const slonn_model *m)
{
    if (m->first_sparse) return false;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        if (ly.D > SLONN_FUSED_MAX_D || ly.N > SLONN_FUSED_MAX_N) return false;
    }
    return true;
}

template <bool BF16, int NC, int GRP, bool COLS>
int launch_fused_g(const slonn_fused_params &P, cudaStream_t st)
{
    const size_t smem = (size_t)P.warp_bytes * SLONN_FUSED_WARPS;
    int rc = set_smem(fused_network_kernel<BF16, NC, GRP, COLS>, smem);
    if (rc) return rc;
    const uint32_t grid = (P.n + SLONN_FUSED_WARPS - 1) / SLONN_FUSED_WARPS;
    fused_network_kernel<BF16, NC, GRP, COLS><<<grid, SLONN_FUSED_WARPS * 32, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

// Batches of at most two blocks per SM: up to four load rounds of a row pass in flight at once (the few
// resident warps can have all the registers); larger batches: one round, five blocks per SM.
template <bool BF16, int NC>
int launch_fused_t(const slonn_fused_params &P, cudaStream_t st)
{
    const uint32_t grid = (P.n + SLONN_FUSED_WARPS - 1) / SLONN_FUSED_WARPS;
    if (NC > 1 && grid <= 2u * 148u)
        return P.cols_bp ? launch_fused_g<BF16, NC, (NC > 4 ? 4 : NC), true>(P, st) : launch_fused_g<BF16, NC, (NC > 4 ? 4 : NC), false>(P, st);
    return P.cols_bp ? launch_fused_g<BF16, NC, 1, true>(P, st) : launch_fused_g<BF16, NC, 1, false>(P, st);
}

int launch_fused(const slonn_model *m, const slonn_batch *b, const uint64_t *indptr, uint32_t stride,
                 const uint16_t *skip_bp, uint32_t max_bp, cudaStream_t st, uint32_t *cols_bp_out)
{
    slonn_fused_params P;
    memset(&P, 0, sizeof(P));
    const uint32_t esz = m->dtype == SLONN_BF16 ? 2u : 4u;
    uint32_t max_rounds = 1, xbuf = 4, ids_cap = 8, words = 1, ent_cap = 0;
    // budgets that take the input-stationary form in layers that offer it
    // (the grouped input list lives in shared memory, which it takes from the L1 cache the row form relies on:
    // only batches whose every budget is low carry it, unless the caller forces it)
    const uint32_t cols_bp = (b->flags & SLONN_FLAG_ROW_KERNELS) ? 0u : (b->flags & SLONN_FLAG_COLUMN_KERNELS) ? 10000u
                             : max_bp <= SLONN_FUSED_COLS_MAX_BP ? SLONN_FUSED_COLS_MAX_BP : 0u;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        slonn_fused_layer &f = P.layer[l];
        f.W = ly.W; f.bias = ly.bias; f.hash_nodes = ly.hash_nodes; f.tables = ly.tables;
        f.D = ly.D; f.N = ly.N; f.nchunks = ly.D * esz / 16u; f.cap = ly.cap;
        f.has_act = ly.has_act; f.a = m->act_index[l]; f.relu = (l + 1 == m->n_layers) ? 0u : 1u;
        f.id_bytes = ly.id_bytes;
        f.WT = ly.WT; f.WH = ly.WH; f.colpos = ly.colpos;
        if (cols_bp && l > 0 && ly.has_act && ly.WT && ly.WH && ly.colpos && m->layer[l - 1].has_act)
            ent_cap = std::max(ent_cap, slonn_layer_nodes(std::min(max_bp, cols_bp), ly.D, slonn_model_pre(m)) + 96u);
        max_rounds = std::max(max_rounds, (f.nchunks + 31u) / 32u);
        if (l > 0) xbuf = std::max(xbuf, (ly.D + 3u) / 4u * 4u);
        if (ly.has_act) {
            ids_cap = std::max(ids_cap, (ly.N + 7u) / 8u * 8u);
            words = std::max(words, (ly.N + 31u) / 32u);
        }
    }
    P.n_layers = m->n_layers; P.n = b->n_queries; P.n_act = m->n_act; P.K = m->K; P.L = m->L;
    P.pre = slonn_model_pre(m);
    P.x = b->x_dense; P.indptr = indptr; P.skip_bp = skip_bp; P.max_bp = max_bp;
    P.out_ids = b->active_ids; P.out_vals = b->active_vals; P.codes = b->codes;
    P.logits = b->logits; P.logit_stride = stride; P.logit_ids = b->logit_ids; P.pred = b->pred;
    P.status = b->status;
    P.xbuf_floats = xbuf; P.ids_cap = ids_cap; P.bitmap_words = words;
    P.cols_bp = ent_cap ? cols_bp : 0u; P.ent_cap = ent_cap; P.budget_bp = b->budget_bp;
    *cols_bp_out = P.cols_bp;
    P.warp_bytes = (uint32_t)align_up(align_up((uint64_t)xbuf * 4 + (uint64_t)ids_cap * 2 + (uint64_t)words * 4, 16) +
                                          (ent_cap ? (uint64_t)ent_cap * 8 + 66 * 4 : 0), 16);
    const bool bf = m->dtype == SLONN_BF16;
    if (bf) {
        if (max_rounds <= 1) return launch_fused_t<true, 1>(P, st);
        if (max_rounds <= 2) return launch_fused_t<true, 2>(P, st);
        if (max_rounds <= 4) return launch_fused_t<true, 4>(P, st);
    } else {
        if (max_rounds <= 1) return launch_fused_t<false, 1>(P, st);
        if (max_rounds <= 2) return launch_fused_t<false, 2>(P, st);
        if (max_rounds <= 4) return launch_fused_t<false, 4>(P, st);
        if (max_rounds <= 8) return launch_fused_t<false, 8>(P, st);
    }
    return SLONN_ERR_DIM;
}

// ---- one cluster per query: latency path for a handful of queries ---------------

// One block of four warps per query (the cluster kernel with a cluster of one): chosen for narrow networks when the
// batch has at most 512 queries (four resident blocks of 128 registers per SM: 592 at a time) and no layer computes
// more than 64 rows per query.  Measured on 784-112-112-10 fp32, 256 queries: 37 us at a 10 % budget against 59 us
// with the per-stage kernels and 43 us with one warp per query; with 102 rows per layer (784-1024-1024-10) the
// per-stage kernels win, and beyond one wave of blocks one warp per query does.  Six or eight resident blocks spill.
#ifndef SLONN_BLOCK_MINB
#define SLONN_BLOCK_MINB 4
#endif
#ifndef SLONN_BLOCK_PATH_MAX_QUERIES
#define SLONN_BLOCK_PATH_MAX_QUERIES 512u
#endif
#define SLONN_BLOCK_PATH_MAX_ROWS 64u
bool cluster_eligible(const slonn_model *m)
{
    if (m->first_sparse) return false;
    for (uint32_t l = 0; l < m->n_layers; ++l)
        if (m->layer[l].D > SLONN_CLUSTER_MAX_D || m->layer[l].N > SLONN_CLUSTER_MAX_N) return false;
    return true;
}

// most rows any layer computes for one query at this budget
uint32_t cluster_max_rows(const slonn_model *m, uint32_t max_bp)
{
    uint32_t r = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l)
        r = std::max(r, m->layer[l].has_act ? slonn_layer_nodes(max_bp, m->layer[l].N, slonn_model_pre(m)) : m->layer[l].N);
    return r;
}

template <bool BF16, int THREADS, int MIN_BLOCKS>
int launch_cluster_t(const slonn_cluster_params &P, size_t smem, cudaStream_t st)
{
    auto kernel = cluster_network_kernel<BF16, THREADS, MIN_BLOCKS>;
    { const int rc = slonn_allow_smem(reinterpret_cast<const void *>(kernel), smem); if (rc) return rc; }
    if (P.cluster > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        return SLONN_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(P.n * P.cluster, 1, 1);
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = P.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0; // the device must be able to co-schedule at least one such cluster
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess || clusters < 1) {
        cudaGetLastError();
        return SLONN_ERR_DIM;
    }
    return cudaLaunchKernelEx(&cfg, kernel, P) == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

// cluster_size 16: a handful of queries, 512 threads per block.  cluster_size 1: one block of four warps per query
// (narrow networks, batches up to a few thousand queries); indptr_in: the planned offsets when lists are written.
int launch_cluster(const slonn_model *m, const slonn_batch *b, uint32_t max_bp, uint32_t stride, cudaStream_t st,
                   uint32_t cluster_size = SLONN_CLUSTER_SIZE, const uint64_t *indptr_in = nullptr)
{
    slonn_cluster_params P;
    memset(&P, 0, sizeof(P));
    const uint32_t esz = m->dtype == SLONN_BF16 ? 2u : 4u;
    uint32_t xbuf = 4, ids_cap = 4, words = 1;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        slonn_cluster_layer &f = P.layer[l];
        f.W = ly.W; f.bias = ly.bias; f.hash_nodes = ly.hash_nodes; f.tables = ly.tables;
        f.D = ly.D; f.N = ly.N; f.nchunks = ly.D * esz / 16u; f.cap = ly.cap;
        f.has_act = ly.has_act; f.a = m->act_index[l]; f.relu = (l + 1 == m->n_layers) ? 0u : 1u;
        f.id_bytes = ly.id_bytes;
        xbuf = std::max(xbuf, std::max((ly.D + 3u) / 4u * 4u, (ly.N + 3u) / 4u * 4u));
        if (ly.has_act) {
            ids_cap = std::max(ids_cap, (ly.N + 3u) / 4u * 4u);
            words = std::max(words, (ly.N + 31u) / 32u);
        }
    }
    P.n_layers = m->n_layers; P.n = b->n_queries; P.n_act = m->n_act; P.K = m->K; P.L = m->L; P.cluster = cluster_size;
    P.pre = slonn_model_pre(m);
    P.x = b->x_dense; P.budget_bp = b->budget_bp; P.max_bp = max_bp;
    P.indptr_in = indptr_in; P.indptr_out = indptr_in ? nullptr : b->active_indptr;
    P.out_ids = b->active_ids; P.out_vals = b->active_vals; P.codes = b->codes;
    P.logits = b->logits; P.logit_stride = stride; P.logit_ids = b->logit_ids; P.pred = b->pred;
    P.status = b->status;
    P.xbuf_floats = xbuf; P.ids_cap = ids_cap; P.bitmap_words = words;
    const size_t smem = (size_t)xbuf * 8 + (size_t)ids_cap * 4 + (size_t)words * 4;
    if (smem > 200 * 1024) return SLONN_ERR_DIM;
    if (cluster_size == 1)
        return m->dtype == SLONN_BF16 ? launch_cluster_t<true, 128, SLONN_BLOCK_MINB>(P, smem, st) : launch_cluster_t<false, 128, SLONN_BLOCK_MINB>(P, smem, st);
    return m->dtype == SLONN_BF16 ? launch_cluster_t<true, SLONN_CLUSTER_THREADS, 1>(P, smem, st)
                                  : launch_cluster_t<false, SLONN_CLUSTER_THREADS, 1>(P, smem, st);
}

} // namespace

// ---- internal entry points used by the table builder --------------------------

// Complete layer l (every node) for n dense input rows -> out [n][N_l].
int slonn_forward_all_rows(const slonn_model *m, uint32_t l, const float *in_dense, uint32_t n, float *out,
                           uint32_t relu, cudaStream_t st)
{
    const slonn_layer &ly = m->layer[l];
    slonn_gather_params gp;
    memset(&gp, 0, sizeof(gp));
    gp.in.kind = SLONN_IN_DENSE; gp.in.dense = in_dense;
    gp.W = ly.W; gp.bias = ly.bias; gp.D = ly.D; gp.N = ly.N;
    gp.nchunks = ly.D * (m->dtype == SLONN_BF16 ? 2u : 4u) / 16u;
    gp.use_list = 0; gp.out_dense = out; gp.out_stride = ly.N; gp.relu = relu;
    return launch_gather(m, gp, n, ly.N, st);
}

// Complete layer 0 for n CSR rows -> out [n][N_0].
int slonn_forward_sparse_first(const slonn_model *m, const uint64_t *indptr, const uint32_t *ids,
                               const float *vals, uint32_t n, float *out, uint32_t relu, uint32_t *status,
                               cudaStream_t st)
{
    const slonn_layer &ly = m->layer[0];
    slonn_sparse_params sp;
    memset(&sp, 0, sizeof(sp));
    sp.x_indptr = indptr; sp.x_ids = ids; sp.x_vals = vals;
    sp.WT = ly.WT; sp.bias = ly.bias; sp.D = ly.D; sp.N = ly.N;
    sp.out_dense = out; sp.out_stride = ly.N; sp.relu = relu;
    sp.blocks_per_query = (ly.N + 127u) / 128u;
    sp.status = status;
    const uint64_t grid = (uint64_t)n * sp.blocks_per_query;
    if (grid == 0 || grid > 0x7fffffffull) return SLONN_ERR_DIM;
    if (m->dtype == SLONN_BF16) sparse_first_layer_kernel<true><<<(uint32_t)grid, 128, 0, st>>>(sp);
    else sparse_first_layer_kernel<false><<<(uint32_t)grid, 128, 0, st>>>(sp);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

extern "C" int slonn_active_capacity(const slonn_model *m, uint32_t n, uint32_t max_bp, uint64_t *entries)
{
    if (!model_ok(m) || !entries) return SLONN_ERR_ARG;
    *entries = active_entries(m, n, eff_max_bp(max_bp));
    return SLONN_OK;
}

extern "C" int slonn_logit_stride(const slonn_model *m, uint32_t max_bp, uint32_t *stride)
{
    if (!model_ok(m) || !stride) return SLONN_ERR_ARG;
    const slonn_layer &last = m->layer[m->n_layers - 1];
    *stride = last.has_act ? slonn_layer_nodes(eff_max_bp(max_bp), last.N, slonn_model_pre(m)) : last.N;
    return SLONN_OK;
}

extern "C" int slonn_workspace_bytes(const slonn_model *m, uint32_t n, uint32_t max_bp, uint32_t flags,
                                     uint64_t *bytes)
{
    if (!model_ok(m) || !bytes) return SLONN_ERR_ARG;
    *bytes = carve(m, n, eff_max_bp(max_bp), flags).total;
    return SLONN_OK;
}

// Every layer for the batch's 100 % queries (compacted in `list` / `count`), four queries per block.  They share
// nothing with the other queries but the output arrays (disjoint entries), so this runs as a pass of its own.
static int run_full_route(const slonn_model *m, const slonn_batch *b, uint32_t n, const uint32_t *list, const uint32_t *count,
                          const uint64_t *indptr, uint32_t *ids, float *vals, float *const dense[2], uint32_t stride,
                          cudaStream_t st, stage_timer *tm)
{
    slonn_input in;
    memset(&in, 0, sizeof(in));
    in.kind = SLONN_IN_DENSE;
    in.dense = b->x_dense;
    int dense_cur = 0;
    const uint32_t esz = m->dtype == SLONN_BF16 ? 2u : 4u;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        const bool is_last = (l + 1 == m->n_layers);
        slonn_full_params fp;
        memset(&fp, 0, sizeof(fp));
        fp.list = list; fp.count = count; fp.in = in;
        fp.W = ly.W; fp.bias = ly.bias; fp.D = ly.D; fp.N = ly.N; fp.nchunks = ly.D * esz / 16u;
        fp.has_act = ly.has_act; fp.n_act = m->n_act; fp.a = m->act_index[l]; fp.indptr = indptr;
        fp.out_ids = ids; fp.out_vals = vals; fp.relu = is_last ? 0u : 1u;
        if (ly.has_act) {
            if (is_last) { fp.out_dense = b->logits; fp.out_dense_ids = b->logit_ids; fp.out_stride = stride; }
        } else {
            fp.out_dense = is_last ? b->logits : dense[dense_cur];
            fp.out_stride = ly.N;
        }
        AT_LAYER(l);
        TIC(SLONN_STAGE_FULL_ROWS, b->budget_bp, 10000u, 10000u);
        const int rc = launch_full_rows(m, fp, n, st);
        TOC();
        if (rc) return rc;
        if (ly.has_act) {
            if (b->codes) { // keys from the signs of the hash nodes' values (every node was computed)
                const uint32_t t = n * m->L;
                dense_codes_kernel<<<(t + 127) / 128, 128, 0, st>>>(list, count, vals, indptr, m->n_act, m->act_index[l],
                                                                   ly.hash_nodes, m->K, m->L, b->codes);
                if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
            }
            in.kind = SLONN_IN_LIST; in.indptr = indptr; in.ids = ids; in.vals = vals;
            in.ip_mul = m->n_act; in.ip_add = m->act_index[l];
        } else {
            in.kind = SLONN_IN_DENSE; in.dense = fp.out_dense;
            dense_cur ^= 1;
        }
    }
    return SLONN_OK;
}

// whether the batch's 100 % queries are taken out of the per-query kernels and run four per block: the batch must be
// able to hold some (largest budget 100 %), and be large enough for the extra launches to vanish in the work
static bool full_route_wanted(const slonn_model *m, uint32_t n, uint32_t max_bp)
{
    if (!full_route_possible(m, max_bp) || !full_route_fits(m) || n < 256) return false;
    uint64_t weights = 0;
    for (uint32_t l = 0; l < m->n_layers; ++l) weights += (uint64_t)m->layer[l].N * m->layer[l].D;
    return (uint64_t)n * weights >= (1ull << 32);
}

static int run_impl(const slonn_model *m, const slonn_batch *b, void *workspace, uint64_t ws_bytes,
                    void *stream, stage_timer *tm)
{
    if (!model_ok(m) || !b || !b->status) return SLONN_ERR_ARG;
    const uint32_t n = b->n_queries;
    const uint32_t max_bp = eff_max_bp(b->max_budget_bp);
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(b->status, 0, 4 * sizeof(uint32_t), st) != cudaSuccess) return SLONN_ERR_CUDA;
    if (n == 0) return SLONN_OK; // an empty batch needs no other buffer
    if (!b->budget_bp || !b->logits) return SLONN_ERR_ARG;
    if (m->first_sparse ? (!b->x_indptr || !b->x_ids || !b->x_vals) : !b->x_dense) return SLONN_ERR_ARG;
    const slonn_layer &last = m->layer[m->n_layers - 1];
    if (last.has_act && !b->logit_ids) return SLONN_ERR_ARG;
    if (b->x_dense && ((uintptr_t)b->x_dense & 15u)) return SLONN_ERR_ALIGN;

    const ws_layout wl = carve(m, n, max_bp, b->flags);
    if (!workspace || ((uintptr_t)workspace & 255u) || ws_bytes < wl.total) return SLONN_ERR_WORKSPACE;
    char *ws = (char *)workspace;
    uint64_t *indptr = b->active_indptr ? b->active_indptr : (uint64_t *)(ws + wl.indptr);
    uint32_t *ids = b->active_ids ? b->active_ids : (uint32_t *)(ws + wl.ids);
    float *vals = b->active_vals ? b->active_vals : (float *)(ws + wl.vals);
    float *dense[2] = {(float *)(ws + wl.dense0), (float *)(ws + wl.dense1)};

    uint32_t stride = 0;
    slonn_logit_stride(m, max_bp, &stride);

    // a handful of queries: one thread-block cluster per query, every layer in one launch (it derives the
    // list offsets itself, so no planning launch either)
    if (b->flags & ~SLONN_FLAG_ALL) return SLONN_ERR_ARG;
    if ((b->flags & SLONN_FLAG_ROW_KERNELS) && (b->flags & SLONN_FLAG_COLUMN_KERNELS)) return SLONN_ERR_ARG;
    if (b->kernel_path > SLONN_PATH_BLOCK) return SLONN_ERR_ARG;
    if (b->kernel_path == SLONN_PATH_CLUSTER && (!cluster_eligible(m) || tc_route(m, max_bp, b->flags))) return SLONN_ERR_DIM;
    if (b->kernel_path == SLONN_PATH_CLUSTER || (b->kernel_path == SLONN_PATH_AUTO && cluster_eligible(m) && n <= 4 && !tc_route(m, max_bp, b->flags) &&
         cluster_max_rows(m, max_bp) <= 1024)) {
        AT_LAYER(SLONN_ALL_LAYERS);
        TIC(SLONN_STAGE_CLUSTER);
        const int rc = launch_cluster(m, b, max_bp, stride, st);
        TOC();
        if (rc != SLONN_ERR_DIM || b->kernel_path == SLONN_PATH_CLUSTER) return rc;
        // the device cannot co-schedule such a cluster: fall through to the other kernels
    }

    // narrow networks with enough queries to fill the GPU take the one-warp-per-query kernel; when the
    // caller wants no active lists back it needs no list offsets either (each warp derives its node
    // counts from the budget), which saves the two planning launches
    if (b->kernel_path == SLONN_PATH_FUSED && !fused_eligible(m)) return SLONN_ERR_DIM;
    if (b->kernel_path == SLONN_PATH_BLOCK && (!fused_eligible(m) || tc_route(m, max_bp, b->flags))) return SLONN_ERR_DIM;
    const bool full_route = !tc_route(m, max_bp, b->flags) && full_route_wanted(m, n, max_bp);
    // narrow networks at batches too small to fill the GPU with one warp per query: one block of four warps per query
    const bool use_block = b->kernel_path == SLONN_PATH_BLOCK ||
                           (b->kernel_path == SLONN_PATH_AUTO && fused_eligible(m) && n <= SLONN_BLOCK_PATH_MAX_QUERIES &&
                            cluster_max_rows(m, max_bp) <= SLONN_BLOCK_PATH_MAX_ROWS && !tc_route(m, max_bp, b->flags) && !full_route);
    const bool use_fused = !use_block && (b->kernel_path == SLONN_PATH_FUSED || (b->kernel_path == SLONN_PATH_AUTO && fused_eligible(m) && n >= 512));
    const bool no_plan = (use_fused || use_block) && !tc_route(m, max_bp, b->flags) && !full_route && !b->active_indptr && !b->active_ids &&
                         !b->active_vals;

    // offsets of every (query, activator layer) list
    if (m->n_act && !no_plan) {
        slonn_plan_params pp;
        memset(&pp, 0, sizeof(pp));
        pp.budget_bp = b->budget_bp; pp.n = n; pp.n_act = m->n_act; pp.max_bp = max_bp;
        pp.pre = slonn_model_pre(m);
        for (uint32_t l = 0; l < m->n_layers; ++l)
            if (m->layer[l].has_act) {
                const uint32_t a = m->act_index[l];
                pp.act_N[a] = m->layer[l].N; pp.act_cap[a] = m->layer[l].cap; pp.act_layer[a] = l;
            }
        pp.indptr = indptr; pp.status = b->status;
        const uint64_t tiles = ((uint64_t)n * m->n_act + SLONN_PLAN_TILE - 1) / SLONN_PLAN_TILE;
        uint64_t *tile_sums = (uint64_t *)(ws + wl.plan_sums);
        AT_LAYER(SLONN_ALL_LAYERS);
        TIC(SLONN_STAGE_PLAN);
        plan_partial_kernel<<<(uint32_t)tiles, SLONN_PLAN_THREADS, 0, st>>>(pp, tile_sums);
        plan_final_kernel<<<(uint32_t)tiles, SLONN_PLAN_THREADS, 0, st>>>(pp, tile_sums);
        TOC();
        if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
    }

    if (use_block) {
        AT_LAYER(SLONN_ALL_LAYERS);
        TIC(SLONN_STAGE_CLUSTER);
        const int rc = launch_cluster(m, b, max_bp, stride, st, 1u, no_plan ? nullptr : indptr);
        TOC();
        if (rc != SLONN_ERR_DIM || b->kernel_path == SLONN_PATH_BLOCK) return rc;
        // the staging does not fit: fall through to the other kernels (the offsets are planned already)
    }

    // queries at a 100 % budget on the tensor cores (on request): they compute every node of every
    // layer, so they are a dense matrix product over the compacted set of such queries
    const uint16_t *skip_bp = nullptr;
    if (tc_route(m, max_bp, b->flags)) {
        uint32_t *tc_list = (uint32_t *)(ws + wl.tc_list), *tc_count = (uint32_t *)(ws + wl.tc_count);
        uint16_t *A[2] = {(uint16_t *)(ws + wl.tc_a0), (uint16_t *)(ws + wl.tc_a1)};
        AT_LAYER(SLONN_ALL_LAYERS);
        TIC(SLONN_STAGE_DENSE_TC, b->budget_bp, 10000u, 10000u);
        int rc = SLONN_OK;
        if (cudaMemsetAsync(tc_count, 0, sizeof(uint32_t), st) != cudaSuccess) rc = SLONN_ERR_CUDA;
        if (!rc) {
            dense_compact_kernel<<<(n + 255) / 256, 256, 0, st>>>(b->budget_bp, n, tc_list, tc_count);
            dense_gather_x_kernel<<<n, 128, 0, st>>>(b->x_dense, m->layer[0].D, tc_list, tc_count, A[0]);
            if (cudaGetLastError() != cudaSuccess) rc = SLONN_ERR_CUDA;
        }
        for (uint32_t l = 0; l < m->n_layers && !rc; ++l) {
            const slonn_layer &ly = m->layer[l];
            const bool is_last = (l + 1 == m->n_layers);
            slonn_dense_epilogue E;
            memset(&E, 0, sizeof(E));
            E.M = n; E.row_count = tc_count; E.row_map = tc_list; E.bias = ly.bias; E.relu = is_last ? 0u : 1u;
            E.status = b->status;
            if (is_last) {
                E.out_f32 = b->logits; E.f32_stride = stride;
            } else {
                E.out_bf16 = A[(l + 1) & 1]; E.ld_bf16 = ly.N;
                if (ly.has_act) { // the lists are written only for a caller that reads them (or their codes)
                    E.out_f32 = (b->active_vals || b->codes) ? vals : nullptr;
                    E.out_ids = b->active_ids ? ids : nullptr;
                    E.indptr = indptr; E.ip_mul = m->n_act; E.ip_add = m->act_index[l];
                }
            }
            rc = slonn_dense_tc_launch(A[l & 1], ly.W, ly.N, ly.D, E, st);
            if (!rc && ly.has_act && b->codes) {
                const uint32_t t = n * m->L;
                dense_codes_kernel<<<(t + 127) / 128, 128, 0, st>>>(tc_list, tc_count, vals, indptr, m->n_act,
                                                                   m->act_index[l], ly.hash_nodes, m->K, m->L, b->codes);
                if (cudaGetLastError() != cudaSuccess) rc = SLONN_ERR_CUDA;
            }
        }
        TOC();
        if (rc) return rc;
        skip_bp = b->budget_bp;
    }

    // narrow networks with enough queries to fill the GPU: one warp per query, every layer in one launch
    // Queries at a 100 % budget all compute the same rows (every node of every layer): they are taken out of the
    // per-query kernels, compacted, and evaluated four per block by full_rows_kernel.  Same fixed-order sums, so
    // nothing about their results changes.
    if (full_route) {
        uint32_t *full_list = (uint32_t *)(ws + wl.tc_list), *full_count = (uint32_t *)(ws + wl.tc_count);
        if (cudaMemsetAsync(full_count, 0, sizeof(uint32_t), st) != cudaSuccess) return SLONN_ERR_CUDA;
        dense_compact_kernel<<<(n + 255) / 256, 256, 0, st>>>(b->budget_bp, n, full_list, full_count);
        if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
        const int rc = run_full_route(m, b, n, full_list, full_count, indptr, ids, vals, dense, stride, st, tm);
        if (rc) return rc;
        skip_bp = b->budget_bp;
    }

    if (use_fused) {
        AT_LAYER(SLONN_ALL_LAYERS);
        uint32_t fused_cols_bp = 0;
        TIC(SLONN_STAGE_FUSED, nullptr, 0u, 0xffffu, skip_bp);
        const int rc = launch_fused(m, b, no_plan ? nullptr : indptr, stride, skip_bp, max_bp, st, &fused_cols_bp);
        if (tm && tm->n > 0) tm->spans[tm->n - 1].cols_bp = fused_cols_bp;
        TOC();
        if (rc || !skip_bp || !b->pred) return rc;
        // predictions of the 100 % queries that another route served (the fused kernel wrote the others and
        // theirs must stay; same rule)
        slonn_argmax_params ap;
        memset(&ap, 0, sizeof(ap));
        ap.logits = b->logits; ap.stride = stride; ap.n = n; ap.pred = b->pred; ap.only_full = skip_bp;
        if (last.has_act) {
            ap.logit_ids = b->logit_ids; ap.indptr = indptr; ap.n_act = m->n_act;
            ap.a = m->act_index[m->n_layers - 1];
        } else {
            ap.fixed_len = last.N;
        }
        TIC(SLONN_STAGE_ARGMAX, b->budget_bp, 10000u, 10000u);
        if (stride >= 2048) argmax_block_kernel<<<n, 256, 0, st>>>(ap);
        else argmax_kernel<<<(n + 7) / 8, 256, 0, st>>>(ap);
        TOC();
        return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
    }

    // input := x
    slonn_input in;
    memset(&in, 0, sizeof(in));
    in.kind = SLONN_IN_DENSE;
    in.dense = b->x_dense;
    int dense_cur = 0;
    uint32_t in_cap = 0; // most entries the current input list holds (list inputs only)
    const group_ws gw = {(uint32_t *)(ws + wl.tc_list), (uint32_t *)(ws + wl.tc_count)};

    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        const bool is_last = (l + 1 == m->n_layers);
        const uint32_t esz = m->dtype == SLONN_BF16 ? 2u : 4u;
        const uint32_t nchunks = ly.D * esz / 16u;
        int rc;
        AT_LAYER(l);
        if (l == 0 && m->first_sparse) {
            float *o = is_last ? b->logits : dense[dense_cur];
            TIC(SLONN_STAGE_SPARSE_FIRST);
            rc = slonn_forward_sparse_first(m, b->x_indptr, b->x_ids, b->x_vals, n, o, is_last ? 0u : 1u,
                                            b->status, st);
            TOC();
            if (rc) return rc;
            in.kind = SLONN_IN_DENSE; in.dense = o;
            dense_cur ^= 1;
            continue;
        }
        slonn_gather_params gp;
        memset(&gp, 0, sizeof(gp));
        gp.in = in; gp.W = ly.W; gp.bias = ly.bias; gp.D = ly.D; gp.N = ly.N; gp.nchunks = nchunks;
        gp.skip_bp = skip_bp;
        gp.n_act = m->n_act; gp.indptr = indptr; gp.ids = ids;
        gp.relu = is_last ? 0u : 1u;
        uint32_t max_rows = ly.N;
        if (ly.has_act) {
            const uint32_t a = m->act_index[l];
            slonn_select_params sp;
            memset(&sp, 0, sizeof(sp));
            sp.in = in; sp.W = ly.W; sp.bias = ly.bias; sp.D = ly.D; sp.N = ly.N; sp.nchunks = nchunks;
            sp.skip_bp = skip_bp;
            sp.hash_nodes = ly.hash_nodes; sp.tables = ly.tables; sp.cap = ly.cap; sp.K = m->K; sp.L = m->L;
            sp.pre = slonn_model_pre(m);
            sp.n_act = m->n_act; sp.a = a; sp.layer = l; sp.indptr = indptr; sp.out_ids = ids;
            sp.codes = b->codes; sp.status = b->status;
            max_rows = slonn_layer_nodes(max_bp, ly.N, slonn_model_pre(m));
            gp.use_list = 1; gp.a = a; gp.out_vals = vals;
            if (is_last) { gp.out_dense = b->logits; gp.out_dense_ids = b->logit_ids; gp.out_stride = stride; }
            rc = launch_act_layer(m, ly, l, sp, gp, b, n, max_bp, max_rows, in_cap, gw, st, tm);
            if (rc) return rc;
            in.kind = SLONN_IN_LIST; in.indptr = indptr; in.ids = ids; in.vals = vals;
            in.ip_mul = m->n_act; in.ip_add = a;
            in_cap = max_rows;
        } else {
            gp.use_list = 0;
            gp.out_dense = is_last ? b->logits : dense[dense_cur];
            gp.out_stride = ly.N;
            // A layer without activator computes every node for every query: the queries the row kernel would
            // serve (budgets above the input-stationary limit) share all their weight rows, so they are
            // compacted and taken four per block.
            bool rows_done = false;
            const uint32_t cols_bp = cols_budget_limit(ly, gp, b, n, max_rows, max_bp);
            if (n >= 256 && (uint64_t)n * ly.N * ly.D >= (1ull << 30) && (size_t)SLONN_FULL_GROUP * ly.D * 4 <= 200 * 1024 &&
                cols_bp < max_bp) {
                uint32_t *glist = (uint32_t *)(ws + wl.tc_list), *gcount = (uint32_t *)(ws + wl.tc_count);
                if (cudaMemsetAsync(gcount, 0, sizeof(uint32_t), st) != cudaSuccess) return SLONN_ERR_CUDA;
                range_compact_kernel<<<(n + 255) / 256, 256, 0, st>>>(b->budget_bp, skip_bp, n, cols_bp ? cols_bp + 1 : 0u, 0xffffu,
                                                                     glist, gcount);
                if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
                slonn_full_params fp;
                memset(&fp, 0, sizeof(fp));
                fp.list = glist; fp.count = gcount; fp.in = in;
                fp.W = ly.W; fp.bias = ly.bias; fp.D = ly.D; fp.N = ly.N; fp.nchunks = nchunks;
                fp.has_act = 0; fp.out_dense = gp.out_dense; fp.out_stride = ly.N; fp.relu = gp.relu;
                TIC(SLONN_STAGE_FULL_ROWS, b->budget_bp, cols_bp ? cols_bp + 1 : 0u, 0xffffu, skip_bp);
                rc = launch_full_rows(m, fp, n, st);
                TOC();
                if (rc) return rc;
                rows_done = true;
            }
            rc = launch_layer_rows(m, ly, gp, b, n, max_bp, max_rows, in_cap, gw, st, tm, rows_done);
            if (rc) return rc;
            in.kind = SLONN_IN_DENSE; in.dense = gp.out_dense;
            dense_cur ^= 1;
        }
    }

    if (b->pred) {
        slonn_argmax_params ap;
        memset(&ap, 0, sizeof(ap));
        ap.logits = b->logits; ap.stride = stride; ap.n = n; ap.pred = b->pred;
        if (last.has_act) {
            ap.logit_ids = b->logit_ids; ap.indptr = indptr; ap.n_act = m->n_act;
            ap.a = m->act_index[m->n_layers - 1];
        } else {
            ap.fixed_len = last.N;
        }
        AT_LAYER(SLONN_ALL_LAYERS);
        TIC(SLONN_STAGE_ARGMAX);
        if (stride >= 2048) argmax_block_kernel<<<n, 256, 0, st>>>(ap);
        else argmax_kernel<<<(n + 7) / 8, 256, 0, st>>>(ap);
        TOC();
        if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
    }
    return SLONN_OK;
}

extern "C" int slonn_run(const slonn_model *m, const slonn_batch *b, void *workspace, uint64_t ws_bytes,
                         void *stream)
{
    return run_impl(m, b, workspace, ws_bytes, stream, nullptr);
}

static int run_with_timer(const slonn_model *m, const slonn_batch *b, void *workspace, uint64_t ws_bytes, void *stream,
                          stage_timer &tm, float *span_ms)
{
    tm.st = (cudaStream_t)stream;
    int rc = run_impl(m, b, workspace, ws_bytes, stream, &tm);
    if (cudaStreamSynchronize(tm.st) != cudaSuccess && rc == SLONN_OK) rc = SLONN_ERR_CUDA;
    for (int i = 0; i < tm.n; ++i) {
        float ms = 0.0f;
        if (rc == SLONN_OK && !tm.failed && cudaEventElapsedTime(&ms, tm.spans[i].a, tm.spans[i].b) != cudaSuccess) rc = SLONN_ERR_CUDA;
        span_ms[i] = ms;
        cudaEventDestroy(tm.spans[i].a);
        cudaEventDestroy(tm.spans[i].b);
    }
    if (tm.failed && rc == SLONN_OK) rc = SLONN_ERR_CUDA;
    return rc;
}

extern "C" int slonn_run_timed(const slonn_model *m, const slonn_batch *b, void *workspace, uint64_t ws_bytes,
                               void *stream, float *stage_ms, uint32_t *stage_launches)
{
    if (!stage_ms || !stage_launches) return SLONN_ERR_ARG;
    stage_timer tm;
    float ms[sizeof(tm.spans) / sizeof(tm.spans[0])];
    const int rc = run_with_timer(m, b, workspace, ws_bytes, stream, tm, ms);
    for (int s = 0; s < SLONN_N_STAGES; ++s) { stage_ms[s] = 0.0f; stage_launches[s] = 0; }
    if (rc == SLONN_OK)
        for (int i = 0; i < tm.n; ++i) {
            stage_ms[tm.spans[i].stage] += ms[i];
            stage_launches[tm.spans[i].stage] += 1;
        }
    return rc;
}

extern "C" int slonn_run_traced(const slonn_model *m, const slonn_batch *b, void *workspace, uint64_t ws_bytes,
                                void *stream, slonn_launch_record *records, uint32_t capacity, uint32_t *n_records)
{
    if (!records || !n_records) return SLONN_ERR_ARG;
    stage_timer tm;
    float ms[sizeof(tm.spans) / sizeof(tm.spans[0])];
    const int rc = run_with_timer(m, b, workspace, ws_bytes, stream, tm, ms);
    *n_records = 0;
    if (rc != SLONN_OK) return rc;
    if ((uint32_t)tm.n > capacity) return SLONN_ERR_ARG;
    for (int i = 0; i < tm.n; ++i) {
        const stage_timer::span &s = tm.spans[i];
        slonn_launch_record &r = records[i];
        r.stage = (uint32_t)s.stage; r.layer = s.layer; r.bp_lo = s.bp_lo; r.bp_hi = s.bp_hi;
        r.skips_full = s.skips_full; r.cols_bp = s.cols_bp; r.ms = ms[i];
    }
    *n_records = (uint32_t)tm.n;
    return SLONN_OK;
}

// ---- run on the library's own fixed scratch area --------------------------------

// Scratch of slonn_run_static.  It lives in the library image, so every GPU that loads the
// library carries these bytes until the process exits.  In host code this name is only a
// stand-in for the symbol, not an address a kernel can use: the device address is looked up
// once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char slonn_static_scratch[SLONN_STATIC_WORKSPACE_BYTES];

namespace {
std::mutex g_static_mu;
void *g_static_ptr[64]; // device address of slonn_static_scratch, per device ordinal
} // namespace

extern "C" int slonn_run_static(const slonn_model *m, const slonn_batch *b, void *stream)
{
    if (!model_ok(m) || !b) return SLONN_ERR_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLONN_ERR_CUDA;
    if (dev != m->device || dev < 0 || dev >= 64) return SLONN_ERR_ARG; // the model's device must be current
    const uint64_t need = carve(m, b->n_queries, eff_max_bp(b->max_budget_bp), b->flags).total;
    if (need > SLONN_STATIC_WORKSPACE_BYTES) return SLONN_ERR_WORKSPACE;
    void *ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        ws = g_static_ptr[dev];
        if (!ws) { // first call on this device: resolve the symbol with this device current
            if (cudaGetSymbolAddress(&ws, slonn_static_scratch) != cudaSuccess || !ws) return SLONN_ERR_CUDA;
            g_static_ptr[dev] = ws;
        }
    }
    return run_impl(m, b, ws, SLONN_STATIC_WORKSPACE_BYTES, stream, nullptr);
}

// ---- budget policy ---------------------------------------------------------------

extern "C" int slonn_lcao_budgets(const uint16_t *profile_bp, const float *profile_ms, uint32_t n_k, const float *t0,
                                  const float *tau, uint32_t n, uint16_t *budget_bp, uint8_t *feasible, void *stream)
{
    if (!profile_bp || !profile_ms || !t0 || !tau || !budget_bp) return SLONN_ERR_ARG;
    if (n_k == 0 || n_k > 4096) return SLONN_ERR_DIM;
    if (n == 0) return SLONN_OK;
    lcao_budget_kernel<<<(n + 255) / 256, 256, n_k * 6 + 8, (cudaStream_t)stream>>>(profile_bp, profile_ms, n_k, t0, tau, n,
                                                                                    budget_bp, feasible);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

// ---- host-buffer variant -----------------------------------------------------

namespace {
struct host_layout {
    uint64_t x, indptr_in, ids_in, vals_in, bp, logits, logit_ids, pred, codes, a_indptr, a_ids, a_vals, status,
        inner, total;
};

host_layout carve_host(const slonn_model *m, uint32_t n, uint32_t max_bp, uint32_t flags, uint64_t x_nnz)
{
    host_layout h;
    memset(&h, 0, sizeof(h));
    uint32_t stride = 0;
    slonn_logit_stride(m, max_bp, &stride);
    const uint64_t ent = active_entries(m, n, max_bp);
    uint64_t o = 0;
    auto take = [&](uint64_t bytes) { uint64_t at = o; o = align_up(o + bytes, 256); return at; };
    if (m->first_sparse) {
        h.indptr_in = take(((uint64_t)n + 1) * 8);
        h.ids_in = take(x_nnz * 4);
        h.vals_in = take(x_nnz * 4);
    } else {
        h.x = take((uint64_t)n * m->dims[0] * 4);
    }
    h.bp = take((uint64_t)n * 2);
    h.logits = take((uint64_t)n * stride * 4);
    h.logit_ids = take((uint64_t)n * stride * 4);
    h.pred = take((uint64_t)n * 4);
    h.codes = take((uint64_t)n * m->n_act * m->L * 2);
    h.a_indptr = take(((uint64_t)n * m->n_act + 1) * 8);
    h.a_ids = take(ent * 4);
    h.a_vals = take(ent * 4);
    h.status = take(16);
    h.inner = o;
    h.total = o + carve(m, n, max_bp, flags).total + 512; // + status words of a batch run in pieces
    return h;
}
} // namespace

extern "C" int slonn_host_workspace_bytes(const slonn_model *m, uint32_t n, uint32_t max_bp, uint32_t flags,
                                          uint64_t x_nnz, uint64_t *bytes)
{
    if (!model_ok(m) || !bytes) return SLONN_ERR_ARG;
    *bytes = carve_host(m, n, eff_max_bp(max_bp), flags, x_nnz).total;
    return SLONN_OK;
}

// Copies in, runs and copies out the queries [q0, q0 + cnt) of a host batch on one stream, using
// `ws` (device) for staging and workspace.  The status words go to status_host (copied back) or,
// when status_dev is given, stay on the device there.
static int run_host_range(const slonn_model *m, const slonn_batch *hb, uint32_t q0, uint32_t cnt, char *ws,
                          uint64_t ws_bytes, cudaStream_t st, uint32_t *status_host, uint32_t *status_dev,
                          uint64_t *up_out, uint64_t *down_out)
{
    const slonn_layer &last = m->layer[m->n_layers - 1];
    const uint32_t max_bp = eff_max_bp(hb->max_budget_bp);
    const uint64_t nnz0 = m->first_sparse ? hb->x_indptr[q0] : 0;
    const uint64_t x_nnz = m->first_sparse ? hb->x_indptr[q0 + cnt] - nnz0 : 0;
    if (m->first_sparse && q0 != 0) return SLONN_ERR_ARG; // CSR rows are only run in one piece
    const host_layout hl = carve_host(m, cnt, max_bp, hb->flags, x_nnz);
    if (ws_bytes < hl.total) return SLONN_ERR_WORKSPACE;
    uint32_t stride = 0;
    slonn_logit_stride(m, max_bp, &stride);
    const uint64_t ent = active_entries(m, cnt, max_bp);
    uint64_t up = 0, down = 0;
#define H2D(dst, src, bytes)                                                                      \
    do {                                                                                          \
        if ((bytes) && cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyHostToDevice, st) != cudaSuccess) \
            return SLONN_ERR_CUDA;                                                                \
        up += (bytes);                                                                            \
    } while (0)
#define D2H(dst, src, bytes)                                                                      \
    do {                                                                                          \
        if ((bytes) && cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToHost, st) != cudaSuccess) \
            return SLONN_ERR_CUDA;                                                                \
        down += (bytes);                                                                          \
    } while (0)

    slonn_batch db = *hb;
    db.n_queries = cnt;
    if (m->first_sparse) {
        H2D(ws + hl.indptr_in, hb->x_indptr, ((uint64_t)cnt + 1) * 8);
        H2D(ws + hl.ids_in, hb->x_ids, x_nnz * 4);
        H2D(ws + hl.vals_in, hb->x_vals, x_nnz * 4);
        db.x_dense = nullptr;
        db.x_indptr = (const uint64_t *)(ws + hl.indptr_in);
        db.x_ids = (const uint32_t *)(ws + hl.ids_in);
        db.x_vals = (const float *)(ws + hl.vals_in);
    } else {
        const uint64_t D0 = m->dims[0];
        H2D(ws + hl.x, hb->x_dense + (uint64_t)q0 * D0, (uint64_t)cnt * D0 * 4);
        db.x_dense = (const float *)(ws + hl.x);
    }
    H2D(ws + hl.bp, hb->budget_bp + q0, (uint64_t)cnt * 2);
    db.budget_bp = (const uint16_t *)(ws + hl.bp);
    db.logits = (float *)(ws + hl.logits);
    db.logit_ids = last.has_act ? (uint32_t *)(ws + hl.logit_ids) : nullptr;
    db.pred = hb->pred ? (uint32_t *)(ws + hl.pred) : nullptr;
    db.codes = hb->codes ? (uint16_t *)(ws + hl.codes) : nullptr;
    db.active_indptr = (uint64_t *)(ws + hl.a_indptr);
    db.active_ids = (uint32_t *)(ws + hl.a_ids);
    db.active_vals = (float *)(ws + hl.a_vals);
    db.status = status_dev ? status_dev : (uint32_t *)(ws + hl.status);

    const int rc = slonn_run(m, &db, ws + hl.inner, ws_bytes - hl.inner, st);
    if (rc) return rc;

    D2H(hb->logits + (uint64_t)q0 * stride, db.logits, (uint64_t)cnt * stride * 4);
    if (last.has_act) D2H(hb->logit_ids + (uint64_t)q0 * stride, db.logit_ids, (uint64_t)cnt * stride * 4);
    if (hb->pred) D2H(hb->pred + q0, db.pred, (uint64_t)cnt * 4);
    if (hb->codes) D2H(hb->codes + (uint64_t)q0 * m->n_act * m->L, db.codes, (uint64_t)cnt * m->n_act * m->L * 2);
    if (hb->active_indptr) D2H(hb->active_indptr, db.active_indptr, ((uint64_t)cnt * m->n_act + 1) * 8);
    if (hb->active_ids) D2H(hb->active_ids, db.active_ids, ent * 4);
    if (hb->active_vals) D2H(hb->active_vals, db.active_vals, ent * 4);
    if (!status_dev) D2H(status_host, db.status, 16);
#undef H2D
#undef D2H
    *up_out += up;
    *down_out += down;
    return SLONN_OK;
}

namespace {
// The two internal streams and three events of a piecewise host call, kept per device between calls.  A call
// that finds its device's set taken (two host calls at once) makes a set of its own and destroys it afterwards.
struct piece_streams {
    cudaStream_t s[2] = {nullptr, nullptr};
    cudaEvent_t start = nullptr, done[2] = {nullptr, nullptr};
    bool create()
    {
        return cudaStreamCreateWithFlags(&s[0], cudaStreamNonBlocking) == cudaSuccess &&
               cudaStreamCreateWithFlags(&s[1], cudaStreamNonBlocking) == cudaSuccess &&
               cudaEventCreateWithFlags(&start, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&done[0], cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&done[1], cudaEventDisableTiming) == cudaSuccess;
    }
    void destroy()
    {
        for (int i = 0; i < 2; ++i) {
            if (s[i]) cudaStreamDestroy(s[i]);
            if (done[i]) cudaEventDestroy(done[i]);
            s[i] = nullptr; done[i] = nullptr;
        }
        if (start) cudaEventDestroy(start);
        start = nullptr;
    }
};
std::mutex g_piece_mu;
piece_streams g_piece_set[64]; // per device ordinal
bool g_piece_made[64], g_piece_taken[64];

// Takes the device's kept set (made on first use) or, when it is taken or the device ordinal is out of range,
// makes a new one; *kept tells which.  false: the CUDA calls failed (whatever was created is destroyed).
bool acquire_piece_streams(int dev, piece_streams *out, bool *kept)
{
    *kept = false;
    if (dev >= 0 && dev < 64) {
        std::lock_guard<std::mutex> lock(g_piece_mu);
        if (!g_piece_taken[dev]) {
            if (!g_piece_made[dev]) {
                if (!g_piece_set[dev].create()) { g_piece_set[dev].destroy(); return false; }
                g_piece_made[dev] = true;
            }
            g_piece_taken[dev] = true;
            *out = g_piece_set[dev];
            *kept = true;
            return true;
        }
    }
    if (!out->create()) { out->destroy(); return false; }
    return true;
}

void release_piece_streams(int dev, piece_streams *ps, bool kept)
{
    if (kept) {
        std::lock_guard<std::mutex> lock(g_piece_mu);
        g_piece_taken[dev] = false;
    } else {
        ps->destroy();
    }
}
} // namespace

extern "C" int slonn_run_host(const slonn_model *m, const slonn_batch *hb, void *workspace, uint64_t ws_bytes,
                              void *stream, uint64_t *h2d_bytes, uint64_t *d2h_bytes)
{
    if (!model_ok(m) || !hb) return SLONN_ERR_ARG;
    if (!hb->budget_bp || !hb->logits || !hb->status) return SLONN_ERR_ARG;
    if (m->first_sparse ? (!hb->x_indptr || !hb->x_ids || !hb->x_vals) : !hb->x_dense) return SLONN_ERR_ARG;
    const slonn_layer &last = m->layer[m->n_layers - 1];
    if (last.has_act && !hb->logit_ids) return SLONN_ERR_ARG;
    const uint32_t n = hb->n_queries;
    const uint32_t max_bp = eff_max_bp(hb->max_budget_bp);
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t x_nnz = m->first_sparse ? hb->x_indptr[n] : 0; // host array: readable here
    const host_layout hl = carve_host(m, n, max_bp, hb->flags, x_nnz);
    if (!workspace || ((uintptr_t)workspace & 255u) || ws_bytes < hl.total) return SLONN_ERR_WORKSPACE;
    char *ws = (char *)workspace;
    uint64_t up = 0, down = 0;

    // Large dense batches go through in pieces on two internal streams, so that the copy of one
    // piece overlaps the kernels of the other.  The per-(query, layer) lists are indexed from the
    // start of the batch, so a caller that wants them back gets the batch in one piece.
    // The first piece's copy overlaps nothing, which argues for small pieces where a query's input is
    // large; kernels on few queries fill the SMs worse, which argues for large ones.  A piece carries
    // about 16 MiB of input, between 1024 and 2048 queries (4096 fp32 inputs per query: four pieces of
    // 1024 queries took 4.5 ms end to end where two of 2048 took 4.9 ms; 1024 inputs per query at
    // mixed budgets: 2048-query pieces 9.6 ms, 1024-query pieces 11.0 ms).
#ifndef SLONN_PIECE_QUERIES
    const uint64_t row_bytes = (uint64_t)m->layer[0].D * sizeof(float);
    const uint32_t piece_min = (uint32_t)std::min<uint64_t>(2048u, std::max<uint64_t>(1024u, (16ull << 20) / std::max<uint64_t>(row_bytes, 1)));
#else
    const uint32_t piece_min = SLONN_PIECE_QUERIES;
#endif
    const uint32_t pieces = std::min(8u, std::max(1u, n / piece_min));
    const bool wants_lists = hb->active_indptr || hb->active_ids || hb->active_vals;
    uint32_t piece = (n + pieces - 1) / pieces;
    piece = (piece + 255u) / 256u * 256u;
    const uint64_t half = ((ws_bytes - 256) / 2) & ~(uint64_t)255; // two piece areas, then the pieces' status words
    bool piecewise = !m->first_sparse && !wants_lists && pieces >= 2 && !(hb->flags & SLONN_FLAG_DENSE_TC);
    if (piecewise && carve_host(m, piece, max_bp, hb->flags, 0).total > half) piecewise = false;

    if (!piecewise) {
        const int rc = run_host_range(m, hb, 0, n, ws, ws_bytes, st, hb->status, nullptr, &up, &down);
        if (rc) return rc;
        if (cudaStreamSynchronize(st) != cudaSuccess) return SLONN_ERR_CUDA;
    } else {
        piece_streams ps;
        bool kept = false;
        if (!acquire_piece_streams(m->device, &ps, &kept)) return SLONN_ERR_CUDA;
        cudaStream_t *s2 = ps.s;
        uint32_t status[9][4]; // at most 8 pieces
        memset(status, 0, sizeof(status));
        int rc = SLONN_OK;
        // the internal streams start after whatever the caller queued on `stream`
        bool ok = cudaEventRecord(ps.start, st) == cudaSuccess && cudaStreamWaitEvent(s2[0], ps.start, 0) == cudaSuccess &&
                  cudaStreamWaitEvent(s2[1], ps.start, 0) == cudaSuccess;
        uint32_t k = 0;
        for (uint32_t q0 = 0; ok && rc == SLONN_OK && q0 < n; q0 += piece, ++k) {
            const uint32_t cnt = std::min(piece, n - q0);
            rc = run_host_range(m, hb, q0, cnt, ws + (k & 1u) * half, half, s2[k & 1u], nullptr,
                                (uint32_t *)(ws + 2 * half) + 4 * k, &up, &down);
        }
        if (ok && rc == SLONN_OK) {
            ok = cudaEventRecord(ps.done[0], s2[0]) == cudaSuccess && cudaEventRecord(ps.done[1], s2[1]) == cudaSuccess &&
                 cudaStreamWaitEvent(st, ps.done[0], 0) == cudaSuccess && cudaStreamWaitEvent(st, ps.done[1], 0) == cudaSuccess &&
                 cudaMemcpyAsync(status, ws + 2 * half, (size_t)k * 16, cudaMemcpyDeviceToHost, st) == cudaSuccess;
            down += (uint64_t)k * 16;
        }
        // nothing below may return before the internal streams are idle and handed back
        const bool synced = cudaStreamSynchronize(s2[0]) == cudaSuccess && cudaStreamSynchronize(s2[1]) == cudaSuccess &&
                            cudaStreamSynchronize(st) == cudaSuccess;
        release_piece_streams(m->device, &ps, kept);
        if (rc) return rc;
        if (!ok || !synced) return SLONN_ERR_CUDA;
        // first error of any piece, query index made batch-relative
        memset(hb->status, 0, 16);
        for (uint32_t i = 0; i < k; ++i)
            if (status[i][0]) {
                hb->status[0] = status[i][0]; hb->status[1] = status[i][1] + i * piece;
                hb->status[2] = status[i][2]; hb->status[3] = status[i][3];
                break;
            }
    }
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return SLONN_OK;
}
