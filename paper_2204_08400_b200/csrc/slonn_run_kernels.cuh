// Kernels of the SLO-aware forward pass (Fig. 2 steps 1, 3, 4 of the paper):
//   plan_*_kernel            budgets -> per (query, activator layer) list offsets
//   hash_select_kernel       FreeHash bits -> keys -> bucket lists -> first B distinct ids
//   gather_dot_kernel        the selected rows' dot products, bias, activation
//   gather_cols_kernel       the same for a sparse (id, value) input: nonzero inputs x selected nodes
//   sparse_first_layer_kernel  layer 0 fed by CSR rows (transposed weights)
//   argmax_kernel            prediction over the computed logits
#pragma once
#include "slonn_common.cuh"
#include "slonn_cols_kernels.cuh"

#define SLONN_THREADS 256
#ifndef SLONN_DEEP_WALK
#define SLONN_DEEP_WALK true // eight list entries per step in the walks whose warps share the segments
#endif

// whether query q's budget lies in [lo, hi] (range_bp == NULL: every query)
__device__ __forceinline__ bool bp_in_range(const uint16_t *range_bp, uint32_t lo, uint32_t hi, uint32_t q)
{
    if (!range_bp) return true;
    const uint32_t bp = range_bp[q];
    return bp >= lo && bp <= hi;
}

#define SLONN_ROWS_PER_WARP 4 // hash rows per warp pass (reduce_rows4)
#ifndef SLONN_SELECT_MIN_BLOCKS
#define SLONN_SELECT_MIN_BLOCKS 4
#endif


// ---------------------------------------------------------------------------
// block-wide exclusive scan of one value per thread (blockDim.x <= 1024)
// ---------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T *warp_sums /* [32] shared */, T *total)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    T incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        T t = __shfl_up_sync(SLONN_FULL_MASK, incl, off);
        if (lane >= (uint32_t)off) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const uint32_t nw = (blockDim.x + 31u) >> 5;
        T w = lane < nw ? warp_sums[lane] : (T)0;
        T wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            T t = __shfl_up_sync(SLONN_FULL_MASK, wi, off);
            if (lane >= (uint32_t)off) wi += t;
        }
        warp_sums[lane] = wi - w; // exclusive warp offsets
        if (lane == 31) *total = wi;
    }
    __syncthreads();
    const T res = warp_sums[warp] + incl - v;
    __syncthreads();
    return res;
}

// ---------------------------------------------------------------------------
// plan: node counts and offsets from the budgets (one block)
// ---------------------------------------------------------------------------
struct slonn_plan_params {
    const uint16_t *budget_bp;
    uint32_t n, n_act, max_bp;
    uint32_t pre; // hash nodes that are always active (0 or K*L)
    uint32_t act_N[SLONN_MAX_LAYERS];
    uint32_t act_cap[SLONN_MAX_LAYERS];
    uint32_t act_layer[SLONN_MAX_LAYERS];
    uint64_t *indptr; // [n * n_act + 1]
    uint32_t *status;
};

__device__ __forceinline__ uint32_t plan_count(const slonn_plan_params &P, uint64_t e, bool check)
{
    const uint32_t q = (uint32_t)(e / P.n_act), a = (uint32_t)(e % P.n_act);
    uint32_t bp = P.budget_bp[q];
    bool bad = (bp < 1u) || (bp > 10000u) || (bp > P.max_bp);
    if (bp < 1u) bp = 1u;
    if (bp > P.max_bp) bp = P.max_bp;
    const uint32_t B = slonn_layer_nodes(bp, P.act_N[a], P.pre);
    if (B - P.pre > P.act_cap[a] && B != P.act_N[a]) bad = true;
    if (bad && check) slonn_report(P.status, SLONN_ERR_BUDGET, q, P.act_layer[a]);
    return B;
}

// Two launches: per-tile sums, then each tile's prefix (tile base = sum of the tiles before it).
#define SLONN_PLAN_THREADS 256
#define SLONN_PLAN_PER_THREAD 8
#define SLONN_PLAN_TILE (SLONN_PLAN_THREADS * SLONN_PLAN_PER_THREAD)

__global__ void __launch_bounds__(SLONN_PLAN_THREADS) plan_partial_kernel(slonn_plan_params P, uint64_t *tile_sums)
{
    __shared__ uint64_t warp_sums[32];
    __shared__ uint64_t total;
    const uint64_t M = (uint64_t)P.n * P.n_act;
    const uint64_t e0 = (uint64_t)blockIdx.x * SLONN_PLAN_TILE + (uint64_t)threadIdx.x * SLONN_PLAN_PER_THREAD;
    uint64_t local = 0;
    for (uint32_t k = 0; k < SLONN_PLAN_PER_THREAD; ++k)
        if (e0 + k < M) local += plan_count(P, e0 + k, true);
    block_exclusive_scan<uint64_t>(local, warp_sums, &total);
    if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(SLONN_PLAN_THREADS) plan_final_kernel(slonn_plan_params P, const uint64_t *tile_sums)
{
    __shared__ uint64_t warp_sums[32];
    __shared__ uint64_t total;
    __shared__ uint64_t base_total;
    const uint64_t M = (uint64_t)P.n * P.n_act;
    // base of this tile: sum of all earlier tiles
    uint64_t part = 0;
    for (uint32_t t = threadIdx.x; t < blockIdx.x; t += blockDim.x) part += tile_sums[t];
    block_exclusive_scan<uint64_t>(part, warp_sums, &base_total);
    const uint64_t base = base_total;
    const uint64_t e0 = (uint64_t)blockIdx.x * SLONN_PLAN_TILE + (uint64_t)threadIdx.x * SLONN_PLAN_PER_THREAD;
    uint32_t cnt[SLONN_PLAN_PER_THREAD];
    uint64_t local = 0;
#pragma unroll
    for (uint32_t k = 0; k < SLONN_PLAN_PER_THREAD; ++k) {
        cnt[k] = (e0 + k < M) ? plan_count(P, e0 + k, false) : 0u;
        local += cnt[k];
    }
    uint64_t run = base + block_exclusive_scan<uint64_t>(local, warp_sums, &total);
#pragma unroll
    for (uint32_t k = 0; k < SLONN_PLAN_PER_THREAD; ++k) {
        if (e0 + k < M) P.indptr[e0 + k] = run;
        run += cnt[k];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) P.indptr[M] = base + total;
}

// ---------------------------------------------------------------------------
// hash + select: one block per query
// ---------------------------------------------------------------------------
struct slonn_select_params {
    const uint16_t *skip_bp;    // nullable: queries with this budget == 10000 are handled elsewhere
    const uint16_t *range_bp;   // nullable: only queries whose budget lies in [bp_lo, bp_hi]
    uint32_t bp_lo, bp_hi;
    slonn_input in;
    const void *W;
    const float *bias;
    uint32_t D, N, nchunks;
    const uint32_t *hash_nodes; // device [L*K]
    const void *tables;         // [L][2^K][cap]
    uint32_t cap, K, L;
    uint32_t pre;               // hash nodes that are always active (0 or K*L)
    uint32_t n_act, a, layer;
    const uint64_t *indptr;     // offsets of (q, a)
    uint32_t *out_ids;          // CSR payload
    uint16_t *codes;            // nullable [n][n_act][L]
    uint32_t *status;
};

template <typename IDT>
__device__ __forceinline__ uint32_t table_entry(const void *tables, uint32_t cap, uint32_t K,
                                                uint32_t b, uint32_t key, uint32_t r)
{
    const IDT *t = reinterpret_cast<const IDT *>(tables);
    return (uint32_t)__ldg(t + (((uint64_t)b << K) + key) * cap + r);
}

// The layer's active set, written ascending to out[0..B) (global or shared memory): the first
// B - pre distinct ids of the rank-interleaved bucket lists, and the first `pre` entries of
// hash_nodes (pre = 0, or K*L for models whose hash nodes are always active and never listed).
// Called by every thread of the block; bitmap ((N+31)/32 words) must be zero and keys[L] set, all
// behind a barrier.  B == N gives every node.  Returns false when the lists did not hold enough
// distinct ids (malformed tables); out is then 0..B-1.
template <typename IDT>
__device__ __forceinline__ bool block_select(const void *tables, uint32_t cap, uint32_t K, uint32_t L, uint32_t N,
                                             uint32_t B, const uint32_t *keys, uint32_t *bitmap, uint32_t *out,
                                             uint32_t *scan_ws, uint32_t *scan_total, const uint32_t *hash_nodes,
                                             uint32_t pre)
{
    const uint32_t nwords = (N + 31u) >> 5;
    if (B == N) { // every node
        for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) out[i] = i;
        return true;
    }
    const uint32_t want = B - pre; // ids to take from the lists
    if (want > cap) { // reported by the plan; keep the output in range
        for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) out[i] = i;
        return true;
    }
    if (pre) {
        for (uint32_t h = threadIdx.x; h < pre; h += blockDim.x) {
            const uint32_t nd = __ldg(hash_nodes + h);
            atomicOr(&bitmap[nd >> 5], 1u << (nd & 31u));
        }
        __syncthreads();
    }

    // (3)+(4) read the L lists rank by rank; the first B distinct ids are the active set.
    // Position pos = rank * L + table.  Positions are taken strictly in order, in steps that
    // never hold more positions than ids still missing (want - total): a step can then add at most
    // that many new ids, so the count never passes `want`, and when it reaches it the marked ids are
    // exactly the distinct ids of a prefix of the position sequence -- the first `want` distinct ones.
    // (Which of two equal ids inside a step wins the atomic does not matter: one does.)
    // Each thread fetches its entries of the next SEL_ROWS rows of blockDim.x positions in one go; while
    // more ids are missing than the whole window holds, the window is one step (one block-wide sum of
    // the new ids), afterwards the steps follow the rows and shrink with the ids still missing.
    constexpr int SEL_ROWS = 8;
    const uint32_t npos = want * L; // `want` distinct ids are always found within rank < want
    const uint32_t T = blockDim.x;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = (T + 31u) >> 5;
    uint32_t total = 0;
    // When the block size is a multiple of L a thread always reads the same table: its list and the
    // rank stride between its positions are fixed, and no division is left in the loop.
    const bool fixed_table = (T % L) == 0u;
    const uint32_t my_b = threadIdx.x % L, my_r = threadIdx.x / L, r_step = T / L;
    const IDT *my_list = reinterpret_cast<const IDT *>(tables) + (((uint64_t)my_b << K) + keys[my_b]) * cap;
    for (uint32_t w0 = 0; w0 < npos && total < want; w0 += SEL_ROWS * T) {
        uint32_t ahead[SEL_ROWS];
        if (fixed_table) {
            const uint32_t r0 = w0 / L + my_r;
#pragma unroll
            for (int u = 0; u < SEL_ROWS; ++u) {
                const uint32_t p = w0 + u * T + threadIdx.x;
                ahead[u] = p < npos ? (uint32_t)__ldg(my_list + r0 + u * r_step) : 0xffffffffu;
            }
        } else {
#pragma unroll
            for (int u = 0; u < SEL_ROWS; ++u) {
                const uint32_t p = w0 + u * T + threadIdx.x;
                ahead[u] = 0xffffffffu;
                if (p < npos) {
                    const uint32_t r = p / L, b = p - r * L;
                    ahead[u] = table_entry<IDT>(tables, cap, K, b, keys[b], r);
                }
            }
        }
        const uint32_t window = min((uint32_t)SEL_ROWS * T, npos - w0);
        if (want - total >= window) { // uniform: the whole window cannot overshoot
            uint32_t wins = 0;
#pragma unroll
            for (int u = 0; u < SEL_ROWS; ++u)
                if (ahead[u] < N) {
                    const uint32_t bit = 1u << (ahead[u] & 31u);
                    wins += ((atomicOr(&bitmap[ahead[u] >> 5], bit) & bit) == 0u) ? 1u : 0u;
                }
            wins = __reduce_add_sync(SLONN_FULL_MASK, wins);
            if (lane == 0) scan_ws[warp] = wins;
            __syncthreads();
            total += __reduce_add_sync(SLONN_FULL_MASK, lane < nwarps ? scan_ws[lane] : 0u);
            __syncthreads(); // scan_ws is reused by the next window and by the emit below
            continue;
        }
#pragma unroll
        for (int u = 0; u < SEL_ROWS; ++u) {
            const uint32_t row0 = w0 + u * T;              // this row holds positions row0 .. row0 + T - 1
            const uint32_t row1 = min(row0 + T, npos);
            const uint32_t mine = row0 + threadIdx.x;
            uint32_t p = row0;
            while (p < row1 && total < want) {             // uniform for the block
                const uint32_t s = min(want - total, row1 - p);
                bool won = false;
                if (mine >= p && mine < p + s && ahead[u] < N) {
                    const uint32_t bit = 1u << (ahead[u] & 31u);
                    won = (atomicOr(&bitmap[ahead[u] >> 5], bit) & bit) == 0u;
                }
                total += (uint32_t)__syncthreads_count(won);
                p += s;
            }
        }
    }
    __syncthreads();
    if (total != want) { // cannot happen with well-formed tables; keep the output in range
        for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) out[i] = i;
        return false;
    }

    // emit ascending ids: popcount prefix over the bitmap words
    const uint32_t wpt = (nwords + blockDim.x - 1) / blockDim.x;
    const uint32_t w0 = threadIdx.x * wpt;
    const uint32_t w1 = min(w0 + wpt, nwords);
    uint32_t cnt = 0;
    for (uint32_t w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
    uint32_t o = block_exclusive_scan<uint32_t>(cnt, scan_ws, scan_total);
    for (uint32_t w = w0; w < w1; ++w) {
        uint32_t bits = bitmap[w];
        while (bits) {
            const uint32_t t = __ffs(bits) - 1;
            bits &= bits - 1;
            out[o++] = (w << 5) + t;
        }
    }
    return true;
}

// LAT: latency variant for a handful of queries -- up to 32 warps per block, one hash row per warp
// with deep load prefetch, instead of 4 rows per warp pass.
template <bool BF16, typename IDT, bool LAT>
__global__ void __launch_bounds__(LAT ? 1024 : SLONN_THREADS, LAT ? 1 : SLONN_SELECT_MIN_BLOCKS) hash_select_kernel(slonn_select_params P)
{
    extern __shared__ float4 smem4[];
    float4 *xs4 = smem4;
    uint32_t *bitmap = reinterpret_cast<uint32_t *>(smem4 + (P.D >> 2));
    __shared__ float zh[128];
    __shared__ uint32_t keys[8];
    __shared__ uint32_t scan_ws[32];
    __shared__ uint32_t scan_total;

    const uint32_t q = blockIdx.x;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    if (!bp_in_range(P.range_bp, P.bp_lo, P.bp_hi, q)) return;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t H = P.K * P.L;
    const uint64_t off = P.indptr[(uint64_t)q * P.n_act + P.a];
    const uint32_t B = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - off);
    const uint32_t nwords = (P.N + 31u) >> 5;

    // (1) FreeHash: z_h = w_h . x + b_h for the layer's K*L hash nodes
    stage_input<BF16>(P.in, q, P.D, P.nchunks, xs4);
    const uint32_t row_u4 = P.nchunks; // uint4 per weight row
    if (LAT) {
        for (uint32_t h = warp; h < H; h += nwarps) {
            const uint32_t nd = __ldg(P.hash_nodes + h);
            const float sum = warp_dot_row1<BF16>(reinterpret_cast<const uint4 *>(P.W) + (uint64_t)nd * row_u4, xs4,
                                                  P.nchunks, lane);
            if (lane == 0) zh[h] = sum + __ldg(P.bias + nd);
        }
    } else
    for (uint32_t h0 = warp * SLONN_ROWS_PER_WARP; h0 < H; h0 += nwarps * SLONN_ROWS_PER_WARP) {
        const uint4 *rows[SLONN_ROWS_PER_WARP];
#pragma unroll
        for (int r = 0; r < SLONN_ROWS_PER_WARP; ++r) {
            const uint32_t nd = __ldg(P.hash_nodes + min(h0 + r, H - 1));
            rows[r] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)nd * row_u4;
        }
        float acc[SLONN_ROWS_PER_WARP];
        warp_dot_rows<BF16, SLONN_ROWS_PER_WARP>(rows, xs4, P.nchunks, lane, acc);
        const float sum = reduce_rows4(acc, lane); // row h0 + (lane >> 3)
        const uint32_t h = h0 + (lane >> 3);
        if ((lane & 7u) == 0u && h < H) zh[h] = sum + __ldg(P.bias + __ldg(P.hash_nodes + h));
    }
    for (uint32_t i = threadIdx.x; i < nwords; i += blockDim.x) bitmap[i] = 0u;
    __syncthreads();

    // (2) keys: bit j of key_b = [z of hash function j of table b > 0]
    if (threadIdx.x < P.L) {
        uint32_t key = 0;
        for (uint32_t j = 0; j < P.K; ++j)
            if (zh[threadIdx.x * P.K + j] > 0.0f) key |= (1u << j);
        keys[threadIdx.x] = key;
        if (P.codes) P.codes[((uint64_t)q * P.n_act + P.a) * P.L + threadIdx.x] = (uint16_t)key;
    }
    __syncthreads();

    if (!block_select<IDT>(P.tables, P.cap, P.K, P.L, P.N, B, keys, bitmap, P.out_ids + off, scan_ws, &scan_total,
                           P.hash_nodes, P.pre) &&
        threadIdx.x == 0)
        slonn_report(P.status, SLONN_ERR_ARG, q, P.layer);
}

// ---------------------------------------------------------------------------
// gather-dot: the selected rows of one layer
// ---------------------------------------------------------------------------
struct slonn_gather_params {
    const uint16_t *skip_bp;  // nullable: queries with this budget == 10000 are handled elsewhere
    slonn_input in;
    const void *W;
    const float *bias;
    uint32_t D, N, nchunks;
    uint32_t use_list;        // 1: rows = active ids of (q, a); 0: every row
    uint32_t n_act, a;
    const uint64_t *indptr;
    const uint32_t *ids;      // CSR payload (use_list)
    float *out_vals;          // CSR payload (use_list), nullable
    float *out_dense;         // [n][N] (!use_list), or strided copy [n][out_stride] (use_list), nullable
    uint32_t *out_dense_ids;  // [n][out_stride] ids beside the strided copy, nullable
    uint32_t out_stride;
    uint32_t relu;
    uint32_t rows_per_cta, ctas_per_query;
    // queries served by this launch: budget in [bp_lo, bp_hi] (range_bp nullable = all)
    const uint16_t *range_bp;
    uint32_t bp_lo, bp_hi;
    // gather_cols_kernel only
    const void *WT;           // transposed copy [D][N], node axis in colpos order
    const uint32_t *colpos;   // [N] node id -> column of WT; NULL = identity
    uint32_t in_cap;          // most entries an input list of this launch can hold
    uint32_t rows_cap;        // most nodes a query of this launch selects
    uint32_t scratch_bytes;   // shared memory in front of the entries (input image, then node order)
};


// R: rows per warp pass, 4 (6-shuffle reduction) or 8 (9 shuffles; pays off for rows of one
// 512-byte round, where the reduction is most of the work).
template <bool BF16, bool LAT, int R>
#ifdef SLONN_GATHER_MIN_BLOCKS
__launch_bounds__(SLONN_THREADS, SLONN_GATHER_MIN_BLOCKS)
#else
__launch_bounds__(SLONN_THREADS)
#endif
__global__ void gather_dot_kernel(slonn_gather_params P)
{
    extern __shared__ float4 smem4[];
    const uint32_t q = blockIdx.x / P.ctas_per_query;
    const uint32_t chunk = blockIdx.x - q * P.ctas_per_query;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    if (!bp_in_range(P.range_bp, P.bp_lo, P.bp_hi, q)) return;
    uint64_t off = 0;
    uint32_t B = P.N;
    if (P.use_list) {
        off = P.indptr[(uint64_t)q * P.n_act + P.a];
        B = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - off);
    }
    const uint32_t r0 = chunk * P.rows_per_cta;
    if (r0 >= B) return;
    const uint32_t r1 = min(B, r0 + P.rows_per_cta);

    stage_input<BF16>(P.in, q, P.D, P.nchunks, smem4);

    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (LAT) { // one row per warp, deep load prefetch
        for (uint32_t r = r0 + warp; r < r1; r += nwarps) {
            const uint32_t nd = P.use_list ? __ldg(P.ids + off + r) : r;
            const float sum = warp_dot_row1<BF16>(reinterpret_cast<const uint4 *>(P.W) + (uint64_t)nd * P.nchunks, smem4,
                                                  P.nchunks, lane);
            if (lane == 0) {
                float z = sum + __ldg(P.bias + nd);
                if (P.relu) z = z > 0.0f ? z : 0.0f;
                if (P.use_list) {
                    if (P.out_vals) P.out_vals[off + r] = z;
                    if (P.out_dense) {
                        P.out_dense[(uint64_t)q * P.out_stride + r] = z;
                        if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q * P.out_stride + r] = nd;
                    }
                } else {
                    P.out_dense[(uint64_t)q * P.out_stride + nd] = z;
                }
            }
        }
    } else
    for (uint32_t r = r0 + warp * R; r < r1; r += nwarps * R) {
        const uint4 *rows[R];
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const uint32_t rr = min(r + k, r1 - 1);
            const uint32_t nd = P.use_list ? __ldg(P.ids + off + rr) : rr;
            rows[k] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)nd * P.nchunks;
        }
        float acc[R];
        warp_dot_rows<BF16, R>(rows, smem4, P.nchunks, lane, acc);
        float sum;
        uint32_t mr;
        bool writer;
        if constexpr (R == 8) {
            sum = reduce_rows8(acc, lane); // row r + (lane >> 2)
            mr = r + (lane >> 2);
            writer = (lane & 3u) == 0u;
        } else {
            sum = reduce_rows4(acc, lane); // row r + (lane >> 3)
            mr = r + (lane >> 3);
            writer = (lane & 7u) == 0u;
        }
        if (writer && mr < r1) {
            const uint32_t nd = P.use_list ? __ldg(P.ids + off + mr) : mr;
            float z = sum + __ldg(P.bias + nd);
            if (P.relu) z = z > 0.0f ? z : 0.0f;
            if (P.use_list) {
                if (P.out_vals) P.out_vals[off + mr] = z;
                if (P.out_dense) {
                    P.out_dense[(uint64_t)q * P.out_stride + mr] = z;
                    if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q * P.out_stride + mr] = nd;
                }
            } else {
                P.out_dense[(uint64_t)q * P.out_stride + nd] = z;
            }
        }
    }
}

// Queries at a 100 % budget compute every node of every layer (Sec. 3.4: the full network), so all of them
// want the same weight rows.  This kernel takes such queries four at a time: a block stages the four
// inputs, and every 16-byte weight chunk a lane loads is multiplied into four queries' partial sums --
// a quarter of the weight loads and of the widening work per multiply-add.  Each (query, row) sum is still
// formed in the library's fixed order, so the results are those of gather_dot_kernel bit for bit.
// `list` / `count`: the batch's 100 % queries (dense_compact_kernel); group g = entries 4g .. 4g + 3.
struct slonn_full_params {
    const uint32_t *list;
    const uint32_t *count;
    slonn_input in;
    const void *W;
    const float *bias;
    uint32_t D, N, nchunks;
    uint32_t has_act;         // 1: results go to the (query, a) list (every node, ascending); 0: dense rows
    uint32_t n_act, a;
    const uint64_t *indptr;
    uint32_t *out_ids;        // CSR payload (has_act)
    float *out_vals;          // CSR payload (has_act)
    float *out_dense;         // [n][out_stride]: hidden layer without activator, or the logits; nullable
    uint32_t *out_dense_ids;  // logit ids of a budgeted last layer; nullable
    uint32_t out_stride;
    uint32_t relu;
    uint32_t rows_per_cta, ctas_per_group;
};

#define SLONN_FULL_GROUP 4
#ifndef SLONN_FULL_MIN_BLOCKS
#define SLONN_FULL_MIN_BLOCKS 2 // with 8 rows per pass (123 registers); 4 rows: 3 blocks at 80 registers beat 2 at 115
#endif

#ifndef SLONN_FULL_R
#define SLONN_FULL_R 8 // rows per warp pass (4 or 8); measured on 2048-4096-4096-1000 at 100 %: 15.2 ms with 4, 14.7 with 8
#endif
template <bool BF16, int R>
__global__ void __launch_bounds__(SLONN_THREADS, SLONN_FULL_MIN_BLOCKS) full_rows_kernel(slonn_full_params P)
{
    extern __shared__ float4 smem4[];
    constexpr int VPC = BF16 ? 8 : 4;
    constexpr int G = SLONN_FULL_GROUP;
    const uint32_t g = blockIdx.x / P.ctas_per_group;
    const uint32_t chunk = blockIdx.x - g * P.ctas_per_group;
    const uint32_t cnt = *P.count;
    if (g * G >= cnt) return;
    const uint32_t r0 = chunk * P.rows_per_cta;
    if (r0 >= P.N) return;
    const uint32_t r1 = min(P.N, r0 + P.rows_per_cta);
    const uint32_t nq = min((uint32_t)G, cnt - g * G);
    const uint32_t per_q = (BF16 ? 2u : 1u) * P.nchunks; // float4 per staged input

    uint32_t q[G];
    uint64_t off[G];
#pragma unroll
    for (int k = 0; k < G; ++k) {
        q[k] = __ldg(P.list + g * G + min((uint32_t)k, nq - 1)); // a short last group repeats its last query
        off[k] = P.has_act ? P.indptr[(uint64_t)q[k] * P.n_act + P.a] : 0;
        stage_input<BF16>(P.in, q[k], P.D, P.nchunks, smem4 + k * per_q);
    }

    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (uint32_t r = r0 + warp * R; r < r1; r += nwarps * R) {
        const uint4 *rows[R];
#pragma unroll
        for (int k = 0; k < R; ++k)
            rows[k] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)min(r + k, r1 - 1) * P.nchunks;
        float acc[G][R];
#pragma unroll
        for (int k = 0; k < G; ++k)
#pragma unroll
            for (int j = 0; j < R; ++j) acc[k][j] = 0.0f;
        for (uint32_t c = lane; c < P.nchunks; c += 32) {
            uint4 w[R];
#pragma unroll
            for (int j = 0; j < R; ++j) w[j] = __ldg(rows[j] + c);
#pragma unroll
            for (int k = 0; k < G; ++k) {
                const float4 *xs4 = smem4 + k * per_q;
                float x[VPC];
                const float4 xa = xs4[c];
                x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w;
                if (BF16) {
                    const float4 xb = xs4[P.nchunks + c];
                    x[VPC - 4] = xb.x; x[VPC - 3] = xb.y; x[VPC - 2] = xb.z; x[VPC - 1] = xb.w;
                }
                chunk_fma<BF16, R, 0, VPC>::run(w, x, acc[k]);
            }
        }
        const uint32_t mr = r + (R == 8 ? (lane >> 2) : (lane >> 3));
        const bool writer = R == 8 ? (lane & 3u) == 0u : (lane & 7u) == 0u;
        const float b = __ldg(P.bias + min(mr, P.N - 1u));
#pragma unroll
        for (int k = 0; k < G; ++k) {
            float sum;
            if constexpr (R == 8) sum = reduce_rows8(acc[k], lane); // row r + (lane >> 2)
            else sum = reduce_rows4(acc[k], lane);                  // row r + (lane >> 3)
            if (writer && mr < r1 && (uint32_t)k < nq) {
                float z = sum + b;
                if (P.relu) z = z > 0.0f ? z : 0.0f;
                if (P.has_act) {
                    P.out_vals[off[k] + mr] = z;
                    P.out_ids[off[k] + mr] = mr;
                    if (P.out_dense) {
                        P.out_dense[(uint64_t)q[k] * P.out_stride + mr] = z;
                        if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q[k] * P.out_stride + mr] = mr;
                    }
                } else {
                    P.out_dense[(uint64_t)q[k] * P.out_stride + mr] = z;
                }
            }
        }
    }
}

// Selected rows of a layer for queries taken FOUR AT A TIME (the batch formulation the paper leaves open in
// Sec. 7): the importance rankings of all buckets start with much the same nodes, so the active sets of any four
// queries overlap heavily.  A block stages four inputs, marks each query's active set in a bitmap and splits the
// union of the four sets in two:
//   rows that at least three of the four queries selected -- evaluated once for all four, every 16-byte weight
//     chunk a lane loads feeding four queries' partial sums (the result of a query that did not select the row is
//     dropped);
//   the other rows -- evaluated for the queries that selected them, one query at a time.
// Each (query, row) sum is formed in the library's fixed order either way, so the values are those of
// gather_dot_kernel bit for bit; they are written to the row's place in the query's id-ascending list, which is
// the popcount of the query's bitmap below the row.
// `list` / `count`: the queries this launch serves (range_compact_kernel); group g = entries 4g .. 4g + 3.
struct slonn_group_params {
    slonn_gather_params G;    // in, W, bias, D, N, nchunks, n_act, a, indptr, ids, out_vals, out_dense(_ids), out_stride, relu
    const uint32_t *list;
    const uint32_t *count;
    uint32_t ctas_per_group;  // blocks that share a group's rows
    uint32_t rows_cap;        // most rows a query of this launch selects
    uint32_t shared_cap;      // entries of the shared-row list: min(N, 4 * rows_cap / 3 + 1)
};

#define SLONN_GROUP 4
#ifndef SLONN_GROUP_MIN_BLOCKS
#define SLONN_GROUP_MIN_BLOCKS 2
#endif

template <bool BF16>
__global__ void __launch_bounds__(SLONN_THREADS, SLONN_GROUP_MIN_BLOCKS) group_rows_kernel(slonn_group_params Q)
{
    extern __shared__ float4 smem4[];
    constexpr int VPC = BF16 ? 8 : 4;
    constexpr int G = SLONN_GROUP, R = 4;
    const slonn_gather_params &P = Q.G;
    __shared__ uint64_t scan_ws[32];
    __shared__ uint64_t scan_total;
    const uint32_t g = blockIdx.x / Q.ctas_per_group;
    const uint32_t chunk = blockIdx.x - g * Q.ctas_per_group;
    const uint32_t cnt = *Q.count;
    if (g * G >= cnt) return;
    const uint32_t nq = min((uint32_t)G, cnt - g * G);
    const uint32_t per_q = (BF16 ? 2u : 1u) * P.nchunks; // float4 per staged input
    const uint32_t nwords = (P.N + 31u) >> 5;

    // shared memory: four staged inputs | four bitmaps | shared-row bitmap | four position prefixes |
    // shared-row list | four lists of a query's other rows
    uint32_t *bm = reinterpret_cast<uint32_t *>(smem4 + G * per_q);
    uint32_t *shbits = bm + G * nwords;
    uint32_t *pre = shbits + nwords;
    uint16_t *shlist = reinterpret_cast<uint16_t *>(pre + G * nwords);
    uint16_t *rem = shlist + ((Q.shared_cap + 7u) & ~7u);
    const uint32_t rem_stride = (Q.rows_cap + 7u) & ~7u;

    uint32_t q[G], B[G];
    uint64_t off[G];
#pragma unroll
    for (int k = 0; k < G; ++k) {
        q[k] = __ldg(Q.list + g * G + min((uint32_t)k, nq - 1)); // a short last group repeats its last query
        off[k] = P.indptr[(uint64_t)q[k] * P.n_act + P.a];
        B[k] = min((uint32_t)(P.indptr[(uint64_t)q[k] * P.n_act + P.a + 1] - off[k]), Q.rows_cap);
        stage_input<BF16>(P.in, q[k], P.D, P.nchunks, smem4 + k * per_q);
    }
    for (uint32_t i = threadIdx.x; i < G * nwords; i += blockDim.x) bm[i] = 0u;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < G; ++k)
        if ((uint32_t)k < nq)
            for (uint32_t i = threadIdx.x; i < B[k]; i += blockDim.x) {
                const uint32_t id = min(__ldg(P.ids + off[k] + i), P.N - 1u);
                atomicOr(&bm[k * nwords + (id >> 5)], 1u << (id & 31u));
            }
    __syncthreads();

    // per bitmap word: the rows at least three queries want, each query's other rows; counts -> offsets
    const uint32_t wpt = (nwords + blockDim.x - 1) / blockDim.x;
    const uint32_t w0 = threadIdx.x * wpt, w1 = min(w0 + wpt, nwords);
    uint64_t c_all = 0, c_rem = 0; // four 16-bit counts each (N <= 65535)
    uint32_t c_sh = 0;
    for (uint32_t w = w0; w < w1; ++w) {
        const uint32_t b0 = bm[w], b1 = bm[nwords + w], b2 = bm[2 * nwords + w], b3 = bm[3 * nwords + w];
        const uint32_t s = (b0 & b1 & (b2 | b3)) | (b2 & b3 & (b0 | b1));
        shbits[w] = s;
        c_sh += __popc(s);
        c_all += (uint64_t)__popc(b0) | ((uint64_t)__popc(b1) << 16) | ((uint64_t)__popc(b2) << 32) | ((uint64_t)__popc(b3) << 48);
        c_rem += (uint64_t)__popc(b0 & ~s) | ((uint64_t)__popc(b1 & ~s) << 16) | ((uint64_t)__popc(b2 & ~s) << 32) |
                 ((uint64_t)__popc(b3 & ~s) << 48);
    }
    uint64_t o_all = block_exclusive_scan<uint64_t>(c_all, scan_ws, &scan_total);
    uint64_t o_rem = block_exclusive_scan<uint64_t>(c_rem, scan_ws, &scan_total);
    const uint64_t rem_total = scan_total;
    uint64_t o_sh = block_exclusive_scan<uint64_t>((uint64_t)c_sh, scan_ws, &scan_total);
    const uint32_t n_sh = (uint32_t)scan_total;
    for (uint32_t w = w0; w < w1; ++w) {
        const uint32_t s = shbits[w];
        uint32_t bits = s;
        while (bits) {
            const uint32_t t = __ffs(bits) - 1;
            bits &= bits - 1;
            if (o_sh < Q.shared_cap) shlist[o_sh] = (uint16_t)((w << 5) + t);
            ++o_sh;
        }
#pragma unroll
        for (int k = 0; k < G; ++k) {
            const uint32_t b = bm[k * nwords + w];
            pre[k * nwords + w] = (uint32_t)(o_all >> (16 * k)) & 0xffffu;
            uint32_t o = (uint32_t)(o_rem >> (16 * k)) & 0xffffu;
            bits = b & ~s;
            while (bits) {
                const uint32_t t = __ffs(bits) - 1;
                bits &= bits - 1;
                if (o < Q.rows_cap) rem[k * rem_stride + o] = (uint16_t)((w << 5) + t);
                ++o;
            }
            o_all += (uint64_t)__popc(b) << (16 * k);
            o_rem += (uint64_t)__popc(b & ~s) << (16 * k);
        }
    }
    __syncthreads();

    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    auto emit = [&](int k, uint32_t n, float sum) { // row n of query k, if the query selected it
        const uint32_t word = bm[k * nwords + (n >> 5)], bit = 1u << (n & 31u);
        if (!(word & bit)) return;
        const uint32_t pos = pre[k * nwords + (n >> 5)] + __popc(word & (bit - 1u));
        float z = sum + __ldg(P.bias + n);
        if (P.relu) z = z > 0.0f ? z : 0.0f;
        if (P.out_vals) P.out_vals[off[k] + pos] = z;
        if (P.out_dense) {
            P.out_dense[(uint64_t)q[k] * P.out_stride + pos] = z;
            if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q[k] * P.out_stride + pos] = n;
        }
    };

    // (A) the rows at least three of the four queries selected: one weight load feeds four sums
    {
        const uint32_t per = (n_sh + Q.ctas_per_group - 1) / Q.ctas_per_group;
        const uint32_t a0 = min(chunk * per, n_sh), a1 = min(a0 + per, n_sh);
        for (uint32_t r = a0 + warp * R; r < a1; r += nwarps * R) {
            const uint4 *rows[R];
#pragma unroll
            for (int j = 0; j < R; ++j)
                rows[j] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)shlist[min(r + j, a1 - 1)] * P.nchunks;
            float acc[G][R];
#pragma unroll
            for (int k = 0; k < G; ++k)
#pragma unroll
                for (int j = 0; j < R; ++j) acc[k][j] = 0.0f;
            for (uint32_t c = lane; c < P.nchunks; c += 32) {
                uint4 w[R];
#pragma unroll
                for (int j = 0; j < R; ++j) w[j] = __ldg(rows[j] + c);
#pragma unroll
                for (int k = 0; k < G; ++k) {
                    const float4 *xs4 = smem4 + k * per_q;
                    float x[VPC];
                    const float4 xa = xs4[c];
                    x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w;
                    if (BF16) {
                        const float4 xb = xs4[P.nchunks + c];
                        x[VPC - 4] = xb.x; x[VPC - 3] = xb.y; x[VPC - 2] = xb.z; x[VPC - 1] = xb.w;
                    }
                    chunk_fma<BF16, R, 0, VPC>::run(w, x, acc[k]);
                }
            }
            const uint32_t mr = r + (lane >> 3);
            const uint32_t n = shlist[min(mr, a1 - 1)];
#pragma unroll
            for (int k = 0; k < G; ++k) {
                const float sum = reduce_rows4(acc[k], lane); // row r + (lane >> 3)
                if ((lane & 7u) == 0u && mr < a1 && (uint32_t)k < nq) emit(k, n, sum);
            }
        }
    }
    // (B) every query's other rows, one query at a time
#pragma unroll
    for (int k = 0; k < G; ++k) {
        if ((uint32_t)k >= nq) break;
        const uint32_t n_rem = min((uint32_t)(rem_total >> (16 * k)) & 0xffffu, Q.rows_cap);
        const uint32_t per = (n_rem + Q.ctas_per_group - 1) / Q.ctas_per_group;
        const uint32_t a0 = min(chunk * per, n_rem), a1 = min(a0 + per, n_rem);
        const uint16_t *mine = rem + k * rem_stride;
        const float4 *xs4 = smem4 + k * per_q;
        for (uint32_t r = a0 + warp * R; r < a1; r += nwarps * R) {
            const uint4 *rows[R];
#pragma unroll
            for (int j = 0; j < R; ++j)
                rows[j] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)mine[min(r + j, a1 - 1)] * P.nchunks;
            float acc[R];
            warp_dot_rows<BF16, R>(rows, xs4, P.nchunks, lane, acc);
            const float sum = reduce_rows4(acc, lane); // row r + (lane >> 3)
            const uint32_t mr = r + (lane >> 3);
            if ((lane & 7u) == 0u && mr < a1) emit(k, mine[mr], sum);
        }
    }
}

// Rows of at most one 512-byte round (one 16-byte chunk per lane): the lane's piece of the input is
// loaded once and kept in registers, a warp fetches 32 row ids with one coalesced load and works
// through them 8 rows at a time, so that the only loads inside the loop are the weight chunks
// themselves.  Same chunk-to-lane assignment, element order and reduction as gather_dot_kernel<.., 8>.
template <bool BF16>
__global__ void __launch_bounds__(SLONN_THREADS, 2) gather_short_kernel(slonn_gather_params P)
{
    extern __shared__ float4 smem4[];
    constexpr int VPC = BF16 ? 8 : 4;
    constexpr int R = 8;
    const uint32_t q = blockIdx.x / P.ctas_per_query;
    const uint32_t chunk = blockIdx.x - q * P.ctas_per_query;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    if (!bp_in_range(P.range_bp, P.bp_lo, P.bp_hi, q)) return;
    uint64_t off = 0;
    uint32_t B = P.N;
    if (P.use_list) {
        off = P.indptr[(uint64_t)q * P.n_act + P.a];
        B = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - off);
    }
    const uint32_t r0 = chunk * P.rows_per_cta;
    if (r0 >= B) return;
    const uint32_t r1 = min(B, r0 + P.rows_per_cta);

    stage_input<BF16>(P.in, q, P.D, P.nchunks, smem4);

    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const bool has_chunk = lane < P.nchunks;
    float x[VPC];
#pragma unroll
    for (int e = 0; e < VPC; ++e) x[e] = 0.0f;
    if (has_chunk) {
        const float4 xa = smem4[lane];
        x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w;
        if (BF16) {
            const float4 xb = smem4[P.nchunks + lane];
            x[VPC - 4] = xb.x; x[VPC - 3] = xb.y; x[VPC - 2] = xb.z; x[VPC - 1] = xb.w;
        }
    }
    const uint4 *Wl = reinterpret_cast<const uint4 *>(P.W) + lane;
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    for (uint32_t base = r0 + warp * 32u; base < r1; base += nwarps * 32u) {
        const uint32_t mine = min(base + lane, r1 - 1);
        const uint32_t myid = P.use_list ? __ldg(P.ids + off + mine) : mine;
#pragma unroll
        for (uint32_t sub = 0; sub < 4; ++sub) {
            const uint32_t r = base + sub * R;
            if (r >= r1) break; // uniform
            uint4 w[R];
#pragma unroll
            for (int k = 0; k < R; ++k) {
                const uint32_t nd = __shfl_sync(SLONN_FULL_MASK, myid, sub * R + k); // rows past r1 repeat the last id
                w[k] = has_chunk ? __ldg(Wl + (uint64_t)nd * P.nchunks) : zero4;
            }
            float acc[R];
#pragma unroll
            for (int k = 0; k < R; ++k) acc[k] = 0.0f;
            chunk_fma<BF16, R, 0, VPC>::run(w, x, acc);
            const float sum = reduce_rows8(acc, lane); // row r + (lane >> 2)
            const uint32_t mr = r + (lane >> 2);
            const uint32_t nd = __shfl_sync(SLONN_FULL_MASK, myid, sub * R + (lane >> 2));
            if ((lane & 3u) == 0u && mr < r1) {
                float z = sum + __ldg(P.bias + nd);
                if (P.relu) z = z > 0.0f ? z : 0.0f;
                if (P.use_list) {
                    if (P.out_vals) P.out_vals[off + mr] = z;
                    if (P.out_dense) {
                        P.out_dense[(uint64_t)q * P.out_stride + mr] = z;
                        if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q * P.out_stride + mr] = nd;
                    }
                } else {
                    P.out_dense[(uint64_t)q * P.out_stride + nd] = z;
                }
            }
        }
    }
}

// Second half of the input-stationary layer, shared by gather_cols_kernel and layer_cols_kernel: puts the
// query's selected nodes in column order and evaluates nodes [r0, r1) of that order against the staged
// input list S.  `order_mem` is block scratch of P.scratch_bytes (the staging image, dead by now).  NC: the
// id list was written by an earlier launch and may be read through the read-only path.
// VEC: compiled with the path for a layer that computes every node and whose width is a multiple of the
// 16 / element size nodes one load holds: a lane takes that many neighbouring columns.
template <bool BF16, int R, bool NC, bool SPLIT = false, bool VEC = false>
__device__ __forceinline__ void cols_order_and_gather(const slonn_gather_params &P, const cols_stage &S, void *order_mem,
                                                      const uint32_t *idlist, float *zpart, uint32_t q, uint64_t off,
                                                      uint32_t B, uint32_t r0, uint32_t r1, uint32_t *scan_ws,
                                                      uint32_t *scan_total_p)
{
    // idlist: the query's id-ascending node list (global or shared memory; unused when every node is computed)
    auto list_id = [&](uint32_t e) -> uint32_t {
        const uint32_t v = NC ? __ldg(idlist + e) : idlist[e];
        return min(v, P.N - 1u);
    };
    // the query's nodes in column order: spos[slot] = column, sidx[slot] = place in the id-ascending list
    const bool ordered = P.use_list && P.colpos;
    uint32_t *bitmap = reinterpret_cast<uint32_t *>(order_mem);
    const uint32_t nwords = (P.N + 31u) >> 5;
    uint32_t *wprefix = bitmap + nwords;
    uint32_t *tmp = wprefix + nwords, *spos = tmp + P.rows_cap, *sidx = spos + P.rows_cap;
    if (ordered) {
        for (uint32_t w = threadIdx.x; w < nwords; w += blockDim.x) bitmap[w] = 0u;
        for (uint32_t e = threadIdx.x; e < B; e += blockDim.x) { spos[e] = 0u; sidx[e] = 0u; }
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < B; e += blockDim.x) {
            const uint32_t pos = min(__ldg(P.colpos + list_id(e)), P.N - 1u);
            tmp[e] = pos;
            atomicOr(&bitmap[pos >> 5], 1u << (pos & 31u));
        }
        __syncthreads();
        const uint32_t wpt = (nwords + blockDim.x - 1) / blockDim.x;
        const uint32_t w0 = threadIdx.x * wpt, w1 = min(w0 + wpt, nwords);
        uint32_t cnt = 0;
        for (uint32_t w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
        uint32_t o = block_exclusive_scan<uint32_t>(cnt, scan_ws, scan_total_p);
        for (uint32_t w = w0; w < w1; ++w) { wprefix[w] = o; o += __popc(bitmap[w]); }
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < B; e += blockDim.x) {
            const uint32_t pos = tmp[e];
            const uint32_t slot = wprefix[pos >> 5] + __popc(bitmap[pos >> 5] & ((1u << (pos & 31u)) - 1u));
            if (slot < B) { spos[slot] = pos; sidx[slot] = e; }
        }
        __syncthreads();
    }

    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if constexpr (SPLIT) {
        // Few queries: the block owns the 32 * R nodes [r0, r1) and its warps share the 32 segments, so that a
        // node's walk over the input list is 32 / nwarps segments long instead of 32; the partial sums meet in
        // shared memory and one thread per node adds them in the fixed tree.
        // zpart: [32][R][32] floats of block scratch
        uint32_t e[R], nd[R], col[R];
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const uint32_t rr = min(r0 + k * 32u + lane, r1 - 1);
            e[k] = rr; nd[k] = rr; col[k] = rr;
            if (ordered) { e[k] = sidx[rr]; col[k] = spos[rr]; }
            if (P.use_list) {
                nd[k] = list_id(e[k]);
                if (!ordered) col[k] = nd[k];
            }
        }
        constexpr uint32_t ESZ = BF16 ? 2u : 4u;
        uint32_t cb[R];
#pragma unroll
        for (int k = 0; k < R; ++k) cb[k] = col[k] * ESZ;
        for (uint32_t p = warp; p < 32; p += nwarps) {
            float a[R];
#pragma unroll
            for (int k = 0; k < R; ++k) a[k] = 0.0f;
            cols_segment<BF16, R, SLONN_DEEP_WALK>(S.ent, S.segstart[p], S.segstart[p + 1], P.WT, P.N * ESZ, cb, a);
#pragma unroll
            for (int k = 0; k < R; ++k) zpart[(p * R + k) * 32u + lane] = a[k];
        }
        __syncthreads();
        if (warp < (uint32_t)R) { // warp k finishes the nodes r0 + 32 k + lane
            uint32_t me = e[0], mnd = nd[0];
#pragma unroll
            for (int k = 1; k < R; ++k)
                if (warp == (uint32_t)k) { me = e[k]; mnd = nd[k]; }
            float acc[32];
#pragma unroll
            for (int p = 0; p < 32; ++p) acc[p] = zpart[(p * R + warp) * 32u + lane];
            float z = cols_tree(acc) + __ldg(P.bias + mnd);
            if (P.relu) z = z > 0.0f ? z : 0.0f;
            if (r0 + warp * 32u + lane < r1) {
                if (P.use_list) {
                    if (P.out_vals) P.out_vals[off + me] = z;
                    if (P.out_dense) {
                        P.out_dense[(uint64_t)q * P.out_stride + me] = z;
                        if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q * P.out_stride + me] = mnd;
                    }
                } else {
                    P.out_dense[(uint64_t)q * P.out_stride + mnd] = z;
                }
            }
        }
    } else if (VEC && !P.use_list && (P.N % (BF16 ? 8u : 4u)) == 0u && (r0 % (BF16 ? 8u : 4u)) == 0u) {
        // every node of the layer, its width a multiple of the nodes a 16-byte load holds: a lane takes that many
        // neighbouring columns and fetches their weights of an input with one load (r1 is such a multiple too)
        constexpr int NV = BF16 ? 8 : 4;
        for (uint32_t r = r0 + warp * (32u * NV); r < r1; r += nwarps * (32u * NV)) {
            const uint32_t c0 = min(r + NV * lane, r1 - NV);
            uint32_t col[NV];
#pragma unroll
            for (int k = 0; k < NV; ++k) col[k] = c0 + k;
            float sum[NV];
            cols_walk<BF16, NV, COLS_LOAD_VEC>(S, P.WT, P.N, col, sum);
            if (r + NV * lane < r1) {
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    float z = sum[k] + __ldg(P.bias + col[k]);
                    if (P.relu) z = z > 0.0f ? z : 0.0f;
                    P.out_dense[(uint64_t)q * P.out_stride + col[k]] = z;
                }
            }
        }
    } else if (R == 2 && !P.use_list && (P.N & 1u) == 0u && (r0 & 1u) == 0u) {
        // every node of the layer (a layer without activator): a lane takes two neighbouring columns and
        // fetches both weights of an input with one load
        for (uint32_t r = r0 + warp * 64u; r < r1; r += nwarps * 64u) {
            const uint32_t c0 = min(r + 2u * lane, (r1 - 1u) & ~1u); // even; c0 + 1 < N because N is even
            const uint32_t col[R] = {c0, c0 + 1u};
            float sum[R];
            cols_walk<BF16, R, COLS_LOAD_PAIR>(S, P.WT, P.N, col, sum);
            if (r + 2u * lane < r1) {
#pragma unroll
                for (int k = 0; k < R; ++k) {
                    if (col[k] < r1) {
                        float z = sum[k] + __ldg(P.bias + col[k]);
                        if (P.relu) z = z > 0.0f ? z : 0.0f;
                        P.out_dense[(uint64_t)q * P.out_stride + col[k]] = z;
                    }
                }
            }
        }
    } else
    for (uint32_t r = r0 + warp * (32u * R); r < r1; r += nwarps * (32u * R)) {
        uint32_t e[R], nd[R], col[R]; // place in the list, node id, column of WT
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const uint32_t rr = min(r + k * 32u + lane, r1 - 1);
            e[k] = rr; nd[k] = rr; col[k] = rr;
            if (ordered) { e[k] = sidx[rr]; col[k] = spos[rr]; }
            if (P.use_list) {
                nd[k] = list_id(e[k]);
                if (!ordered) col[k] = nd[k];
            }
        }
        float sum[R];
        cols_walk<BF16, R>(S, P.WT, P.N, col, sum);
#pragma unroll
        for (int k = 0; k < R; ++k) {
            float z = sum[k] + __ldg(P.bias + nd[k]);
            if (P.relu) z = z > 0.0f ? z : 0.0f;
            if (r + k * 32u + lane < r1) {
                if (P.use_list) {
                    if (P.out_vals) P.out_vals[off + e[k]] = z;
                    if (P.out_dense) {
                        P.out_dense[(uint64_t)q * P.out_stride + e[k]] = z;
                        if (P.out_dense_ids) P.out_dense_ids[(uint64_t)q * P.out_stride + e[k]] = nd[k];
                    }
                } else {
                    P.out_dense[(uint64_t)q * P.out_stride + nd[k]] = z;
                }
            }
        }
    }
}

// Input-stationary variant for a layer whose input is query q's (id, value) list: lane = one
// selected node (32 nodes per warp pass), loop over the query's nonzero inputs grouped by partial
// sum, one weight WT[j][column of n] per lane and input.  The query's selected nodes are first put in
// column order (a bitmap over the columns, popcount prefix: the position of each node among the
// query's columns), so that the 32 lanes of a pass read neighbouring columns.  Same sums, same
// order, same results as gather_dot_kernel; results are written at the node's place in the
// id-ascending list.
// SPLIT: the variant for batches of tens of queries -- one block per (query, 32 * R nodes), the segments
// of the input list spread over the block's warps (see cols_order_and_gather).
template <bool BF16, int R, bool SPLIT, bool VEC = false>
#ifdef SLONN_GATHER_COLS_MIN_BLOCKS
__launch_bounds__(SLONN_THREADS, SLONN_GATHER_COLS_MIN_BLOCKS)
#else
__launch_bounds__(SLONN_THREADS)
#endif
__global__ void gather_cols_kernel(slonn_gather_params P)
{
    extern __shared__ float4 smem4[];
    constexpr int V = BF16 ? 8 : 4;
    __shared__ uint32_t segcnt[32];
    __shared__ uint32_t segstart[33];
    __shared__ uint32_t scan_ws[32];
    __shared__ uint32_t scan_total;
    const uint32_t q = blockIdx.x / P.ctas_per_query;
    const uint32_t chunk = blockIdx.x - q * P.ctas_per_query;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    if (!bp_in_range(P.range_bp, P.bp_lo, P.bp_hi, q)) return;
    uint64_t off = 0;
    uint32_t B = P.N;
    if (P.use_list) {
        off = P.indptr[(uint64_t)q * P.n_act + P.a];
        B = min((uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - off), P.rows_cap);
    }
    const uint32_t r0 = chunk * P.rows_per_cta;
    if (r0 >= B) return;
    const uint32_t r1 = min(B, r0 + P.rows_per_cta);

    // shared memory: [scratch: input image while staging, node order afterwards][entries]
    cols_stage S;
    S.xs = reinterpret_cast<float *>(smem4);
    S.ent = reinterpret_cast<uint2 *>(reinterpret_cast<char *>(smem4) + P.scratch_bytes);
    S.segcnt = segcnt;
    S.segstart = segstart;
    const uint64_t s0 = P.in.indptr[(uint64_t)q * P.in.ip_mul + P.in.ip_add];
    const uint32_t len = min((uint32_t)(P.in.indptr[(uint64_t)q * P.in.ip_mul + P.in.ip_add + 1] - s0), P.in_cap);
    cols_stage_list<V>(S, P.in.ids, P.in.vals, s0, len, P.D);

    cols_order_and_gather<BF16, R, true, SPLIT, VEC>(P, S, smem4, P.ids + off, reinterpret_cast<float *>(S.ent + cols_ent_cap(P.D, P.in_cap)),
                                                 q, off, B, r0, r1, scan_ws, &scan_total);
}

// A whole list-fed activator layer for one query per block, input-stationary: the input list is grouped
// once and serves the FreeHash projection (lane = hash function, over the side-by-side hash rows WH, the 32
// segments spread over the warps and their partial sums added by one thread per function in the fixed tree),
// then keys, bucket lists and the top-k% cut exactly as in hash_select_kernel, then the selected nodes as in
// gather_cols_kernel.  One launch and one staging instead of two of each.
struct slonn_layer_cols_params {
    slonn_gather_params G;      // use_list = 1; in, WT, colpos, bias, D, N, indptr, ids (= out of the selection), outputs, filters
    const void *WH;             // [D][32]
    const uint32_t *hash_nodes; // [L*K], L*K <= 32
    const void *tables;
    uint32_t cap, K, L, pre, layer;
    uint16_t *codes;            // nullable
    uint32_t *status;
};

// SPLIT: the variant for batches of tens of queries -- one block per (query, 64 nodes).  Every block of a
// query groups the input list, computes the hash functions and runs the selection itself (the same result
// in each; only the first block writes keys and list to global memory), then evaluates its 64 nodes with
// the segments of the input list spread over its warps.
// TIGHT: compiled for 40 registers, so that seven blocks of up to seven warps fit an SM (measured on a 4096-wide
// layer with 4096 queries: +3 % at a 10 % budget, where a block has seven warps; with eight warps per block, at
// 25 %, the tighter allocation costs 9-15 %, so those launches take the other instantiation).
template <bool BF16, typename IDT, bool SPLIT, bool TIGHT>
__launch_bounds__(SLONN_THREADS, (SPLIT || TIGHT) ? 6 : 5) // 40 or 48 registers
__global__ void layer_cols_kernel(slonn_layer_cols_params Q)
{
    extern __shared__ float4 smem4[];
    constexpr int V = BF16 ? 8 : 4;
    constexpr int R = 2;
    const slonn_gather_params &P = Q.G;
    __shared__ uint32_t segcnt[32];
    __shared__ uint32_t segstart[33];
    __shared__ uint32_t scan_ws[32];
    __shared__ uint32_t scan_total;
    __shared__ uint32_t keys[8];
    __shared__ float zh[32];
    const uint32_t q = SPLIT ? blockIdx.x / P.ctas_per_query : blockIdx.x;
    const uint32_t chunk = SPLIT ? blockIdx.x - q * P.ctas_per_query : 0u;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    if (!bp_in_range(P.range_bp, P.bp_lo, P.bp_hi, q)) return;
    const uint64_t off = P.indptr[(uint64_t)q * P.n_act + P.a];
    const uint32_t B = min((uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - off), P.rows_cap);
    const uint32_t r0 = SPLIT ? chunk * P.rows_per_cta : 0u;
    if (r0 >= B) return;
    const uint32_t r1 = SPLIT ? min(B, r0 + P.rows_per_cta) : B;
    const bool writer = chunk == 0u; // the block that publishes the query's keys and list
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t H = Q.K * Q.L;
    const uint32_t nwords = (P.N + 31u) >> 5;

    // shared memory: [scratch: input image, then the hash functions' partial sums, then node order][entries]
    // [selection bitmap][SPLIT: partial sums of hash functions and nodes, the query's node list]
    cols_stage S;
    S.xs = reinterpret_cast<float *>(smem4);
    S.ent = reinterpret_cast<uint2 *>(reinterpret_cast<char *>(smem4) + P.scratch_bytes);
    S.segcnt = segcnt;
    S.segstart = segstart;
    uint32_t *idmap = reinterpret_cast<uint32_t *>(S.ent + cols_ent_cap(P.D, P.in_cap));
    // [32][R][32] of its own when the node loop needs it too (SPLIT); else [32][32] at the start of the scratch,
    // which is free between the staging and the node order
    float *zpart = SPLIT ? reinterpret_cast<float *>(idmap + nwords) : reinterpret_cast<float *>(smem4);
    uint32_t *own_list = reinterpret_cast<uint32_t *>(zpart + 32 * R * 32); // [rows_cap], SPLIT only
    const uint64_t s0 = P.in.indptr[(uint64_t)q * P.in.ip_mul + P.in.ip_add];
    const uint32_t len = min((uint32_t)(P.in.indptr[(uint64_t)q * P.in.ip_mul + P.in.ip_add + 1] - s0), P.in_cap);
    cols_stage_list<V>(S, P.in.ids, P.in.vals, s0, len, P.D);

    // (1) FreeHash: partial sum p of hash function `lane`, segments spread over the warps
    {
        constexpr uint32_t ESZ = BF16 ? 2u : 4u;
        const uint32_t cb[1] = {lane * ESZ};
        for (uint32_t p = warp; p < 32; p += nwarps) {
            float a[1] = {0.0f};
            cols_segment<BF16, 1, SLONN_DEEP_WALK>(S.ent, segstart[p], segstart[p + 1], Q.WH, 32u * ESZ, cb, a);
            zpart[p * 32u + lane] = a[0];
        }
    }
    for (uint32_t i = threadIdx.x; i < nwords; i += blockDim.x) idmap[i] = 0u;
    __syncthreads();
    if (threadIdx.x < H) {
        float acc[32];
#pragma unroll
        for (int p = 0; p < 32; ++p) acc[p] = zpart[p * 32 + threadIdx.x];
        zh[threadIdx.x] = cols_tree(acc) + __ldg(P.bias + __ldg(Q.hash_nodes + threadIdx.x));
    }
    __syncthreads();
    // (2) keys
    if (threadIdx.x < Q.L) {
        uint32_t key = 0;
        for (uint32_t j = 0; j < Q.K; ++j)
            if (zh[threadIdx.x * Q.K + j] > 0.0f) key |= (1u << j);
        keys[threadIdx.x] = key;
        if (Q.codes && writer) Q.codes[((uint64_t)q * P.n_act + P.a) * Q.L + threadIdx.x] = (uint16_t)key;
    }
    __syncthreads();
    // (3) + (4) bucket lists, first B distinct ids, ascending: into the layer's list, or, when several blocks
    // work on the query, into this block's own copy, which the first block then publishes
    uint32_t *global_list = const_cast<uint32_t *>(P.ids) + off;
    uint32_t *list = SPLIT ? own_list : global_list;
    if (!block_select<IDT>(Q.tables, Q.cap, Q.K, Q.L, P.N, B, keys, idmap, list, scan_ws, &scan_total, Q.hash_nodes, Q.pre) &&
        threadIdx.x == 0 && writer)
        slonn_report(Q.status, SLONN_ERR_ARG, q, Q.layer);
    __syncthreads();
    if (SPLIT && writer)
        for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) global_list[i] = own_list[i];
    // (5) the selected nodes
    cols_order_and_gather<BF16, R, false, SPLIT>(P, S, smem4, list, zpart, q, off, B, r0, r1, scan_ws, &scan_total);
}

// ---------------------------------------------------------------------------
// layer 0 fed by CSR rows (sparse operand): thread n owns output node n and walks
// the row's nonzeros in id order; nonzero number j goes to partial sum j mod 32.
// WT is the transposed weight copy [D][N], so each nonzero reads one contiguous row.
// ---------------------------------------------------------------------------
struct slonn_sparse_params {
    const uint64_t *x_indptr;
    const uint32_t *x_ids;
    const float *x_vals;
    const void *WT;
    const float *bias;
    uint32_t D, N;
    float *out_dense; // [n][out_stride]
    uint32_t out_stride;
    uint32_t relu;
    uint32_t blocks_per_query; // ceil(N / 128)
    uint32_t *status;
};

template <bool BF16>
__global__ void __launch_bounds__(128) sparse_first_layer_kernel(slonn_sparse_params P)
{
    __shared__ uint32_t s_ids[128];
    __shared__ float s_vals[128];
    const uint32_t q = blockIdx.x / P.blocks_per_query;
    const uint32_t n = (blockIdx.x - q * P.blocks_per_query) * blockDim.x + threadIdx.x;
    const uint64_t s0 = P.x_indptr[q];
    const uint32_t nnz = (uint32_t)(P.x_indptr[q + 1] - s0);
    float acc[32];
#pragma unroll
    for (int p = 0; p < 32; ++p) acc[p] = 0.0f;
    for (uint32_t base = 0; base < nnz; base += 128) {
        __syncthreads();
        if (base + threadIdx.x < nnz) {
            uint32_t id = P.x_ids[s0 + base + threadIdx.x];
            float v = P.x_vals[s0 + base + threadIdx.x];
            if (id >= P.D) { slonn_report(P.status, SLONN_ERR_ARG, q, 0); id = 0; v = 0.0f; }
            s_ids[threadIdx.x] = id;
            s_vals[threadIdx.x] = v;
        }
        __syncthreads();
        if (n < P.N) {
            const uint32_t m = min(128u, nnz - base);
            for (uint32_t jb = 0; jb < m; jb += 32) {
                // 32 loads in flight (entries past the end re-read the last one and are not used)
                float w[32];
#pragma unroll
                for (uint32_t p = 0; p < 32; ++p) {
                    const uint64_t idx = (uint64_t)s_ids[min(jb + p, m - 1)] * P.N + n;
                    if (BF16) w[p] = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(P.WT) + idx) << 16);
                    else w[p] = __ldg(reinterpret_cast<const float *>(P.WT) + idx);
                }
#pragma unroll
                for (uint32_t p = 0; p < 32; ++p)
                    if (jb + p < m) acc[p] = fmaf(w[p], s_vals[jb + p], acc[p]);
            }
        }
    }
    if (n >= P.N) return;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
        for (int p = 0; p < off; ++p) acc[p] = acc[p] + acc[p + off];
    }
    float z = acc[0] + __ldg(P.bias + n);
    if (P.relu) z = z > 0.0f ? z : 0.0f;
    P.out_dense[(uint64_t)q * P.out_stride + n] = z;
}

// ---------------------------------------------------------------------------
// argmax over each query's computed logits (one warp per query)
// ---------------------------------------------------------------------------
struct slonn_argmax_params {
    const float *logits;       // [n][stride]
    const uint32_t *logit_ids; // nullable: position -> node id
    uint32_t stride, n;
    uint32_t fixed_len;        // used when indptr == NULL
    const uint64_t *indptr;    // budgeted last layer: length of (q, a)
    uint32_t n_act, a;
    uint32_t *pred;
    const uint16_t *only_full; // nullable: only queries whose budget is 10000 bp (the others were served elsewhere)
};

__global__ void __launch_bounds__(256) argmax_kernel(slonn_argmax_params P)
{
    const uint32_t q = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t lane = threadIdx.x & 31u;
    if (q >= P.n) return;
    if (P.only_full && P.only_full[q] != 10000u) return;
    uint32_t len = P.fixed_len;
    if (P.indptr)
        len = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - P.indptr[(uint64_t)q * P.n_act + P.a]);
    const float *lg = P.logits + (uint64_t)q * P.stride;
    float best = 0.0f;
    uint32_t bi = 0xffffffffu;
    for (uint32_t i = lane; i < len; i += 32) {
        const float v = lg[i];
        if (bi == 0xffffffffu || v > best) { best = v; bi = i; }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const float ob = __shfl_xor_sync(SLONN_FULL_MASK, best, off);
        const uint32_t oi = __shfl_xor_sync(SLONN_FULL_MASK, bi, off);
        if (oi != 0xffffffffu && (bi == 0xffffffffu || ob > best || (ob == best && oi < bi))) {
            best = ob;
            bi = oi;
        }
    }
    if (lane == 0 && bi != 0xffffffffu)
        P.pred[q] = P.logit_ids ? P.logit_ids[(uint64_t)q * P.stride + bi] : bi;
}


// The same with one block per query, for logit rows of thousands of entries.
__global__ void __launch_bounds__(256) argmax_block_kernel(slonn_argmax_params P)
{
    __shared__ float wbest[8];
    __shared__ uint32_t wbi[8];
    const uint32_t q = blockIdx.x;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    if (P.only_full && P.only_full[q] != 10000u) return; // uniform for the block
    uint32_t len = P.fixed_len;
    if (P.indptr)
        len = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + P.a + 1] - P.indptr[(uint64_t)q * P.n_act + P.a]);
    const float *lg = P.logits + (uint64_t)q * P.stride;
    float best = 0.0f;
    uint32_t bi = 0xffffffffu;
    for (uint32_t i0 = threadIdx.x; i0 < len; i0 += 8 * blockDim.x) {
        float v[8]; // eight loads in flight per thread
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = i0 + u * blockDim.x;
            v[u] = i < len ? lg[i] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = i0 + u * blockDim.x;
            if (i < len && (bi == 0xffffffffu || v[u] > best)) { best = v[u]; bi = i; }
        }
    }
    for (int round = 0; round < 2; ++round) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const float ob = __shfl_xor_sync(SLONN_FULL_MASK, best, off);
            const uint32_t oi = __shfl_xor_sync(SLONN_FULL_MASK, bi, off);
            if (oi != 0xffffffffu && (bi == 0xffffffffu || ob > best || (ob == best && oi < bi))) { best = ob; bi = oi; }
        }
        if (round == 1) break;
        if (lane == 0) { wbest[warp] = best; wbi[warp] = bi; }
        __syncthreads();
        best = lane < (blockDim.x >> 5) ? wbest[lane] : 0.0f;
        bi = lane < (blockDim.x >> 5) ? wbi[lane] : 0xffffffffu;
    }
    if (threadIdx.x == 0 && bi != 0xffffffffu)
        P.pred[q] = P.logit_ids ? P.logit_ids[(uint64_t)q * P.stride + bi] : bi;
}

// ---------------------------------------------------------------------------
// tensor-core route for 100 % budgets: which queries, their inputs as bf16 rows, their codes
// ---------------------------------------------------------------------------
// list[0 .. *count) = the queries whose budget lies in [lo, hi] and is not skipped (any order)
__global__ void range_compact_kernel(const uint16_t *bp, const uint16_t *skip_bp, uint32_t n, uint32_t lo, uint32_t hi,
                                     uint32_t *list, uint32_t *count)
{
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t lane = threadIdx.x & 31u;
    bool take = false;
    if (q < n) {
        const uint32_t v = bp[q];
        take = v >= lo && v <= hi && !(skip_bp && v == 10000u);
    }
    const uint32_t mask = __ballot_sync(SLONN_FULL_MASK, take);
    if (mask == 0u) return;
    uint32_t base = 0;
    if (lane == (uint32_t)(__ffs(mask) - 1)) base = atomicAdd(count, (uint32_t)__popc(mask));
    base = __shfl_sync(SLONN_FULL_MASK, base, __ffs(mask) - 1);
    if (take) list[base + __popc(mask & ((1u << lane) - 1u))] = q;
}

__global__ void dense_compact_kernel(const uint16_t *bp, uint32_t n, uint32_t *list, uint32_t *count)
{
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t lane = threadIdx.x & 31u;
    const bool full = q < n && bp[q] == 10000u;
    const uint32_t mask = __ballot_sync(SLONN_FULL_MASK, full);
    if (mask == 0u) return;
    uint32_t base = 0;
    if (lane == (uint32_t)(__ffs(mask) - 1)) base = atomicAdd(count, (uint32_t)__popc(mask));
    base = __shfl_sync(SLONN_FULL_MASK, base, __ffs(mask) - 1);
    if (full) list[base + __popc(mask & ((1u << lane) - 1u))] = q;
}

__device__ __forceinline__ uint32_t pack_bf16x2_rne(float a, float b)
{
    uint32_t ua = __float_as_uint(a), ub = __float_as_uint(b);
    ua = (ua & 0x7fffffffu) > 0x7f800000u ? (ua >> 16) | 0x40u : (ua + 0x7fffu + ((ua >> 16) & 1u)) >> 16;
    ub = (ub & 0x7fffffffu) > 0x7f800000u ? (ub >> 16) | 0x40u : (ub + 0x7fffu + ((ub >> 16) & 1u)) >> 16;
    return (ua & 0xffffu) | (ub << 16);
}

// A[m][:] = bf16(x[list[m]][:]) for m < *count; D a multiple of 4
__global__ void dense_gather_x_kernel(const float *x, uint32_t D, const uint32_t *list, const uint32_t *count,
                                      uint16_t *A)
{
    const uint32_t m = blockIdx.x;
    if (m >= *count) return;
    const float4 *src = reinterpret_cast<const float4 *>(x + (uint64_t)list[m] * D);
    uint2 *dst = reinterpret_cast<uint2 *>(A + (uint64_t)m * D);
    for (uint32_t i = threadIdx.x; i < (D >> 2); i += blockDim.x) {
        const float4 v = __ldg(src + i);
        dst[i] = make_uint2(pack_bf16x2_rne(v.x, v.y), pack_bf16x2_rne(v.z, v.w));
    }
}

// codes of the tensor-core queries: bit j of key_b = [activation of hash node (b, j) > 0]
// (hidden layers are ReLU, so the activation is positive exactly when the pre-activation is)
__global__ void dense_codes_kernel(const uint32_t *list, const uint32_t *count, const float *vals,
                                   const uint64_t *indptr, uint32_t n_act, uint32_t a, const uint32_t *hash_nodes,
                                   uint32_t K, uint32_t L, uint16_t *codes)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t m = t / L, b = t - m * L;
    if (m >= *count) return;
    const uint32_t q = list[m];
    const float *v = vals + indptr[(uint64_t)q * n_act + a]; // all nodes are active: position = node id
    uint32_t key = 0;
    for (uint32_t j = 0; j < K; ++j)
        if (v[hash_nodes[b * K + j]] > 0.0f) key |= (1u << j);
    codes[((uint64_t)q * n_act + a) * L + b] = (uint16_t)key;
}


// ---------------------------------------------------------------------------
// LCAO (Eq. 3 of the paper): per query the largest profiled k with t0 + T(k) <= tau
// ---------------------------------------------------------------------------
__global__ void lcao_budget_kernel(const uint16_t *profile_bp, const float *profile_ms, uint32_t n_k, const float *t0,
                                   const float *tau, uint32_t n, uint16_t *budget_bp, uint8_t *feasible)
{
    extern __shared__ float s_prof[]; // n_k latencies, then n_k budgets (as uint16)
    uint16_t *s_bp = reinterpret_cast<uint16_t *>(s_prof + n_k);
    for (uint32_t i = threadIdx.x; i < n_k; i += blockDim.x) { s_prof[i] = profile_ms[i]; s_bp[i] = profile_bp[i]; }
    __syncthreads();
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= n) return;
    const float base = t0[q], limit = tau[q];
    bool found = false;
    uint32_t best = 0, smallest = 0xffffu;
    for (uint32_t i = 0; i < n_k; ++i) {
        const uint32_t bp = s_bp[i];
        smallest = min(smallest, bp);
        if (__fadd_rn(base, s_prof[i]) <= limit && (!found || bp > best)) { best = bp; found = true; }
    }
    budget_bp[q] = (uint16_t)(found ? best : smallest);
    if (feasible) feasible[q] = found ? 1 : 0;
}
