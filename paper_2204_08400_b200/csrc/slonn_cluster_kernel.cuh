// Latency path for a handful of queries (the paper's setting: batch size 1, Sec. 4): one
// thread-block CLUSTER carries one query through every layer in a single launch.  The same kernel
// with a cluster of ONE block of four warps serves narrow networks at batches of tens to a few
// thousand queries, where one warp per query leaves most of the GPU waiting on a long chain of
// dependent loads: four warps share a query's rows, the cluster barriers become block barriers and
// the remote stores local ones.
//
// Each block of the cluster keeps a full copy of the current layer input in its shared memory.
// Per layer:
//   1. the K*L hash rows are split over all warps of the cluster; every sum is written to every
//      block's shared memory (distributed shared memory stores);        cluster barrier
//   2. every block forms the keys and runs the same first-B-distinct selection redundantly, so
//      each holds the same ascending id list without a broadcast;
//   3. the selected rows are split over all warps of the cluster (one row per warp, deep load
//      prefetch); each activation is scattered into every block's copy of the next layer's
//      input;                                                           cluster barrier
// Two hardware cluster barriers per layer replace two kernel launches per layer.  Every block
// executes the same number of barriers whatever the data (no early exit).  Arithmetic is the
// library's fixed-order dot product (warp_dot_row1), so results are identical to the other paths.
#pragma once
#include <cooperative_groups.h>

#include "slonn_run_kernels.cuh"

#define SLONN_CLUSTER_MAX_D 8192
#define SLONN_CLUSTER_MAX_N 8192
#ifndef SLONN_CLUSTER_THREADS
#define SLONN_CLUSTER_THREADS 512
#endif
#ifndef SLONN_CLUSTER_DEPTH
#define SLONN_CLUSTER_DEPTH 8 // 16-byte chunks per lane in flight (12 and 16 spill at 512 threads: 152 / 185 us instead of 118)
#endif
#ifndef SLONN_CLUSTER_SIZE
#define SLONN_CLUSTER_SIZE 16 // blocks (SMs) per query; above 8 needs the non-portable cluster size opt-in
#endif

struct slonn_cluster_layer {
    const void *W;
    const float *bias;
    const uint32_t *hash_nodes;
    const void *tables;
    uint32_t D, N, nchunks, cap;
    uint32_t has_act, a, relu, id_bytes;
};

struct slonn_cluster_params {
    slonn_cluster_layer layer[SLONN_MAX_LAYERS];
    uint32_t n_layers, n, n_act, K, L, cluster;
    uint32_t pre;            // hash nodes that are always active (0 or K*L)
    const float *x;          // [n][D0]
    const uint16_t *budget_bp; // [n]
    uint32_t max_bp;
    uint64_t *indptr_out;    // [n * n_act + 1], nullable: written for the caller (the kernel derives its own offsets)
    const uint64_t *indptr_in; // [n * n_act + 1], nullable: offsets planned by an earlier launch (many queries)
    uint32_t *out_ids;       // CSR payload, nullable
    float *out_vals;         // CSR payload, nullable
    uint16_t *codes;         // nullable
    float *logits;
    uint32_t logit_stride;
    uint32_t *logit_ids;     // budgeted last layer only
    uint32_t *pred;          // nullable
    uint32_t *status;
    uint32_t xbuf_floats;    // floats per input buffer (two buffers)
    uint32_t ids_cap;        // entries of the id list
    uint32_t bitmap_words;
};

// Node count of activator layer l for query q (same rule and the same clamping as the plan kernels).
__device__ __forceinline__ uint32_t cluster_count(const slonn_cluster_params &P, uint32_t q, uint32_t l, bool *bad)
{
    uint32_t bp = P.budget_bp[q];
    *bad = (bp < 1u) || (bp > 10000u) || (bp > P.max_bp);
    if (bp < 1u) bp = 1u;
    if (bp > P.max_bp) bp = P.max_bp;
    const uint32_t B = slonn_layer_nodes(bp, P.layer[l].N, P.pre);
    if (B - P.pre > P.layer[l].cap && B != P.layer[l].N) *bad = true;
    return B;
}

template <bool BF16, int THREADS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS)
cluster_network_kernel(const __grid_constant__ slonn_cluster_params P)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ float4 smem4[];
    __shared__ float zh[128];
    __shared__ uint32_t keys[8];
    __shared__ uint32_t scan_ws[32];
    __shared__ uint32_t scan_total;

    const uint32_t C = P.cluster;
    const uint32_t rank = cluster.block_rank();
    const uint32_t q = blockIdx.x / C;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t gwarp = rank * nwarps + warp, gwarps = C * nwarps; // warp index within the cluster

    float *xbuf[2] = {reinterpret_cast<float *>(smem4), reinterpret_cast<float *>(smem4) + P.xbuf_floats};
    uint32_t *ids_s = reinterpret_cast<uint32_t *>(reinterpret_cast<float *>(smem4) + 2 * P.xbuf_floats);
    uint32_t *bitmap = ids_s + P.ids_cap;

    // List offsets: with a handful of queries every block simply adds up the counts of the (query,
    // layer) entries before its own instead of waiting for a separate planning launch.
    __shared__ uint64_t s_off[SLONN_MAX_LAYERS];
    __shared__ uint32_t s_cnt[SLONN_MAX_LAYERS];
    const bool need_offsets = P.out_ids || P.out_vals || P.indptr_out;
    if (threadIdx.x == 0 && (P.indptr_in || !need_offsets)) {
        // offsets planned by an earlier launch, or not needed at all (no list is written)
        bool bad;
        for (uint32_t l = 0; l < P.n_layers; ++l) {
            if (!P.layer[l].has_act) continue;
            s_cnt[l] = cluster_count(P, q, l, &bad);
            s_off[l] = P.indptr_in ? P.indptr_in[(uint64_t)q * P.n_act + P.layer[l].a] : 0;
            if (bad && rank == 0) slonn_report(P.status, SLONN_ERR_BUDGET, q, l);
        }
    } else if (threadIdx.x == 0) {
        uint64_t run = 0;
        bool bad;
        for (uint32_t qq = 0; qq <= q; ++qq)
            for (uint32_t l = 0; l < P.n_layers; ++l) {
                if (!P.layer[l].has_act) continue;
                const uint32_t B = cluster_count(P, qq, l, &bad);
                if (qq == q) {
                    s_off[l] = run; s_cnt[l] = B;
                    if (bad && rank == 0) slonn_report(P.status, SLONN_ERR_BUDGET, q, l);
                }
                if (rank == 0 && q + 1 == P.n && P.indptr_out) P.indptr_out[(uint64_t)qq * P.n_act + P.layer[l].a] = run;
                run += B;
            }
        if (rank == 0 && q + 1 == P.n && P.indptr_out) P.indptr_out[(uint64_t)P.n * P.n_act] = run;
    }

    // input := x (every block its own copy, in the staging order of layer 0)
    uint32_t cur = 0;
    {
        const slonn_cluster_layer &l0 = P.layer[0];
        const float4 *src = reinterpret_cast<const float4 *>(P.x + (uint64_t)q * l0.D);
        float4 *dst = reinterpret_cast<float4 *>(xbuf[0]);
#pragma unroll 4
        for (uint32_t i = threadIdx.x; i < (l0.D >> 2); i += blockDim.x) {
            const float4 v = __ldg(src + i);
            if (BF16) dst[(i & 1u) * l0.nchunks + (i >> 1)] = v;
            else dst[i] = v;
        }
    }
    // every block of the cluster must be running before a peer's shared memory is written (the hash sums of
    // the first layer are the first such stores); this also orders the staging above within the block
    cluster.sync();

    for (uint32_t l = 0; l < P.n_layers; ++l) {
        const slonn_cluster_layer &ly = P.layer[l];
        const bool is_last = (l + 1 == P.n_layers);
        const uint32_t nxt = cur ^ 1u;
        const float4 *xs4 = reinterpret_cast<const float4 *>(xbuf[cur]);
        const uint32_t next_chunks = is_last ? 0u : P.layer[l + 1].nchunks;

        // the buffer the activations of this layer are scattered into starts at zero
        {
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            float4 *dst = reinterpret_cast<float4 *>(xbuf[nxt]);
            for (uint32_t i = threadIdx.x; i < ((ly.N + 3u) >> 2); i += blockDim.x) dst[i] = z;
        }
        uint64_t off = 0;
        uint32_t B = ly.N;
        if (ly.has_act) {
            off = s_off[l];
            B = s_cnt[l];
            // 1. FreeHash rows, spread over the cluster; each sum goes to every block
            const uint32_t H = P.K * P.L;
            for (uint32_t h = gwarp; h < H; h += gwarps) {
                const uint32_t nd = __ldg(ly.hash_nodes + h);
                const float sum = warp_dot_row1<BF16, SLONN_CLUSTER_DEPTH>(reinterpret_cast<const uint4 *>(ly.W) + (uint64_t)nd * ly.nchunks,
                                                      xs4, ly.nchunks, lane);
                const float z = sum + __ldg(ly.bias + nd);
                if (lane < C) *cluster.map_shared_rank(&zh[h], lane) = z;
            }
            for (uint32_t i = threadIdx.x; i < ((ly.N + 31u) >> 5); i += blockDim.x) bitmap[i] = 0u;
        }
        cluster.sync(); // hash sums delivered, every block's next buffer zeroed

        bool implicit_ids = true;
        if (ly.has_act) {
            // 2. keys and selection, redundantly in every block
            if (threadIdx.x < P.L) {
                uint32_t key = 0;
                for (uint32_t j = 0; j < P.K; ++j)
                    if (zh[threadIdx.x * P.K + j] > 0.0f) key |= (1u << j);
                keys[threadIdx.x] = key;
                if (rank == 0 && P.codes) P.codes[((uint64_t)q * P.n_act + ly.a) * P.L + threadIdx.x] = (uint16_t)key;
            }
            __syncthreads();
            bool ok;
            if (ly.id_bytes == 2)
                ok = block_select<uint16_t>(ly.tables, ly.cap, P.K, P.L, ly.N, B, keys, bitmap, ids_s, scan_ws,
                                            &scan_total, ly.hash_nodes, P.pre);
            else
                ok = block_select<uint32_t>(ly.tables, ly.cap, P.K, P.L, ly.N, B, keys, bitmap, ids_s, scan_ws,
                                            &scan_total, ly.hash_nodes, P.pre);
            if (!ok && rank == 0 && threadIdx.x == 0) slonn_report(P.status, SLONN_ERR_ARG, q, l);
            __syncthreads();
            implicit_ids = false;
            if (rank == 0 && P.out_ids)
                for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) P.out_ids[off + i] = ids_s[i];
        }

        // 3. the selected rows, one per warp, spread over the cluster
        for (uint32_t r = gwarp; r < B; r += gwarps) {
            const uint32_t nd = implicit_ids ? r : ids_s[r];
            const float sum = warp_dot_row1<BF16, SLONN_CLUSTER_DEPTH>(reinterpret_cast<const uint4 *>(ly.W) + (uint64_t)nd * ly.nchunks, xs4,
                                                  ly.nchunks, lane);
            float z = sum + __ldg(ly.bias + nd);
            if (ly.relu) z = z > 0.0f ? z : 0.0f;
            if (lane == 0) {
                if (ly.has_act && P.out_vals) P.out_vals[off + r] = z;
                if (is_last) {
                    if (ly.has_act) {
                        P.logits[(uint64_t)q * P.logit_stride + r] = z;
                        P.logit_ids[(uint64_t)q * P.logit_stride + r] = nd;
                    } else {
                        P.logits[(uint64_t)q * P.logit_stride + nd] = z;
                    }
                }
            }
            // next layer's input (or, after the last layer, the logits by position for the argmax)
            if (!is_last) {
                if (lane < C) *cluster.map_shared_rank(&xbuf[nxt][xs_index<BF16>(nd, next_chunks)], lane) = z;
            } else if (lane == 0) {
                *cluster.map_shared_rank(&xbuf[nxt][r], 0) = z;
            }
        }
        cluster.sync(); // every activation of this layer delivered
        cur = nxt;

        if (is_last && rank == 0 && P.pred) {
            // prediction: lowest node id among the largest computed logits (block 0 holds them by position)
            const float *lg = xbuf[cur];
            float best = 0.0f;
            uint32_t bi = 0xffffffffu;
            for (uint32_t i = threadIdx.x; i < B; i += blockDim.x) {
                const float v = lg[i];
                if (bi == 0xffffffffu || v > best) { best = v; bi = i; }
            }
            // positions ascend with node ids, so the lowest position is the lowest id
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const float ob = __shfl_xor_sync(SLONN_FULL_MASK, best, o);
                const uint32_t oi = __shfl_xor_sync(SLONN_FULL_MASK, bi, o);
                if (oi != 0xffffffffu && (bi == 0xffffffffu || ob > best || (ob == best && oi < bi))) { best = ob; bi = oi; }
            }
            __shared__ float wbest[32];
            __shared__ uint32_t wbi[32];
            if (lane == 0) { wbest[warp] = best; wbi[warp] = bi; }
            __syncthreads();
            if (warp == 0) {
                best = lane < nwarps ? wbest[lane] : 0.0f;
                bi = lane < nwarps ? wbi[lane] : 0xffffffffu;
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) {
                    const float ob = __shfl_xor_sync(SLONN_FULL_MASK, best, o);
                    const uint32_t oi = __shfl_xor_sync(SLONN_FULL_MASK, bi, o);
                    if (oi != 0xffffffffu && (bi == 0xffffffffu || ob > best || (ob == best && oi < bi))) { best = ob; bi = oi; }
                }
                if (lane == 0 && bi != 0xffffffffu) P.pred[q] = implicit_ids ? bi : ids_s[bi];
            }
        }
    }
}
