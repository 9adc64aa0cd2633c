// Whole-network kernel for narrow layers: one warp carries one query through
// every layer (hash -> keys -> bucket lists -> top-k% -> selected rows ->
// next layer) with the layer input held in registers.  Used when every layer's
// input width is at most 1024 and every activator layer at most 4096 nodes
// wide; wider networks use the per-stage kernels.
//
// Same arithmetic as everywhere else in the library: lane p owns partial sum
// p and takes 16-byte weight chunks p, p+32, ... in ascending order; partials
// are added pairwise with strides 16, 8, 4, 2, 1; bias last.
//
// A layer fed by the sparse output of the activator layer below takes, for queries whose budget leaves
// that output sparse, the input-stationary form (slonn_cols_kernels.cuh): the warp groups the nonzero
// inputs by partial sum in its own shared memory, then lanes own nodes -- the K*L hash nodes in one pass
// over the layer's side-by-side hash rows, the selected nodes 64 per pass over the transposed weights.
// Same sums in the same order, so which form a query takes does not show in its results.
#pragma once
#include "slonn_common.cuh"
#include "slonn_cols_kernels.cuh"

#define SLONN_FUSED_ROWS 4          // rows per pass; the 6-shuffle reduction is written for 4
#ifndef SLONN_FUSED_WARPS
#define SLONN_FUSED_WARPS 4         // queries (warps) per block
#endif
#ifndef SLONN_FUSED_MIN_BLOCKS
#define SLONN_FUSED_MIN_BLOCKS 5    // resident blocks per SM the register allocation must allow
#endif
#define SLONN_FUSED_MAX_D 1024
#define SLONN_FUSED_MAX_N 4096

struct slonn_fused_layer {
    const void *W;
    const float *bias;
    const uint32_t *hash_nodes;
    const void *tables;
    uint32_t D, N, nchunks, cap;
    uint32_t has_act, a, relu, id_bytes;
    const void *WT;          // transposed copy [D][N] in colpos order, or NULL
    const void *WH;          // hash rows side by side [D][32], or NULL
    const uint32_t *colpos;  // node id -> column of WT
};

struct slonn_fused_params {
    slonn_fused_layer layer[SLONN_MAX_LAYERS];
    uint32_t n_layers, n, n_act, K, L;
    uint32_t pre;            // hash nodes that are always active (0 or K*L)
    const uint16_t *skip_bp; // nullable: queries with this budget == 10000 are handled elsewhere
    const uint16_t *budget_bp; // [n]
    const float *x;          // [n][D0]
    const uint64_t *indptr;  // [n * n_act + 1]; NULL when no active list is written (counts then come from the budgets)
    uint32_t max_bp;         // the batch's stated largest budget
    uint32_t *out_ids;       // CSR payload, nullable
    float *out_vals;         // CSR payload, nullable
    uint16_t *codes;         // nullable
    float *logits;
    uint32_t logit_stride;
    uint32_t *logit_ids;     // budgeted last layer only
    uint32_t *pred;          // nullable
    uint32_t *status;
    uint32_t xbuf_floats, ids_cap, bitmap_words, warp_bytes; // per-warp shared memory carve
    uint32_t cols_bp;        // budgets up to this take the input-stationary form where a layer offers it (0 = never)
    uint32_t ent_cap;        // entries of a warp's grouped input list (0 = no room set aside)
};

template <bool BF16>
struct fused_traits {
    static constexpr int VPC = BF16 ? 8 : 4; // input values per 16-byte weight chunk
};

// x registers <- dense global row
template <bool BF16, int NC>
__device__ __forceinline__ void fused_load_x_global(float (&xr)[NC * fused_traits<BF16>::VPC], const float *row,
                                                    uint32_t nchunks, uint32_t lane)
{
    constexpr int VPC = fused_traits<BF16>::VPC;
    const float4 *x4 = reinterpret_cast<const float4 *>(row);
#pragma unroll
    for (int i = 0; i < NC; ++i) {
        const uint32_t c = lane + 32u * i;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (c < nchunks) {
            if (BF16) { a = __ldg(x4 + 2 * c); b = __ldg(x4 + 2 * c + 1); }
            else a = __ldg(x4 + c);
        }
        xr[i * VPC + 0] = a.x; xr[i * VPC + 1] = a.y; xr[i * VPC + 2] = a.z; xr[i * VPC + 3] = a.w;
        if (BF16) { xr[i * VPC + 4] = b.x; xr[i * VPC + 5] = b.y; xr[i * VPC + 6] = b.z; xr[i * VPC + 7] = b.w; }
    }
}

// x registers <- this warp's staged vector (xs_index layout for `nchunks`)
template <bool BF16, int NC>
__device__ __forceinline__ void fused_load_x_shared(float (&xr)[NC * fused_traits<BF16>::VPC], const float4 *xs4,
                                                    uint32_t nchunks, uint32_t lane)
{
    constexpr int VPC = fused_traits<BF16>::VPC;
#pragma unroll
    for (int i = 0; i < NC; ++i) {
        const uint32_t c = lane + 32u * i;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (c < nchunks) {
            a = xs4[c];
            if (BF16) b = xs4[nchunks + c];
        }
        xr[i * VPC + 0] = a.x; xr[i * VPC + 1] = a.y; xr[i * VPC + 2] = a.z; xr[i * VPC + 3] = a.w;
        if (BF16) { xr[i * VPC + 4] = b.x; xr[i * VPC + 5] = b.y; xr[i * VPC + 6] = b.z; xr[i * VPC + 7] = b.w; }
    }
}

// Fixed-order partial sums of R rows against the register-resident input: lane p ends
// with partial p of every row (the caller reduces them).
// GRP: 32-chunk rounds whose loads are issued together (1 when the batch fills the GPU and registers are
// better spent on resident warps; all of them when a few warps have an SM to themselves).
template <bool BF16, int NC, int R, int GRP>
__device__ __forceinline__ void fused_dot_rows(const uint4 *const (&rows)[R],
                                               const float (&xr)[NC * fused_traits<BF16>::VPC], uint32_t nchunks,
                                               uint32_t lane, float (&acc)[R])
{
    constexpr int VPC = fused_traits<BF16>::VPC;
    constexpr int G = NC < GRP ? NC : GRP; // rounds whose loads are issued together
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0f;
#pragma unroll
    for (int i0 = 0; i0 < NC; i0 += G) {
        uint4 w[G][R];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint32_t c = lane + 32u * (i0 + g);
            if (c < nchunks) {
#pragma unroll
                for (int r = 0; r < R; ++r) w[g][r] = __ldg(rows[r] + c);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint32_t c = lane + 32u * (i0 + g);
            if (c < nchunks) chunk_fma<BF16, R, 0, VPC>::run(w[g], &xr[(i0 + g) * VPC], acc);
        }
    }
}

template <typename IDT>
__device__ __forceinline__ uint32_t fused_table_entry(const void *tables, uint32_t cap, uint32_t K, uint32_t b,
                                                      uint32_t key, uint32_t r)
{
    const IDT *t = reinterpret_cast<const IDT *>(tables);
    return (uint32_t)__ldg(t + (((uint64_t)b << K) + key) * cap + r);
}

// The first `pre` hash nodes and the first B - pre distinct ids of the rank-interleaved bucket
// lists -> ids_s[0..B) ascending.  mykey: lane b holds the key of table b.  One warp, no block barrier.
__device__ __forceinline__ void fused_select(const slonn_fused_layer &ly, uint32_t K, uint32_t L, uint32_t mykey,
                                             uint32_t B, uint32_t pre, uint32_t *bitmap, uint16_t *ids_s, uint32_t lane)
{
    const uint32_t nwords = (ly.N + 31u) >> 5;
    for (uint32_t w = lane; w < nwords; w += 32) bitmap[w] = 0u;
    __syncwarp();
    if (pre) {
        for (uint32_t h = lane; h < pre; h += 32) {
            const uint32_t nd = __ldg(ly.hash_nodes + h);
            atomicOr(&bitmap[nd >> 5], 1u << (nd & 31u));
        }
        __syncwarp();
    }
    const uint32_t want = B - pre;
    const uint32_t npos = want * L;
    uint32_t total = 0;
    for (uint32_t base = 0; base < npos && total < want; base += 32) {
        const uint32_t pos = base + lane;
        uint32_t id = 0xffffffffu - lane; // distinct dummies for lanes past the end
        bool fresh = false;
        const uint32_t r = pos / L, b = pos - r * L;
        const uint32_t key = __shfl_sync(SLONN_FULL_MASK, mykey, b & 31u);
        if (pos < npos) {
            id = ly.id_bytes == 2 ? fused_table_entry<uint16_t>(ly.tables, ly.cap, K, b, key, r)
                                  : fused_table_entry<uint32_t>(ly.tables, ly.cap, K, b, key, r);
            if (id < ly.N) fresh = ((bitmap[id >> 5] >> (id & 31u)) & 1u) == 0u;
        }
        const uint32_t same = __match_any_sync(SLONN_FULL_MASK, id);
        const bool take = fresh && ((uint32_t)(__ffs(same) - 1) == lane);
        const uint32_t bal = __ballot_sync(SLONN_FULL_MASK, take);
        const uint32_t need = want - total;
        const uint32_t rank = __popc(bal & ((1u << lane) - 1u));
        if (take && rank < need) atomicOr(&bitmap[id >> 5], 1u << (id & 31u));
        const uint32_t c = (uint32_t)__popc(bal);
        total += c < need ? c : need;
        __syncwarp();
    }
    uint32_t running = 0;
    for (uint32_t w0 = 0; w0 < nwords; w0 += 32) {
        const uint32_t w = w0 + lane;
        uint32_t bits = w < nwords ? bitmap[w] : 0u;
        const uint32_t cnt = __popc(bits);
        uint32_t incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(SLONN_FULL_MASK, incl, off);
            if (lane >= (uint32_t)off) incl += t;
        }
        uint32_t o = running + incl - cnt;
        while (bits) {
            const uint32_t t = __ffs(bits) - 1;
            bits &= bits - 1;
            if (o < B) ids_s[o] = (uint16_t)((w << 5) + t);
            ++o;
        }
        running += __shfl_sync(SLONN_FULL_MASK, incl, 31);
    }
    __syncwarp();
}

// COLS: compiled with the input-stationary form (chosen on the host per batch; without it the kernel is
// the plain row form and carries none of the extra state).
template <bool BF16, int NC, int GRP, bool COLS>
__global__ void __launch_bounds__(SLONN_FUSED_WARPS * 32, GRP == 1 ? SLONN_FUSED_MIN_BLOCKS : 1)
fused_network_kernel(const __grid_constant__ slonn_fused_params P)
{
    constexpr int VPC = fused_traits<BF16>::VPC;
    constexpr int R = SLONN_FUSED_ROWS;
    extern __shared__ float4 smem4[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t q = blockIdx.x * SLONN_FUSED_WARPS + warp;
    if (q >= P.n) return;
    if (P.skip_bp && P.skip_bp[q] == 10000u) return;
    unsigned char *wbase = reinterpret_cast<unsigned char *>(smem4) + (size_t)warp * P.warp_bytes;
    float4 *xbuf4 = reinterpret_cast<float4 *>(wbase);
    float *xbuf = reinterpret_cast<float *>(wbase);
    uint16_t *ids_s = reinterpret_cast<uint16_t *>(wbase + (size_t)P.xbuf_floats * 4);
    uint32_t *bitmap = reinterpret_cast<uint32_t *>(wbase + (size_t)P.xbuf_floats * 4 + (size_t)P.ids_cap * 2);

    // grouped nonzero inputs of the input-stationary form (this warp's own)
    cols_stage S;
    S.xs = nullptr;
    S.ent = reinterpret_cast<uint2 *>(wbase + (((size_t)P.xbuf_floats * 4 + (size_t)P.ids_cap * 2 + (size_t)P.bitmap_words * 4 + 15) & ~(size_t)15)); // 16-byte aligned: read as uint4
    S.segcnt = reinterpret_cast<uint32_t *>(S.ent + P.ent_cap);
    S.segstart = S.segcnt + 32;

    float xr[NC * VPC];
    float best = 0.0f;          // running argmax over the last layer (per lane)
    uint32_t best_id = 0xffffffffu;
    uint32_t prev_B = 0;        // entries of the list in ids_s left by the layer below (0 = none / every node)
    const uint32_t my_bp = (COLS && P.cols_bp) ? (uint32_t)P.budget_bp[q] : 0u;

    for (uint32_t l = 0; l < P.n_layers; ++l) {
        const slonn_fused_layer &ly = P.layer[l];
        const bool is_last = (l + 1 == P.n_layers);
        // the input-stationary form: this layer keeps the copies it needs, the input is a list that fits
        // the warp's entry buffer, and the query's budget leaves it sparse
        const bool cols = COLS && P.cols_bp && ly.has_act && ly.WT && ly.WH && prev_B && prev_B + 96u <= P.ent_cap && my_bp <= P.cols_bp;
        // input := previous activation (registers, or the grouped list of its nonzeros)
        if (COLS && cols) cols_stage_warp<BF16>(S, ids_s, prev_B, xbuf, ly.nchunks, lane);
        else if (l == 0) fused_load_x_global<BF16, NC>(xr, P.x + (uint64_t)q * ly.D, ly.nchunks, lane);
        else fused_load_x_shared<BF16, NC>(xr, xbuf4, ly.nchunks, lane);
        __syncwarp();
        uint32_t next_chunks = 0;
        if (!is_last) { // clear the staging vector the selected nodes' activations go to
            next_chunks = P.layer[l + 1].nchunks;
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t i = lane; i < (ly.N >> 2); i += 32) xbuf4[i] = z;
            __syncwarp();
        }

        uint32_t B = ly.N;
        uint64_t off = 0;
        bool implicit_ids = true;
        if (ly.has_act) {
            if (P.indptr) {
                off = P.indptr[(uint64_t)q * P.n_act + ly.a];
                B = (uint32_t)(P.indptr[(uint64_t)q * P.n_act + ly.a + 1] - off);
            } else { // no list is written, so no offsets were planned: the count follows from the budget alone
                uint32_t bp = P.budget_bp[q];
                bool bad = (bp < 1u) || (bp > 10000u) || (bp > P.max_bp);
                bp = min(max(bp, 1u), P.max_bp);
                B = slonn_layer_nodes(bp, ly.N, P.pre);
                if (B - P.pre > ly.cap && B != ly.N) bad = true;
                if (bad && lane == 0) slonn_report(P.status, SLONN_ERR_BUDGET, q, l);
            }
            // FreeHash: signs of the K*L sampled nodes' pre-activations
            const uint32_t H = P.K * P.L;
            uint32_t mykey = 0;
            if (COLS && cols) { // lane h computes hash node h from the side-by-side hash rows
                const uint32_t col[1] = {lane};
                float sum[1];
                cols_walk<BF16, 1>(S, ly.WH, 32u, col, sum);
                const float z = sum[0] + __ldg(ly.bias + __ldg(ly.hash_nodes + min(lane, H - 1)));
                const uint32_t signs = __ballot_sync(SLONN_FULL_MASK, lane < H && z > 0.0f);
                if (lane < P.L) mykey = (signs >> (lane * P.K)) & ((1u << P.K) - 1u);
            } else
            for (uint32_t h0 = 0; h0 < H; h0 += R) {
                const uint4 *rows[R];
#pragma unroll
                for (int k = 0; k < R; ++k) {
                    const uint32_t nd = __ldg(ly.hash_nodes + min(h0 + k, H - 1));
                    rows[k] = reinterpret_cast<const uint4 *>(ly.W) + (uint64_t)nd * ly.nchunks;
                }
                float acc[R];
                fused_dot_rows<BF16, NC, R, GRP>(rows, xr, ly.nchunks, lane, acc);
                // lanes 8k..8k+7 hold the sum of row k; collect the R signs with one ballot
                const uint32_t mynode = __ldg(ly.hash_nodes + min(h0 + (lane >> 3), H - 1));
                const float z = reduce_rows4(acc, lane) + __ldg(ly.bias + mynode);
                const uint32_t signs = __ballot_sync(SLONN_FULL_MASK, z > 0.0f);
#pragma unroll
                for (int k = 0; k < R; ++k) {
                    const uint32_t h = h0 + k;
                    if (h < H) {
                        const uint32_t tb = h / P.K, j = h - tb * P.K;
                        if (lane == tb && ((signs >> (8 * k)) & 1u)) mykey |= (1u << j);
                    }
                }
            }
            if (P.codes && lane < P.L) P.codes[((uint64_t)q * P.n_act + ly.a) * P.L + lane] = (uint16_t)mykey;
            if (B != ly.N && B - P.pre <= ly.cap) {
                fused_select(ly, P.K, P.L, mykey, B, P.pre, bitmap, ids_s, lane);
                implicit_ids = false;
            }
            if (P.out_ids) {
                for (uint32_t i = lane; i < B; i += 32) P.out_ids[off + i] = implicit_ids ? i : (uint32_t)ids_s[i];
            }
        }

        // the selected nodes
        if (COLS && cols) {
            for (uint32_t r0 = 0; r0 < B; r0 += 64) {
                uint32_t nd[2], col[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint32_t rr = min(r0 + k * 32u + lane, B - 1);
                    nd[k] = implicit_ids ? rr : (uint32_t)ids_s[rr];
                    col[k] = __ldg(ly.colpos + nd[k]);
                }
                float sum[2];
                cols_walk<BF16, 2>(S, ly.WT, ly.N, col, sum);
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint32_t r = r0 + k * 32u + lane;
                    if (r < B) {
                        float z = sum[k] + __ldg(ly.bias + nd[k]);
                        if (ly.relu) z = z > 0.0f ? z : 0.0f;
                        if (P.out_vals) P.out_vals[off + r] = z;
                        if (!is_last) {
                            xbuf[xs_index<BF16>(nd[k], next_chunks)] = z;
                        } else {
                            P.logits[(uint64_t)q * P.logit_stride + r] = z;
                            P.logit_ids[(uint64_t)q * P.logit_stride + r] = nd[k];
                            if (best_id == 0xffffffffu || z > best) { best = z; best_id = nd[k]; }
                        }
                    }
                }
            }
        } else
        for (uint32_t r0 = 0; r0 < B; r0 += R) {
            const uint4 *rows[R];
#pragma unroll
            for (int k = 0; k < R; ++k) {
                const uint32_t rr = min(r0 + k, B - 1);
                const uint32_t nd = implicit_ids ? rr : (uint32_t)ids_s[rr];
                rows[k] = reinterpret_cast<const uint4 *>(ly.W) + (uint64_t)nd * ly.nchunks;
            }
            float acc[R];
            fused_dot_rows<BF16, NC, R, GRP>(rows, xr, ly.nchunks, lane, acc);
            const float sum = reduce_rows4(acc, lane); // row r0 + (lane >> 3)
            const uint32_t r = r0 + (lane >> 3);
            if ((lane & 7u) == 0u && r < B) {
                const uint32_t nd = implicit_ids ? r : (uint32_t)ids_s[r];
                float z = sum + __ldg(ly.bias + nd);
                if (ly.relu) z = z > 0.0f ? z : 0.0f;
                if (ly.has_act && P.out_vals) P.out_vals[off + r] = z;
                if (!is_last) {
                    xbuf[xs_index<BF16>(nd, next_chunks)] = z;
                } else {
                    if (ly.has_act) {
                        P.logits[(uint64_t)q * P.logit_stride + r] = z;
                        P.logit_ids[(uint64_t)q * P.logit_stride + r] = nd;
                    } else {
                        P.logits[(uint64_t)q * P.logit_stride + nd] = z;
                    }
                    if (best_id == 0xffffffffu || z > best) { best = z; best_id = nd; }
                }
            }
        }
        __syncwarp();
        if (COLS) prev_B = (ly.has_act && !implicit_ids) ? B : 0u;
    }

    if (P.pred) { // lowest node id among the largest logits
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const float ob = __shfl_xor_sync(SLONN_FULL_MASK, best, off);
            const uint32_t oi = __shfl_xor_sync(SLONN_FULL_MASK, best_id, off);
            if (oi != 0xffffffffu && (best_id == 0xffffffffu || ob > best || (ob == best && oi < best_id))) {
                best = ob;
                best_id = oi;
            }
        }
        if (lane == 0 && best_id != 0xffffffffu) P.pred[q] = best_id;
    }
}
