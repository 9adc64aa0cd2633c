// Input-stationary ("column") kernels for layers whose input is a sparse (id, value) list
// (Sec. 3.3: the output of a layer with a Node Activator holds only the computed nodes; every
// other input of the next layer is exactly 0 and contributes nothing).
//
// The row kernels read every selected weight row whole and multiply most of it by zeros.  Here
// the roles are swapped: a lane owns one selected node n and keeps that node's 32 partial sums in
// registers; the warp walks the NONZERO inputs j and each lane reads the single weight WT[j][n]
// from the transposed copy.  Work is (nonzero inputs) x (selected nodes) multiply-adds instead of
// (layer width) x (selected nodes).
//
// The summation order is the library's fixed one: input j belongs to partial (j / V) mod 32 and a
// partial takes its inputs in ascending j; skipping an input that is exactly 0 leaves a partial
// unchanged (fmaf(w, 0, a) == a for finite w).  To get "ascending j within each partial" with a
// warp-uniform loop, the nonzero inputs are first grouped by partial (32 segments, each ascending in
// j); the loop over segments is unrolled so that partial p is a fixed register.  The 32 partials
// are then added in the tree 16, 8, 4, 2, 1 inside the lane, which performs the same additions as
// the shuffle butterfly of the row kernels.
#pragma once
#include "slonn_common.cuh"

// Shared-memory image of one query's nonzero inputs, grouped by partial sum.
struct cols_stage {
    float *xs;          // [32 * smax] scratch: inputs in segment-major order (zero = absent)
    uint2 *ent;         // [cols_ent_cap] entries (j, bits of x_j), segment after segment
    uint32_t *segcnt;   // [32]
    uint32_t *segstart; // [33]
};

// floats per segment of the scratch: the chunks a partial owns, V inputs each
__host__ __device__ __forceinline__ uint32_t cols_smax(uint32_t D, uint32_t V)
{
    const uint32_t nchunks = (D + V - 1) / V;
    return ((nchunks + 31u) / 32u) * V;
}

// entries the staged list can take: every nonzero input, each of the 32 segments filled up to a multiple of 4
__host__ __device__ __forceinline__ uint32_t cols_ent_cap(uint32_t D, uint32_t in_cap)
{
    return (in_cap < D ? in_cap : D) + 96u;
}

// bytes of the input image a block scatters the list into while staging
__host__ __device__ __forceinline__ size_t cols_image_bytes(uint32_t D, uint32_t V)
{
    return (size_t)32 * cols_smax(D, V) * 4;
}

// Builds the grouped nonzero list of query segment [s0, s0 + len) of (ids, vals).  Whole block; ends
// with a barrier.
template <int V>
__device__ __forceinline__ void cols_stage_list(const cols_stage &S, const uint32_t *ids, const float *vals, uint64_t s0,
                                                uint32_t len, uint32_t D)
{
    const uint32_t smax = cols_smax(D, V);
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (uint32_t i = threadIdx.x; i < 32u * smax; i += blockDim.x) S.xs[i] = 0.0f;
    __syncthreads();
#pragma unroll 4
    for (uint32_t i = threadIdx.x; i < len; i += blockDim.x) {
        const uint32_t j = __ldg(ids + s0 + i);
        const float v = __ldg(vals + s0 + i);
        if (j < D) {
            const uint32_t c = j / V, p = c & 31u;
            S.xs[p * smax + (c >> 5) * V + (j - c * V)] = v;
        }
    }
    __syncthreads();
    // nonzeros per segment, counted on the scattered image (so that a repeated id counts once)
    for (uint32_t p = warp; p < 32; p += nwarps) {
        uint32_t cnt = 0;
        for (uint32_t pos0 = 0; pos0 < smax; pos0 += 32) {
            const uint32_t pos = pos0 + lane;
            const float v = pos < smax ? S.xs[p * smax + pos] : 0.0f;
            cnt += __popc(__ballot_sync(SLONN_FULL_MASK, v != 0.0f));
        }
        if (lane == 0) S.segcnt[p] = cnt;
    }
    __syncthreads();
    if (warp == 0) { // segments start at multiples of 4 entries
        const uint32_t c = (S.segcnt[lane] + 3u) & ~3u;
        uint32_t incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(SLONN_FULL_MASK, incl, off);
            if (lane >= (uint32_t)off) incl += t;
        }
        S.segstart[lane] = incl - c;
        if (lane == 31) S.segstart[32] = incl;
    }
    __syncthreads();
    for (uint32_t p = warp; p < 32; p += nwarps) {
        uint32_t base = S.segstart[p];
        for (uint32_t pos0 = 0; pos0 < smax; pos0 += 32) {
            const uint32_t pos = pos0 + lane;
            const float v = pos < smax ? S.xs[p * smax + pos] : 0.0f;
            const uint32_t m = __ballot_sync(SLONN_FULL_MASK, v != 0.0f);
            if (v != 0.0f) {
                const uint32_t blk = pos / V;
                const uint32_t j = (blk * 32u + p) * V + (pos - blk * V);
                S.ent[base + __popc(m & ((1u << lane) - 1u))] = make_uint2(j, __float_as_uint(v));
            }
            base += __popc(m);
        }
        // fill up to the next multiple of 4 with copies of the last input carrying the value 0
        // (a multiply-add by 0 leaves the partial sum as it is)
        __syncwarp();
        const uint32_t pad = S.segstart[p + 1] - base;
        if (lane < pad) S.ent[base + lane] = make_uint2(S.ent[base - 1].x, 0u);
    }
    __syncthreads();
}

template <bool BF16>
__device__ __forceinline__ float cols_weight(const void *WT, uint32_t idx)
{
    if (BF16) return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(WT) + idx) << 16);
    return __ldg(reinterpret_cast<const float *>(WT) + idx);
}

// The weight `off` BYTES into WT.  Offsets are 32-bit (a transposed copy is kept only for layers of less
// than 4 GiB), so an address is the matrix base plus one 32-bit sum per load.
template <bool BF16>
__device__ __forceinline__ float cols_weight_at(const void *WT, uint32_t off)
{
    const char *p = reinterpret_cast<const char *>(WT) + off;
    if (BF16) return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p)) << 16);
    return __ldg(reinterpret_cast<const float *>(p));
}

// Two neighbouring weights with one load, the first `off` bytes into WT (a multiple of two element sizes).
template <bool BF16>
__device__ __forceinline__ void cols_weight2_at(const void *WT, uint32_t off, float &w0, float &w1)
{
    const char *p = reinterpret_cast<const char *>(WT) + off;
    if (BF16) {
        const uint32_t u = __ldg(reinterpret_cast<const uint32_t *>(p));
        w0 = __uint_as_float(u << 16);
        w1 = __uint_as_float(u & 0xffff0000u);
    } else {
        const float2 v = __ldg(reinterpret_cast<const float2 *>(p));
        w0 = v.x;
        w1 = v.y;
    }
}

// Two neighbouring weights WT[idx], WT[idx + 1] with one load; idx even.
template <bool BF16>
__device__ __forceinline__ void cols_weight2(const void *WT, uint32_t idx, float &w0, float &w1)
{
    if (BF16) {
        const uint32_t u = __ldg(reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint16_t *>(WT) + idx));
        w0 = __uint_as_float(u << 16);
        w1 = __uint_as_float(u & 0xffff0000u);
    } else {
        const float2 v = __ldg(reinterpret_cast<const float2 *>(reinterpret_cast<const float *>(WT) + idx));
        w0 = v.x;
        w1 = v.y;
    }
}

// Entries [k, e) of one segment of the staged list (a multiple of four) for R nodes per lane:
// a[r] = fmaf(weight(row of the entry, column byte offset cb[r]), value of the entry, a[r]), entries in order.
// ldb: bytes per row of WT.  DEEP: eight entries at a time while the segment has that many left (8 * R loads
// in flight instead of 4 * R) -- for launches in which a block's chain of dependent loads, not the number of
// resident warps, sets the pace.
template <bool BF16, int R, bool DEEP>
__device__ __forceinline__ void cols_segment(const uint2 *ent, uint32_t k, uint32_t e, const void *WT, uint32_t ldb,
                                             const uint32_t (&cb)[R], float (&a)[R])
{
    if (DEEP) {
        for (; k + 8 <= e; k += 8) {
            uint4 q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const uint4 *>(ent + k + 2 * i);
            float w[R][8];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    w[r][2 * i] = cols_weight_at<BF16>(WT, q[i].x * ldb + cb[r]);
                    w[r][2 * i + 1] = cols_weight_at<BF16>(WT, q[i].z * ldb + cb[r]);
                }
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    a[r] = fmaf(w[r][2 * i], __uint_as_float(q[i].y), a[r]);
                    a[r] = fmaf(w[r][2 * i + 1], __uint_as_float(q[i].w), a[r]);
                }
        }
    }
    for (; k < e; k += 4) {
        const uint4 e0 = *reinterpret_cast<const uint4 *>(ent + k), e1 = *reinterpret_cast<const uint4 *>(ent + k + 2);
        float w[R][4];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            w[r][0] = cols_weight_at<BF16>(WT, e0.x * ldb + cb[r]);
            w[r][1] = cols_weight_at<BF16>(WT, e0.z * ldb + cb[r]);
            w[r][2] = cols_weight_at<BF16>(WT, e1.x * ldb + cb[r]);
            w[r][3] = cols_weight_at<BF16>(WT, e1.z * ldb + cb[r]);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            a[r] = fmaf(w[r][0], __uint_as_float(e0.y), a[r]);
            a[r] = fmaf(w[r][1], __uint_as_float(e0.w), a[r]);
            a[r] = fmaf(w[r][2], __uint_as_float(e1.y), a[r]);
            a[r] = fmaf(w[r][3], __uint_as_float(e1.w), a[r]);
        }
    }
}

// The 16 / element size neighbouring weights that start `off` bytes into WT (a multiple of 16), with one load.
template <bool BF16>
__device__ __forceinline__ void cols_weights16_at(const void *WT, uint32_t off, float (&f)[BF16 ? 8 : 4])
{
    const uint4 q = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const char *>(WT) + off));
    if constexpr (BF16) {
        f[0] = bf16_lo(q.x); f[1] = bf16_hi(q.x); f[2] = bf16_lo(q.y); f[3] = bf16_hi(q.y);
        f[4] = bf16_lo(q.z); f[5] = bf16_hi(q.z); f[6] = bf16_lo(q.w); f[7] = bf16_hi(q.w);
    } else {
        f[0] = __uint_as_float(q.x); f[1] = __uint_as_float(q.y); f[2] = __uint_as_float(q.z); f[3] = __uint_as_float(q.w);
    }
}

// a[0] + ... + a[31] in the fixed tree: strides 16, 8, 4, 2, 1
__device__ __forceinline__ float cols_tree(float (&acc)[32])
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
        for (int p = 0; p < off; ++p) acc[p] = acc[p] + acc[p + off];
    }
    return acc[0];
}

// The complete sums of R nodes (columns col[0..R)) over the staged nonzero inputs, bias not included.
//
// The 32 partial sums are taken in bit-reversed order (0, 16, 8, 24, 4, ...) and added as soon as both
// operands of a tree node exist: a[0] + a[16] after the second segment, (a[0] + a[16]) + (a[8] + a[24])
// after the fourth, and so on -- the same additions as "for off in 16, 8, 4, 2, 1: a[p] += a[p + off]",
// with at most five pending partial results per node instead of 32 registers.
// A segment holds a multiple of 4 entries; 4 entries x R loads are in flight at a time.
// Row j of WT starts at element j * ld.
// LOAD = COLS_LOAD_PAIR (R = 2): the two nodes are the neighbouring columns col[0] (even) and col[0] + 1 of a WT
// with even ld, fetched with one load per input.  LOAD = COLS_LOAD_VEC (R = 16 / element size): the nodes are the
// R neighbouring columns from col[0] (a multiple of R) of a WT whose ld is a multiple of R, one 16-byte load per input.
enum { COLS_LOAD_ONE = 0, COLS_LOAD_PAIR = 1, COLS_LOAD_VEC = 2 };
template <bool BF16, int R, int LOAD = COLS_LOAD_ONE>
__device__ __forceinline__ void cols_walk(const cols_stage &S, const void *WT, uint32_t ld, const uint32_t (&col)[R],
                                          float (&sum)[R])
{
    float p0[R], p1[R], p2[R], p3[R], p4[R];
    constexpr uint32_t ESZ = BF16 ? 2u : 4u;
    const uint32_t ldb = ld * ESZ; // bytes per row of WT
    uint32_t cb[R];                // byte offset of each node's column
#pragma unroll
    for (int r = 0; r < R; ++r) cb[r] = col[r] * ESZ;
#ifndef SLONN_COLS_UNROLL
#define SLONN_COLS_UNROLL 32 // measured: full unrolling of the segment loop beats 1, 4 and 8
#endif
#ifndef SLONN_COLS_INNER
#define SLONN_COLS_INNER 1
#endif
    constexpr int UNROLL_SEG = SLONN_COLS_UNROLL, UNROLL_BATCH = SLONN_COLS_INNER;
#pragma unroll UNROLL_SEG
    for (uint32_t i = 0; i < 32; ++i) {
        const uint32_t P = __brev(i) >> 27;
        uint32_t k = S.segstart[P];
        const uint32_t e = S.segstart[P + 1];
        float a[R];
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = 0.0f;
#pragma unroll UNROLL_BATCH
        for (; k < e; k += 4) {
            const uint4 e0 = *reinterpret_cast<const uint4 *>(S.ent + k), e1 = *reinterpret_cast<const uint4 *>(S.ent + k + 2);
            float w[R][4];
            const uint32_t t0 = e0.x * ldb, t1 = e0.z * ldb, t2 = e1.x * ldb, t3 = e1.z * ldb; // row offsets
            if constexpr (LOAD == COLS_LOAD_VEC) {
                static_assert(LOAD != COLS_LOAD_VEC || R == (BF16 ? 8 : 4), "one 16-byte load holds R weights");
                float f0[BF16 ? 8 : 4], f1[BF16 ? 8 : 4], f2[BF16 ? 8 : 4], f3[BF16 ? 8 : 4];
                cols_weights16_at<BF16>(WT, t0 + cb[0], f0);
                cols_weights16_at<BF16>(WT, t1 + cb[0], f1);
                cols_weights16_at<BF16>(WT, t2 + cb[0], f2);
                cols_weights16_at<BF16>(WT, t3 + cb[0], f3);
#pragma unroll
                for (int r = 0; r < R; ++r) { w[r][0] = f0[r]; w[r][1] = f1[r]; w[r][2] = f2[r]; w[r][3] = f3[r]; }
            } else if constexpr (LOAD == COLS_LOAD_PAIR) {
                cols_weight2_at<BF16>(WT, t0 + cb[0], w[0][0], w[R - 1][0]);
                cols_weight2_at<BF16>(WT, t1 + cb[0], w[0][1], w[R - 1][1]);
                cols_weight2_at<BF16>(WT, t2 + cb[0], w[0][2], w[R - 1][2]);
                cols_weight2_at<BF16>(WT, t3 + cb[0], w[0][3], w[R - 1][3]);
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    w[r][0] = cols_weight_at<BF16>(WT, t0 + cb[r]);
                    w[r][1] = cols_weight_at<BF16>(WT, t1 + cb[r]);
                    w[r][2] = cols_weight_at<BF16>(WT, t2 + cb[r]);
                    w[r][3] = cols_weight_at<BF16>(WT, t3 + cb[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) a[r] = fmaf(w[r][0], __uint_as_float(e0.y), a[r]);
#pragma unroll
            for (int r = 0; r < R; ++r) a[r] = fmaf(w[r][1], __uint_as_float(e0.w), a[r]);
#pragma unroll
            for (int r = 0; r < R; ++r) a[r] = fmaf(w[r][2], __uint_as_float(e1.y), a[r]);
#pragma unroll
            for (int r = 0; r < R; ++r) a[r] = fmaf(w[r][3], __uint_as_float(e1.w), a[r]);
        }
        // fold into the pending tree nodes: level t pairs partials whose index differs in bit (4 - t)
        if (!(i & 1u)) {
#pragma unroll
            for (int r = 0; r < R; ++r) p0[r] = a[r];
            continue;
        }
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = p0[r] + a[r];
        if (!(i & 2u)) {
#pragma unroll
            for (int r = 0; r < R; ++r) p1[r] = a[r];
            continue;
        }
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = p1[r] + a[r];
        if (!(i & 4u)) {
#pragma unroll
            for (int r = 0; r < R; ++r) p2[r] = a[r];
            continue;
        }
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = p2[r] + a[r];
        if (!(i & 8u)) {
#pragma unroll
            for (int r = 0; r < R; ++r) p3[r] = a[r];
            continue;
        }
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = p3[r] + a[r];
        if (!(i & 16u)) {
#pragma unroll
            for (int r = 0; r < R; ++r) p4[r] = a[r];
            continue;
        }
#pragma unroll
        for (int r = 0; r < R; ++r) sum[r] = p4[r] + a[r];
    }
}

// The same grouping done by ONE warp from its own staged vector: ids[0..len) ascending node ids of the
// list, their values read from xs (the warp's dense input image, element j at xs_index<BF16>(j, nchunks)).
// S.segcnt / S.segstart / S.ent are the warp's own.  Ends with __syncwarp().
template <bool BF16>
__device__ __forceinline__ void cols_stage_warp(const cols_stage &S, const uint16_t *ids, uint32_t len, const float *xs,
                                                uint32_t nchunks, uint32_t lane)
{
    constexpr uint32_t V = BF16 ? 8u : 4u;
    S.segcnt[lane] = 0u;
    __syncwarp();
    // entries per segment; lists are ascending, so the order inside a segment is the list's order
    for (uint32_t i0 = 0; i0 < len; i0 += 32) {
        const uint32_t i = i0 + lane;
        const uint32_t id = i < len ? (uint32_t)ids[i] : 0u;
        const float v = i < len ? xs[xs_index<BF16>(id, nchunks)] : 0.0f;
        const uint32_t p = (id / V) & 31u;
        const uint32_t same = __match_any_sync(SLONN_FULL_MASK, v != 0.0f ? p : 32u + lane);
        if (v != 0.0f && (uint32_t)(__ffs(same) - 1) == lane) S.segcnt[p] += __popc(same);
        __syncwarp();
    }
    {
        const uint32_t c = (S.segcnt[lane] + 3u) & ~3u;
        uint32_t incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(SLONN_FULL_MASK, incl, off);
            if (lane >= (uint32_t)off) incl += t;
        }
        S.segstart[lane] = incl - c;
        if (lane == 31) S.segstart[32] = incl;
        S.segcnt[lane] = 0u; // reused as the fill level while placing
    }
    __syncwarp();
    for (uint32_t i0 = 0; i0 < len; i0 += 32) {
        const uint32_t i = i0 + lane;
        const uint32_t id = i < len ? (uint32_t)ids[i] : 0u;
        const float v = i < len ? xs[xs_index<BF16>(id, nchunks)] : 0.0f;
        const uint32_t p = (id / V) & 31u;
        const uint32_t same = __match_any_sync(SLONN_FULL_MASK, v != 0.0f ? p : 32u + lane);
        if (v != 0.0f) S.ent[S.segstart[p] + S.segcnt[p] + __popc(same & ((1u << lane) - 1u))] = make_uint2(id, __float_as_uint(v));
        __syncwarp();
        if (v != 0.0f && (uint32_t)(__ffs(same) - 1) == lane) S.segcnt[p] += __popc(same);
        __syncwarp();
    }
    { // fill every segment up to a multiple of 4 with copies of its last input carrying the value 0
        const uint32_t at = S.segstart[lane] + S.segcnt[lane], end = S.segstart[lane + 1];
        for (uint32_t k = at; k < end; ++k) S.ent[k] = make_uint2(S.ent[at - 1].x, 0u);
    }
    __syncwarp();
}
