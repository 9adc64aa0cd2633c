// Shared declarations of the SLO-NN library: the model object, launch parameter
// blocks and the fixed-order warp dot product that every kernel uses.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <mutex>
#include <unordered_map>

#include "../../include/slonn.h"

#define SLONN_FULL_MASK 0xffffffffu
#define SLONN_MAGIC 0x534c4f4eu /* "SLON" */

// ---- model -----------------------------------------------------------------

struct slonn_layer {
    const void *W;        // caller-owned, row-major [N][D]
    const float *bias;    // caller-owned [N]
    uint32_t D, N;
    uint32_t has_act;
    uint32_t cap;         // entries per bucket list
    uint32_t id_bytes;    // 2 or 4
    void *tables;         // library-owned [L][2^K][cap] ids
    uint64_t table_bytes;
    uint32_t *hash_nodes; // library-owned device copy, [L*K]
    void *WT;             // library-owned transposed copy [D][N]: layer 0 fed by CSR rows, and layers whose
                          // input is an activator layer's list (node axis in colpos order when colpos != NULL)
    uint32_t *colpos;     // library-owned [N]: node id -> column of WT; NULL = identity
    void *WH;             // library-owned [D][32]: the hash rows side by side (list-input activator layers)
};

struct slonn_model {
    uint32_t magic;
    int device;
    uint32_t n_layers;
    uint32_t dims[SLONN_MAX_LAYERS + 1];
    int32_t dtype;
    uint32_t K, L, H;
    uint32_t list_cap;
    uint32_t first_sparse;
    uint32_t free_hash;   // 1: hash nodes always active and absent from the lists
    uint32_t n_act;
    uint32_t act_index[SLONN_MAX_LAYERS]; // index of the layer among activator layers
    slonn_layer layer[SLONN_MAX_LAYERS];
    uint32_t hash_nodes_host[SLONN_MAX_LAYERS][128];
};

// ---- helpers ---------------------------------------------------------------

// k% -> node count: nearest whole node, at least one (budget in basis points).
__host__ __device__ __forceinline__ uint32_t slonn_budget_nodes(uint32_t bp, uint32_t N)
{
    uint64_t b = ((uint64_t)bp * N + 5000u) / 10000u;
    if (b < 1) b = 1;
    if (b > N) b = N;
    return (uint32_t)b;
}

// Nodes a layer of N nodes computes at budget bp.  pre = 0: the budget's node count.  pre = K*L
// (models whose hash nodes are always active): that many nodes from the lists, of which there are
// N - pre, plus the pre hash nodes.
__host__ __device__ __forceinline__ uint32_t slonn_layer_nodes(uint32_t bp, uint32_t N, uint32_t pre)
{
    const uint32_t B = slonn_budget_nodes(bp, N);
    if (pre == 0) return B;
    const uint32_t rest = N - pre;
    return (B < rest ? B : rest) + pre;
}

__device__ __forceinline__ void slonn_report(uint32_t *status, int code, uint32_t q, uint32_t layer)
{
    if (atomicCAS(status, 0u, (uint32_t)(-code)) == 0u) {
        status[1] = q;
        status[2] = layer;
    }
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Element e (compile-time) of a 16-byte weight chunk, widened to fp32.
template <bool BF16, int E>
__device__ __forceinline__ float chunk_elem(const uint4 &w)
{
    if (BF16) {
        const uint32_t u = (E >> 1) == 0 ? w.x : (E >> 1) == 1 ? w.y : (E >> 1) == 2 ? w.z : w.w;
        return (E & 1) ? bf16_hi(u) : bf16_lo(u);
    }
    return __uint_as_float(E == 0 ? w.x : E == 1 ? w.y : E == 2 ? w.z : w.w);
}

// acc[r] = fmaf(w[r][E], x[E], acc[r]) for every row, elements in ascending order; rows are
// interleaved so that consecutive instructions belong to independent accumulation chains.
template <bool BF16, int R, int E, int VPC>
struct chunk_fma {
    __device__ static __forceinline__ void run(const uint4 (&w)[R], const float *x, float (&acc)[R])
    {
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = fmaf(chunk_elem<BF16, E>(w[r]), x[E], acc[r]);
        chunk_fma<BF16, R, E + 1, VPC>::run(w, x, acc);
    }
};
template <bool BF16, int R, int VPC>
struct chunk_fma<BF16, R, VPC, VPC> {
    __device__ static __forceinline__ void run(const uint4 (&)[R], const float *, float (&)[R]) {}
};

// Sums of 4 rows' 32 partials with 6 shuffles instead of 20.  Same additions as the xor
// butterfly 16, 8, 4, 2, 1 of each row (each step adds the same two operands), but after
// stride 16 a lane only carries two of the rows and after stride 8 one.  Returns the sum of
// row (lane >> 3); the 8 lanes of a group hold the same value.
__device__ __forceinline__ float reduce_rows4(const float (&a)[4], uint32_t lane)
{
    const bool hi16 = (lane & 16u) != 0u;
    float k0 = hi16 ? a[2] : a[0], k1 = hi16 ? a[3] : a[1];
    const float s0 = hi16 ? a[0] : a[2], s1 = hi16 ? a[1] : a[3];
    k0 = k0 + __shfl_xor_sync(SLONN_FULL_MASK, s0, 16);
    k1 = k1 + __shfl_xor_sync(SLONN_FULL_MASK, s1, 16);
    const bool hi8 = (lane & 8u) != 0u;
    float k = hi8 ? k1 : k0;
    const float s = hi8 ? k0 : k1;
    k = k + __shfl_xor_sync(SLONN_FULL_MASK, s, 8);
    k = k + __shfl_xor_sync(SLONN_FULL_MASK, k, 4);
    k = k + __shfl_xor_sync(SLONN_FULL_MASK, k, 2);
    k = k + __shfl_xor_sync(SLONN_FULL_MASK, k, 1);
    return k;
}

// The same for 8 rows with 9 shuffles: after stride 16 a lane carries four of the rows, after
// stride 8 two, after stride 4 one.  Returns the sum of row (lane >> 2); the 4 lanes of a group
// hold the same value.
__device__ __forceinline__ float reduce_rows8(const float (&a)[8], uint32_t lane)
{
    const bool hi16 = (lane & 16u) != 0u;
    float k[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float keep = hi16 ? a[4 + i] : a[i];
        const float send = hi16 ? a[i] : a[4 + i];
        k[i] = keep + __shfl_xor_sync(SLONN_FULL_MASK, send, 16);
    }
    const bool hi8 = (lane & 8u) != 0u;
    float m[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float keep = hi8 ? k[2 + i] : k[i];
        const float send = hi8 ? k[i] : k[2 + i];
        m[i] = keep + __shfl_xor_sync(SLONN_FULL_MASK, send, 8);
    }
    const bool hi4 = (lane & 4u) != 0u;
    float v = hi4 ? m[1] : m[0];
    const float s4 = hi4 ? m[0] : m[1];
    v = v + __shfl_xor_sync(SLONN_FULL_MASK, s4, 4);
    v = v + __shfl_xor_sync(SLONN_FULL_MASK, v, 2);
    v = v + __shfl_xor_sync(SLONN_FULL_MASK, v, 1);
    return v;
}

// Where input element j lives in the staged copy of a query's input vector.
// fp32 weights: plain order.  bf16 weights: a 16-byte weight chunk holds 8
// elements, so the 8 matching inputs are split into two float4 planes (first
// four in plane 0, last four in plane 1) to keep 128-bit shared loads
// conflict-free.
template <bool BF16>
__device__ __forceinline__ uint32_t xs_index(uint32_t j, uint32_t nchunks)
{
    if (BF16) return (((j >> 2) & 1u) * nchunks + (j >> 3)) * 4u + (j & 3u);
    return j;
}

// Fixed-order partial sums of R weight rows with the staged input, one warp.
// Lane p owns partial sum p: it takes 16-byte chunks p, p+32, ... of each row
// and accumulates their elements in ascending order with fused multiply-adds
// (rows interleaved, so neighbouring instructions are independent).  The caller
// adds the 32 partials of each row in the order 16, 8, 4, 2, 1 (reduce_rows4)
// and then the bias.
template <bool BF16, int R>
__device__ __forceinline__ void warp_dot_rows(const uint4 *const (&rows)[R], const float4 *xs4,
                                              uint32_t nchunks, uint32_t lane, float (&acc)[R])
{
    constexpr int VPC = BF16 ? 8 : 4;
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0f;
#pragma unroll 2
    for (uint32_t c = lane; c < nchunks; c += 32) {
        uint4 w[R];
#pragma unroll
        for (int r = 0; r < R; ++r) w[r] = __ldg(rows[r] + c);
        float x[VPC];
        const float4 xa = xs4[c];
        x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w;
        if (BF16) {
            const float4 xb = xs4[nchunks + c];
            x[VPC - 4] = xb.x; x[VPC - 3] = xb.y; x[VPC - 2] = xb.z; x[VPC - 1] = xb.w;
        }
        chunk_fma<BF16, R, 0, VPC>::run(w, x, acc);
    }
}

// Fixed-order dot product of ONE weight row, for launches where latency matters more than
// throughput (a handful of queries): up to DEPTH of the lane's 16-byte chunks are in flight at once
// (chunks of this lane loaded before the first one is used).  Same chunk-to-lane assignment, same
// order within a lane, xor butterfly 16, 8, 4, 2, 1; every lane returns the sum (bias not included).
template <bool BF16, int DEPTH = 8>
__device__ __forceinline__ float warp_dot_row1(const uint4 *row, const float4 *xs4, uint32_t nchunks, uint32_t lane)
{
    constexpr int VPC = BF16 ? 8 : 4;
    float acc[1] = {0.0f};
    for (uint32_t c0 = lane; c0 < nchunks; c0 += 32 * DEPTH) {
        uint4 w[DEPTH][1];
#pragma unroll
        for (int i = 0; i < DEPTH; ++i)
            if (c0 + 32 * i < nchunks) w[i][0] = __ldg(row + c0 + 32 * i);
#pragma unroll
        for (int i = 0; i < DEPTH; ++i) {
            const uint32_t c = c0 + 32 * i;
            if (c < nchunks) {
                float x[VPC];
                const float4 xa = xs4[c];
                x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w;
                if (BF16) {
                    const float4 xb = xs4[nchunks + c];
                    x[VPC - 4] = xb.x; x[VPC - 3] = xb.y; x[VPC - 2] = xb.z; x[VPC - 1] = xb.w;
                }
                chunk_fma<BF16, 1, 0, VPC>::run(w[i], x, acc);
            }
        }
    }
    float a = acc[0];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) a = a + __shfl_xor_sync(SLONN_FULL_MASK, a, off);
    return a;
}

// ---- layer input descriptor --------------------------------------------------

enum { SLONN_IN_DENSE = 0, SLONN_IN_LIST = 1 };

struct slonn_input {
    int kind;
    const float *dense;     // DENSE: [n][D]
    const uint64_t *indptr; // LIST: segment (q * ip_mul + ip_add) of ids / vals
    const uint32_t *ids;
    const float *vals;
    uint32_t ip_mul, ip_add;
};

// Stages query q's input vector (D floats) into shared memory in xs_index order.
// Must be called by the whole block; ends with a barrier.
template <bool BF16>
__device__ __forceinline__ void stage_input(const slonn_input &in, uint32_t q, uint32_t D,
                                            uint32_t nchunks, float4 *xs4)
{
    const uint32_t nvec = D >> 2;
    if (in.kind == SLONN_IN_DENSE) {
        const float4 *src = reinterpret_cast<const float4 *>(in.dense + (uint64_t)q * D);
#pragma unroll 4
        for (uint32_t i = threadIdx.x; i < nvec; i += blockDim.x) {
            const float4 v = __ldg(src + i);
            if (BF16) xs4[(i & 1u) * nchunks + (i >> 1)] = v;
            else xs4[i] = v;
        }
    } else {
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t i = threadIdx.x; i < nvec; i += blockDim.x) xs4[i] = z;
        __syncthreads();
        const uint64_t s0 = in.indptr[(uint64_t)q * in.ip_mul + in.ip_add];
        const uint32_t len = (uint32_t)(in.indptr[(uint64_t)q * in.ip_mul + in.ip_add + 1] - s0);
        float *xs = reinterpret_cast<float *>(xs4);
#pragma unroll 4
        for (uint32_t i = threadIdx.x; i < len; i += blockDim.x) {
            const uint32_t j = in.ids[s0 + i];
            if (j < D) xs[xs_index<BF16>(j, nchunks)] = in.vals[s0 + i];
        }
    }
    __syncthreads();
}

// hash nodes that are active whatever the budget (0 unless the model was built that way)
// Lets `kernel` be launched with `bytes` of dynamic shared memory on the current device.  The 48 KB a launch gets
// without opting in and the 227 KB a block can have both count the kernel's static shared memory (at most 1120
// bytes in this library): the opt-in starts at 46 KB and ends at 225 KB (SLONN_ERR_DIM above).  The limit of a
// kernel is only ever raised, so that two host threads launching the same kernel with different sizes cannot
// take each other's allowance away between the opt-in and the launch.
inline int slonn_allow_smem(const void *kernel, size_t bytes)
{
    if (bytes <= 46 * 1024) return SLONN_OK;
    if (bytes > 225 * 1024) return SLONN_ERR_DIM;
    static std::mutex mu;
    static std::unordered_map<uint64_t, size_t> allowed; // (kernel, device) -> bytes opted in to so far
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLONN_ERR_CUDA;
    const uint64_t key = (uint64_t)reinterpret_cast<uintptr_t>(kernel) * 64u + (uint64_t)(dev & 63);
    std::lock_guard<std::mutex> lock(mu);
    size_t &have = allowed[key];
    if (bytes > have) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return SLONN_ERR_CUDA;
        have = bytes;
    }
    return SLONN_OK;
}

inline uint32_t slonn_model_pre(const slonn_model *m) { return m->free_hash ? m->H : 0u; }

// ---- internal host entry points shared between translation units ---------------
int slonn_forward_all_rows(const slonn_model *m, uint32_t l, const float *in_dense, uint32_t n, float *out,
                           uint32_t relu, cudaStream_t st);
int slonn_forward_sparse_first(const slonn_model *m, const uint64_t *indptr, const uint32_t *ids,
                               const float *vals, uint32_t n, float *out, uint32_t relu, uint32_t *status,
                               cudaStream_t st);
