// Node-Activator training on the device (Algorithm 1 of the paper, with the
// variance-proportional FreeHash sampling of Sec. 3.4), plus model lifetime.
//
// Per activator layer l, with A = the layer's complete activations on the
// calibration rows ([n_cal][N] fp32):
//   column_stats_kernel   per node: sum and population variance over the rows (fp64, row order)
//   (host)                K*L distinct hash nodes drawn in proportion to variance
//   row_keys_kernel       per row and table: key from the signs of the hash nodes' activations
//   bucket_*_kernel       rows grouped by key, row order kept inside a bucket
//   bucket_score_kernel   NodeScore[b][key][node] = sum of A over the bucket's rows (fp64, row order)
//   segment_sort_kernel   node ids ordered by score, highest first, equal scores by lower id
//   fill_tables_kernel    lists copied into the table; buckets no row reached get the global ranking
// fp64 sums use explicit add/multiply intrinsics so that no multiply-add is fused.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>

#include "slonn_common.cuh"

namespace {

#define CK(call)                                         \
    do {                                                 \
        if ((call) != cudaSuccess) { rc = SLONN_ERR_CUDA; goto fail; } \
    } while (0)

// ---------------------------------------------------------------------------
__global__ void transpose_kernel(const void *W, void *WT, uint32_t N, uint32_t D, uint32_t esz)
{
    // WT[d][n] = W[n][d]; plain tiled transpose through shared memory
    __shared__ uint32_t tile[32][33];
    const uint32_t d0 = blockIdx.x * 32, n0 = blockIdx.y * 32;
    for (uint32_t i = threadIdx.y; i < 32; i += blockDim.y) {
        const uint32_t n = n0 + i, d = d0 + threadIdx.x;
        uint32_t v = 0;
        if (n < N && d < D)
            v = esz == 2 ? (uint32_t)reinterpret_cast<const uint16_t *>(W)[(uint64_t)n * D + d]
                         : reinterpret_cast<const uint32_t *>(W)[(uint64_t)n * D + d];
        tile[i][threadIdx.x] = v;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.y; i < 32; i += blockDim.y) {
        const uint32_t d = d0 + i, n = n0 + threadIdx.x;
        if (n < N && d < D) {
            const uint32_t v = tile[threadIdx.x][i];
            if (esz == 2) reinterpret_cast<uint16_t *>(WT)[(uint64_t)d * N + n] = (uint16_t)v;
            else reinterpret_cast<uint32_t *>(WT)[(uint64_t)d * N + n] = v;
        }
    }
}

// WT[d][colpos[n]] = W[n][d]: transposed copy with the node axis re-ordered
__global__ void transpose_permuted_kernel(const void *W, void *WT, uint32_t N, uint32_t D, uint32_t esz,
                                          const uint32_t *colpos)
{
    __shared__ uint32_t tile[32][33];
    const uint32_t d0 = blockIdx.x * 32, n0 = blockIdx.y * 32;
    for (uint32_t i = threadIdx.y; i < 32; i += blockDim.y) {
        const uint32_t n = n0 + i, d = d0 + threadIdx.x;
        uint32_t v = 0;
        if (n < N && d < D)
            v = esz == 2 ? (uint32_t)reinterpret_cast<const uint16_t *>(W)[(uint64_t)n * D + d]
                         : reinterpret_cast<const uint32_t *>(W)[(uint64_t)n * D + d];
        tile[i][threadIdx.x] = v;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.y; i < 32; i += blockDim.y) {
        const uint32_t d = d0 + i, n = n0 + threadIdx.x;
        if (n < N && d < D) {
            const uint32_t v = tile[threadIdx.x][i];
            const uint64_t at = (uint64_t)d * N + colpos[n];
            if (esz == 2) reinterpret_cast<uint16_t *>(WT)[at] = (uint16_t)v;
            else reinterpret_cast<uint32_t *>(WT)[at] = v;
        }
    }
}

// WH[d][h] = W[hash_nodes[h]][d] for h < H, zero for H <= h < 32: the layer's hash rows side by side,
// so that one input d needs one 64- or 128-byte line for all hash functions
__global__ void hash_matrix_kernel(const void *W, void *WH, uint32_t D, uint32_t esz, const uint32_t *hash_nodes,
                                   uint32_t H)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t d = t >> 5, h = t & 31u;
    if (d >= D) return;
    uint32_t v = 0;
    if (h < H) {
        const uint64_t at = (uint64_t)hash_nodes[h] * D + d;
        v = esz == 2 ? (uint32_t)reinterpret_cast<const uint16_t *>(W)[at] : reinterpret_cast<const uint32_t *>(W)[at];
    }
    if (esz == 2) reinterpret_cast<uint16_t *>(WH)[t] = (uint16_t)v;
    else reinterpret_cast<uint32_t *>(WH)[t] = v;
}

// How early each node appears in the layer's ranked lists: score[n] = sum over all lists of
// max(0, T - rank of n in the list).  Integer sums, so the result does not depend on thread order.
template <typename IDT>
__global__ void popularity_kernel(const IDT *tables, uint64_t n_lists, uint32_t cap, uint32_t T, uint32_t N,
                                  unsigned long long *score)
{
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t list = t / T;
    const uint32_t r = (uint32_t)(t - list * T);
    if (list >= n_lists) return;
    const uint32_t id = (uint32_t)tables[list * cap + r];
    if (id < N) atomicAdd(score + id, (unsigned long long)(T - r));
}

// Library-owned copies for the input-stationary kernels (layers whose input is the (id, value) list of
// an activator layer below them):
//   WT      transposed weights [D][N]; on a layer that has its own activator the node axis is stored in
//           the order of `colpos`: nodes that sit early in many ranked lists first, so that the nodes a
//           query selects lie close together in every row of WT
//   colpos  [N] node id -> column of WT (activator layers only; NULL = identity)
//   WH      [D][32] the layer's hash rows side by side (activator layers with K*L <= 32)
// and the plain transposed copy of a first layer fed by CSR rows.  phase 0: the CSR first layer (needed
// by the calibration pass); phase 1: the rest (needs the finished tables).
// Copies of 4 GiB or more are left out: the kernels address them with 32-bit byte offsets (such layers keep the row kernels).
int make_transposed_copies(slonn_model *m, cudaStream_t st, int phase)
{
    const uint32_t esz = m->dtype == SLONN_BF16 ? 2u : 4u;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        slonn_layer &ly = m->layer[l];
        const bool csr_first = (l == 0 && m->first_sparse);
        const bool list_input = (l > 0 && m->layer[l - 1].has_act && (uint64_t)ly.N * ly.D * esz < (1ull << 32));
        if (phase == 0 ? !csr_first : !list_input) continue;
        if (cudaMalloc(&ly.WT, (uint64_t)ly.N * ly.D * esz) != cudaSuccess) return SLONN_ERR_NOMEM;
        const dim3 grid((ly.D + 31) / 32, (ly.N + 31) / 32), block(32, 8);
        if (!ly.has_act || csr_first) {
            transpose_kernel<<<grid, block, 0, st>>>(ly.W, ly.WT, ly.N, ly.D, esz);
            if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
            continue;
        }
        // order of the node axis: by popularity in the lists, equal scores by lower id
        const uint64_t n_lists = (uint64_t)m->L << m->K;
        const uint32_t T = std::max(1u, std::min(ly.cap, (ly.N + 7u) / 8u));
        unsigned long long *d_score = nullptr;
        if (cudaMalloc(&d_score, sizeof(unsigned long long) * ly.N) != cudaSuccess) return SLONN_ERR_NOMEM;
        std::vector<unsigned long long> score(ly.N);
        std::vector<uint32_t> order(ly.N), colpos(ly.N);
        bool ok = cudaMemsetAsync(d_score, 0, sizeof(unsigned long long) * ly.N, st) == cudaSuccess;
        if (ok) {
            const uint64_t threads = n_lists * T;
            const uint32_t blocks = (uint32_t)((threads + 255) / 256);
            if (ly.id_bytes == 2)
                popularity_kernel<uint16_t><<<blocks, 256, 0, st>>>((const uint16_t *)ly.tables, n_lists, ly.cap, T, ly.N, d_score);
            else
                popularity_kernel<uint32_t><<<blocks, 256, 0, st>>>((const uint32_t *)ly.tables, n_lists, ly.cap, T, ly.N, d_score);
            ok = cudaGetLastError() == cudaSuccess &&
                 cudaMemcpyAsync(score.data(), d_score, sizeof(unsigned long long) * ly.N, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
                 cudaStreamSynchronize(st) == cudaSuccess;
        }
        cudaFree(d_score);
        if (!ok) return SLONN_ERR_CUDA;
        for (uint32_t i = 0; i < ly.N; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return score[a] > score[b]; });
        for (uint32_t i = 0; i < ly.N; ++i) colpos[order[i]] = i;
        if (cudaMalloc(&ly.colpos, sizeof(uint32_t) * ly.N) != cudaSuccess) return SLONN_ERR_NOMEM;
        if (cudaMemcpyAsync(ly.colpos, colpos.data(), sizeof(uint32_t) * ly.N, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SLONN_ERR_CUDA;
        transpose_permuted_kernel<<<grid, block, 0, st>>>(ly.W, ly.WT, ly.N, ly.D, esz, ly.colpos);
        if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
        if (m->H <= 32) {
            if (cudaMalloc(&ly.WH, (uint64_t)ly.D * 32 * esz) != cudaSuccess) return SLONN_ERR_NOMEM;
            hash_matrix_kernel<<<(ly.D * 32 + 255) / 256, 256, 0, st>>>(ly.W, ly.WH, ly.D, esz, ly.hash_nodes, m->H);
            if (cudaGetLastError() != cudaSuccess) return SLONN_ERR_CUDA;
        }
        if (cudaStreamSynchronize(st) != cudaSuccess) return SLONN_ERR_CUDA; // colpos.data() is read by the copy above
    }
    return SLONN_OK;
}

// sum[i] = sum over rows of A[x][i]; var[i] = mean of (A[x][i] - mean_i)^2.  One thread per node.
__global__ void column_stats_kernel(const float *A, uint32_t n_rows, uint32_t N, double *sum, double *var)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    double s = 0.0;
    for (uint32_t x = 0; x < n_rows; ++x) s = __dadd_rn(s, (double)A[(uint64_t)x * N + i]);
    const double mean = __ddiv_rn(s, (double)n_rows);
    double v = 0.0;
    for (uint32_t x = 0; x < n_rows; ++x) {
        const double d = __dsub_rn((double)A[(uint64_t)x * N + i], mean);
        v = __dadd_rn(v, __dmul_rn(d, d));
    }
    sum[i] = s;
    var[i] = __ddiv_rn(v, (double)n_rows);
}

// keys[b][x]: bit j = [activation of hash node (b, j) on row x > 0]
__global__ void row_keys_kernel(const float *A, uint32_t n_rows, uint32_t N, const uint32_t *hash_nodes,
                                uint32_t K, uint32_t L, uint32_t *keys)
{
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (uint64_t)n_rows * L) return;
    const uint32_t b = (uint32_t)(t / n_rows), x = (uint32_t)(t % n_rows);
    uint32_t key = 0;
    for (uint32_t j = 0; j < K; ++j)
        if (A[(uint64_t)x * N + hash_nodes[b * K + j]] > 0.0f) key |= (1u << j);
    keys[(uint64_t)b * n_rows + x] = key;
}

// One thread per (table, key): how many rows carry that key.
__global__ void bucket_count_kernel(const uint32_t *keys, uint32_t n_rows, uint32_t nb, uint32_t L,
                                    uint32_t *count)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nb * L) return;
    const uint32_t b = t / nb, key = t % nb;
    uint32_t c = 0;
    for (uint32_t x = 0; x < n_rows; ++x) c += (keys[(uint64_t)b * n_rows + x] == key) ? 1u : 0u;
    count[t] = c;
}

// start[t] = exclusive prefix of count within a table (one block per table).
__global__ void bucket_start_kernel(const uint32_t *count, uint32_t nb, uint32_t *start)
{
    __shared__ uint32_t carry;
    const uint32_t b = blockIdx.x;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (uint32_t base = 0; base < nb; base += blockDim.x) {
        // serial within the block is enough: nb <= 65536, build time only
        if (threadIdx.x == 0) {
            uint32_t run = carry;
            const uint32_t end = min(nb, base + blockDim.x);
            for (uint32_t k = base; k < end; ++k) {
                start[b * nb + k] = run;
                run += count[b * nb + k];
            }
            carry = run;
        }
        __syncthreads();
    }
}

// One thread per (table, key): the rows of that bucket, in row order.
__global__ void bucket_fill_kernel(const uint32_t *keys, uint32_t n_rows, uint32_t nb, uint32_t L,
                                   const uint32_t *start, uint32_t *members)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nb * L) return;
    const uint32_t b = t / nb, key = t % nb;
    uint32_t o = start[t];
    for (uint32_t x = 0; x < n_rows; ++x)
        if (keys[(uint64_t)b * n_rows + x] == key) members[(uint64_t)b * n_rows + o++] = x;
}

// score[bk][i] = sum over the bucket's rows (row order) of A[x][i], fp64.
__global__ void bucket_score_kernel(const float *A, uint32_t n_rows, uint32_t N, uint32_t nb,
                                    const uint32_t *start, const uint32_t *count, const uint32_t *members,
                                    uint32_t bk0, double *score /* [segments in this pass][N] */)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t bk = bk0 + blockIdx.y;
    if (i >= N) return;
    const uint32_t b = bk / nb;
    const uint32_t *mem = members + (uint64_t)b * n_rows + start[bk];
    const uint32_t c = count[bk];
    double s = 0.0;
    for (uint32_t k = 0; k < c; ++k) s = __dadd_rn(s, (double)A[(uint64_t)mem[k] * N + i]);
    score[(uint64_t)blockIdx.y * N + i] = s;
}

// Sort key: ascending unsigned order == descending score; zeros of either sign are equal.
__device__ __forceinline__ uint64_t score_sort_key(double s)
{
    if (s == 0.0) s = 0.0;
    uint64_t u = (uint64_t)__double_as_longlong(s);
    u = (u >> 63) ? ~u : (u | 0x8000000000000000ull); // ascending-order image
    return ~u;                                          // descending
}

// One block per segment: stable LSD radix sort (8 bits per pass) of the segment's
// N (key, id) pairs; ids start ascending, so equal scores keep the lower id first.
// seg_active[s] == 0 skips the segment.  The sorted ids end in ids_out[s][0..N).
// The n_last ids in `last` (nullable) get the largest key, which no score maps to, so they end
// behind every other id without changing the order of the others.
#define SORT_THREADS 256
__global__ void __launch_bounds__(SORT_THREADS)
segment_sort_kernel(const double *score, uint32_t N, const uint32_t *seg_active, uint64_t *keyA, uint64_t *keyB,
                    uint32_t *idA, uint32_t *idB, uint32_t *ids_out, const uint32_t *last, uint32_t n_last)
{
    __shared__ uint32_t hist[256];
    __shared__ uint32_t bin_base[256];
    __shared__ uint32_t warp_cnt[SORT_THREADS / 32][256];
    __shared__ uint32_t warp_off[SORT_THREADS / 32][256];
    __shared__ uint32_t s_skip;
    const uint32_t seg = blockIdx.x;
    if (seg_active && !seg_active[seg]) return;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint64_t *ka = keyA + (uint64_t)seg * N, *kb = keyB + (uint64_t)seg * N;
    uint32_t *ia = idA + (uint64_t)seg * N, *ib = idB + (uint64_t)seg * N;
    const double *sc = score + (uint64_t)seg * N;
    for (uint32_t i = threadIdx.x; i < N; i += blockDim.x) {
        ka[i] = score_sort_key(sc[i]);
        ia[i] = i;
    }
    for (uint32_t d = threadIdx.x; d < 256; d += blockDim.x)
        for (uint32_t w = 0; w < SORT_THREADS / 32; ++w) warp_cnt[w][d] = 0;
    __syncthreads();
    if (last) {
        for (uint32_t h = threadIdx.x; h < n_last; h += blockDim.x) ka[last[h]] = ~0ull;
        __syncthreads();
    }
    for (uint32_t pass = 0; pass < 8; ++pass) {
        const uint32_t shift = pass * 8;
        for (uint32_t d = threadIdx.x; d < 256; d += blockDim.x) hist[d] = 0;
        if (threadIdx.x == 0) s_skip = 0;
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < N; i += blockDim.x)
            atomicAdd(&hist[(uint32_t)(ka[i] >> shift) & 255u], 1u);
        __syncthreads();
        if (threadIdx.x < 256 && hist[threadIdx.x] == N) s_skip = 1; // every key shares this digit
        __syncthreads();
        if (s_skip) { __syncthreads(); continue; }
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (uint32_t d = 0; d < 256; ++d) { bin_base[d] = run; run += hist[d]; }
        }
        __syncthreads();
        for (uint32_t base = 0; base < N; base += blockDim.x) {
            const uint32_t i = base + threadIdx.x;
            const bool valid = i < N;
            uint64_t key = 0;
            uint32_t id = 0, digit = 0x100u + lane; // distinct dummies for lanes past the end
            if (valid) { key = ka[i]; id = ia[i]; digit = (uint32_t)(key >> shift) & 255u; }
            const uint32_t peers = __match_any_sync(SLONN_FULL_MASK, digit);
            const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
            const bool leader = valid && rank == 0;
            if (leader) warp_cnt[warp][digit] = __popc(peers);
            __syncthreads();
            if (threadIdx.x < 256) {
                const uint32_t d = threadIdx.x;
                uint32_t run = bin_base[d];
                for (uint32_t w = 0; w < SORT_THREADS / 32; ++w) {
                    warp_off[w][d] = run;
                    run += warp_cnt[w][d];
                }
                bin_base[d] = run;
            }
            __syncthreads();
            if (valid) {
                const uint32_t dst = warp_off[warp][digit] + rank;
                kb[dst] = key;
                ib[dst] = id;
            }
            if (leader) warp_cnt[warp][digit] = 0;
            __syncthreads();
        }
        uint64_t *tk = ka; ka = kb; kb = tk;
        uint32_t *ti = ia; ia = ib; ib = ti;
        __syncthreads();
    }
    uint32_t *out = ids_out + (uint64_t)seg * N;
    for (uint32_t i = threadIdx.x; i < N; i += blockDim.x) out[i] = ia[i];
}

// tables[bk][0..cap) = the bucket's sorted ids, or the global ranking for a bucket no row reached.
template <typename IDT>
__global__ void fill_tables_kernel(const uint32_t *sorted /* [segs][N] */, const uint32_t *global_sorted,
                                   const uint32_t *count, uint32_t bk0, uint32_t N, uint32_t cap, IDT *tables)
{
    const uint32_t bk = bk0 + blockIdx.y;
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= cap) return;
    const uint32_t *src = count[bk] ? sorted + (uint64_t)blockIdx.y * N : global_sorted;
    tables[(uint64_t)bk * cap + r] = (IDT)src[r];
}

// ---------------------------------------------------------------------------
// host: hash-node sampling (Sec. 3.4: probability proportional to activation variance).
// The not-yet-drawn nodes are kept as a dense array in id order together with the running
// sums of their variances; a draw is a search in those running sums and removes its node.
// The running sums are rebuilt front to back after every removal, so a draw sees exactly
// the left-to-right fp64 sums of the remaining variances.  Uniform numbers come from a
// SplitMix64 stream (53 bits each).  When the remaining variances sum to zero the draw is
// uniform over the remaining nodes.
// ---------------------------------------------------------------------------
class splitmix_stream {
public:
    explicit splitmix_stream(uint64_t seed) : state_(seed) {}
    double uniform53()
    {
        uint64_t z = (state_ += 0x9E3779B97F4A7C15ull);
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return (double)((z ^ (z >> 31)) >> 11) * 0x1.0p-53;
    }
private:
    uint64_t state_;
};

void sample_hash_nodes(const std::vector<double> &var, uint32_t H, uint64_t seed, uint32_t layer, uint32_t *out)
{
    std::vector<uint32_t> pool(var.size()); // ids still available, ascending
    std::iota(pool.begin(), pool.end(), 0u);
    std::vector<double> running(var.size()); // running[k] = var[pool[0]] + ... + var[pool[k]]
    splitmix_stream rng(seed ^ (0xD6E8FEB86659FD93ull * (uint64_t)(layer + 1)));
    for (uint32_t d = 0; d < H; ++d) {
        const double u = rng.uniform53();
        double s = 0.0;
        for (size_t k = 0; k < pool.size(); ++k) running[k] = (s += var[pool[k]]);
        const auto first = running.begin(), last = running.begin() + pool.size();
        size_t k;
        if (s > 0.0) {
            // first node whose running sum exceeds u * total (its own variance is then positive); if rounding
            // leaves none, the last node with a positive variance
            k = (size_t)(std::upper_bound(first, last, u * s) - first);
            if (k == pool.size())
                do { --k; } while (k > 0 && !(var[pool[k]] > 0.0));
        } else {
            k = std::min((size_t)(u * (double)pool.size()), pool.size() - 1);
        }
        out[d] = pool[k];
        pool.erase(pool.begin() + (std::ptrdiff_t)k);
    }
}

// ---------------------------------------------------------------------------
// tables of one layer from its complete calibration activations
// ---------------------------------------------------------------------------
int train_layer(slonn_model *m, uint32_t l, const float *A, uint32_t n_cal, uint64_t seed,
                const uint32_t *override_nodes, cudaStream_t st)
{
    slonn_layer &ly = m->layer[l];
    const uint32_t N = ly.N, K = m->K, L = m->L, H = m->H, nb = 1u << K, nseg = nb * L;
    int rc = SLONN_OK;
    double *d_sum = nullptr, *d_var = nullptr, *d_score = nullptr;
    uint32_t *d_keys = nullptr, *d_count = nullptr, *d_start = nullptr, *d_members = nullptr;
    uint64_t *d_keyA = nullptr, *d_keyB = nullptr;
    uint32_t *d_idA = nullptr, *d_idB = nullptr, *d_sorted = nullptr, *d_gsorted = nullptr;
    std::vector<double> var(N);

    CK(cudaMalloc(&d_sum, sizeof(double) * N));
    CK(cudaMalloc(&d_var, sizeof(double) * N));
    column_stats_kernel<<<(N + 127) / 128, 128, 0, st>>>(A, n_cal, N, d_sum, d_var);
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(var.data(), d_var, sizeof(double) * N, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));

    if (override_nodes) {
        for (uint32_t h = 0; h < H; ++h) {
            if (override_nodes[h] >= N) { rc = SLONN_ERR_ARG; goto fail; }
            for (uint32_t g = 0; g < h; ++g)
                if (override_nodes[g] == override_nodes[h]) { rc = SLONN_ERR_ARG; goto fail; }
            m->hash_nodes_host[l][h] = override_nodes[h];
        }
    } else {
        sample_hash_nodes(var, H, seed, l, m->hash_nodes_host[l]);
    }
    CK(cudaMalloc(&ly.hash_nodes, sizeof(uint32_t) * H));
    CK(cudaMemcpyAsync(ly.hash_nodes, m->hash_nodes_host[l], sizeof(uint32_t) * H, cudaMemcpyHostToDevice, st));

    // rows -> buckets
    CK(cudaMalloc(&d_keys, sizeof(uint32_t) * (uint64_t)n_cal * L));
    CK(cudaMalloc(&d_members, sizeof(uint32_t) * (uint64_t)n_cal * L));
    CK(cudaMalloc(&d_count, sizeof(uint32_t) * nseg));
    CK(cudaMalloc(&d_start, sizeof(uint32_t) * nseg));
    {
        const uint64_t t = (uint64_t)n_cal * L;
        row_keys_kernel<<<(uint32_t)((t + 255) / 256), 256, 0, st>>>(A, n_cal, N, ly.hash_nodes, K, L, d_keys);
        CK(cudaGetLastError());
        bucket_count_kernel<<<(nseg + 127) / 128, 128, 0, st>>>(d_keys, n_cal, nb, L, d_count);
        CK(cudaGetLastError());
        bucket_start_kernel<<<L, 256, 0, st>>>(d_count, nb, d_start);
        CK(cudaGetLastError());
        bucket_fill_kernel<<<(nseg + 127) / 128, 128, 0, st>>>(d_keys, n_cal, nb, L, d_start, d_members);
        CK(cudaGetLastError());
    }

    // table storage
    // lists hold every node, or (hash nodes always active) every node that is not a hash node:
    // those are sorted behind all others below and fall off the end of the list
    {
        const uint32_t listable = m->free_hash ? N - H : N;
        ly.cap = (m->list_cap == 0 || m->list_cap > listable) ? listable : m->list_cap;
    }
    ly.id_bytes = N <= 65536u ? 2u : 4u;
    ly.table_bytes = (uint64_t)nseg * ly.cap * ly.id_bytes;
    CK(cudaMalloc(&ly.tables, ly.table_bytes));

    // global ranking (sum over all rows), used for buckets no row reached
    CK(cudaMalloc(&d_gsorted, sizeof(uint32_t) * N));
    {
        uint64_t *gkA = nullptr, *gkB = nullptr;
        uint32_t *giA = nullptr, *giB = nullptr;
        bool ok = cudaMalloc(&gkA, 8ull * N) == cudaSuccess && cudaMalloc(&gkB, 8ull * N) == cudaSuccess &&
                  cudaMalloc(&giA, 4ull * N) == cudaSuccess && cudaMalloc(&giB, 4ull * N) == cudaSuccess;
        if (ok) {
            segment_sort_kernel<<<1, SORT_THREADS, 0, st>>>(d_sum, N, nullptr, gkA, gkB, giA, giB, d_gsorted,
                                                            m->free_hash ? ly.hash_nodes : nullptr, H);
            ok = cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess;
        }
        cudaFree(gkA); cudaFree(gkB); cudaFree(giA); cudaFree(giB);
        if (!ok) { rc = SLONN_ERR_CUDA; goto fail; }
    }

    // buckets, a bounded number of segments at a time (36 bytes of scratch per node and segment)
    {
        uint64_t segs = (2ull << 30) / (36ull * N);
        segs = std::max<uint64_t>(1, std::min<uint64_t>(segs, nseg));
        const uint32_t S = (uint32_t)std::min<uint64_t>(segs, 65535);
        CK(cudaMalloc(&d_score, sizeof(double) * (uint64_t)S * N));
        CK(cudaMalloc(&d_keyA, 8ull * S * N));
        CK(cudaMalloc(&d_keyB, 8ull * S * N));
        CK(cudaMalloc(&d_idA, 4ull * S * N));
        CK(cudaMalloc(&d_idB, 4ull * S * N));
        CK(cudaMalloc(&d_sorted, 4ull * S * N));
        for (uint32_t bk0 = 0; bk0 < nseg; bk0 += S) {
            const uint32_t cnt = std::min(S, nseg - bk0);
            bucket_score_kernel<<<dim3((N + 255) / 256, cnt), 256, 0, st>>>(A, n_cal, N, nb, d_start, d_count,
                                                                            d_members, bk0, d_score);
            CK(cudaGetLastError());
            segment_sort_kernel<<<cnt, SORT_THREADS, 0, st>>>(d_score, N, d_count + bk0, d_keyA, d_keyB, d_idA,
                                                              d_idB, d_sorted, m->free_hash ? ly.hash_nodes : nullptr, H);
            CK(cudaGetLastError());
            const dim3 g((ly.cap + 255) / 256, cnt);
            if (ly.id_bytes == 2)
                fill_tables_kernel<uint16_t><<<g, 256, 0, st>>>(d_sorted, d_gsorted, d_count, bk0, N, ly.cap,
                                                                (uint16_t *)ly.tables);
            else
                fill_tables_kernel<uint32_t><<<g, 256, 0, st>>>(d_sorted, d_gsorted, d_count, bk0, N, ly.cap,
                                                                (uint32_t *)ly.tables);
            CK(cudaGetLastError());
        }
        CK(cudaStreamSynchronize(st));
    }
fail:
    cudaFree(d_sum); cudaFree(d_var); cudaFree(d_score); cudaFree(d_keys); cudaFree(d_count);
    cudaFree(d_start); cudaFree(d_members); cudaFree(d_keyA); cudaFree(d_keyB); cudaFree(d_idA);
    cudaFree(d_idB); cudaFree(d_sorted); cudaFree(d_gsorted);
    return rc;
}

} // namespace

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
extern "C" int slonn_version(void) { return SLONN_VERSION; }

extern "C" const char *slonn_strerror(int code)
{
    switch (code) {
    case SLONN_OK: return "ok";
    case SLONN_ERR_ARG: return "bad argument";
    case SLONN_ERR_DIM: return "bad dimension";
    case SLONN_ERR_DTYPE: return "unknown weight type";
    case SLONN_ERR_ALIGN: return "buffer or weight row not 16-byte aligned";
    case SLONN_ERR_BUDGET: return "budget out of range";
    case SLONN_ERR_NOMEM: return "out of memory";
    case SLONN_ERR_CUDA: return "CUDA runtime error";
    case SLONN_ERR_TIMEOUT: return "device-side wait timed out";
    case SLONN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    default: return "unknown error";
    }
}

extern "C" void slonn_free(slonn_model *m)
{
    if (!m || m->magic != SLONN_MAGIC) return;
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        cudaFree(m->layer[l].tables);
        cudaFree(m->layer[l].hash_nodes);
        cudaFree(m->layer[l].WT);
        cudaFree(m->layer[l].colpos);
        cudaFree(m->layer[l].WH);
    }
    m->magic = 0;
    delete m;
}

extern "C" int slonn_model_info(const slonn_model *m, uint32_t layer, uint32_t *hash_nodes,
                                const void **tables_dev, uint64_t *table_bytes, uint32_t *id_bytes, uint32_t *cap)
{
    if (!m || m->magic != SLONN_MAGIC || layer >= m->n_layers) return SLONN_ERR_ARG;
    const slonn_layer &ly = m->layer[layer];
    if (hash_nodes && ly.has_act) memcpy(hash_nodes, m->hash_nodes_host[layer], sizeof(uint32_t) * m->H);
    if (tables_dev) *tables_dev = ly.tables;
    if (table_bytes) *table_bytes = ly.table_bytes;
    if (id_bytes) *id_bytes = ly.id_bytes;
    if (cap) *cap = ly.cap;
    return SLONN_OK;
}

extern "C" int slonn_model_tables_to_host(const slonn_model *m, uint32_t layer, void *dst_host, uint64_t dst_bytes)
{
    if (!m || m->magic != SLONN_MAGIC || layer >= m->n_layers || !dst_host) return SLONN_ERR_ARG;
    const slonn_layer &ly = m->layer[layer];
    if (!ly.has_act || !ly.tables) return SLONN_ERR_ARG;
    if (dst_bytes < ly.table_bytes) return SLONN_ERR_WORKSPACE;
    return cudaMemcpy(dst_host, ly.tables, ly.table_bytes, cudaMemcpyDeviceToHost) == cudaSuccess ? SLONN_OK
                                                                                                : SLONN_ERR_CUDA;
}

// The run kernels stage a query's layer input in shared memory as fp32 (and, on an activator layer, a bitmap of
// the layer's nodes beside it): widths that cannot fit are refused when the model is made.
static bool widths_fit(uint32_t D, uint32_t N, bool has_act, bool csr_input)
{
    if (csr_input) return true;
    const uint64_t staged = (uint64_t)D * 4 + (has_act ? (uint64_t)((N + 31u) / 32u) * 4 : 0);
    return D <= SLONN_MAX_INPUT_WIDTH && staged <= (uint64_t)SLONN_MAX_INPUT_WIDTH * 4;
}

extern "C" int slonn_build(const slonn_build_desc *desc, const void *const *W, const float *const *bias,
                           const slonn_rows *calib, void *stream, slonn_model **out)
{
    if (!desc || !W || !bias || !out || !desc->dims || !desc->has_activator) return SLONN_ERR_ARG;
    if (desc->n_layers < 1 || desc->n_layers > SLONN_MAX_LAYERS) return SLONN_ERR_DIM;
    if (desc->dtype != SLONN_F32 && desc->dtype != SLONN_BF16) return SLONN_ERR_DTYPE;
    if (desc->K < 1 || desc->K > 16 || desc->L < 1 || desc->L > 8) return SLONN_ERR_DIM;
    const uint32_t esz = desc->dtype == SLONN_BF16 ? 2u : 4u;
    uint32_t n_act = 0;
    for (uint32_t l = 0; l < desc->n_layers; ++l) {
        const uint32_t D = desc->dims[l], N = desc->dims[l + 1];
        if (D == 0 || N == 0) return SLONN_ERR_DIM;
        if (!W[l] || !bias[l]) return SLONN_ERR_ARG;
        const bool sparse0 = (l == 0 && desc->first_layer_sparse);
        if (!widths_fit(D, N, desc->has_activator[l] != 0, sparse0)) return SLONN_ERR_DIM;
        if (!sparse0 && (((uint64_t)D * esz) & 15u)) return SLONN_ERR_ALIGN;
        if ((uintptr_t)W[l] & 15u) return SLONN_ERR_ALIGN;
        if (desc->has_activator[l]) {
            if (sparse0) return SLONN_ERR_ARG;
            if (desc->K * desc->L > N) return SLONN_ERR_DIM;
            if (desc->free_hash_nodes && desc->K * desc->L >= N) return SLONN_ERR_DIM;
            ++n_act;
        }
    }
    if (n_act) {
        if (!calib || calib->n_rows == 0) return SLONN_ERR_ARG;
        if (desc->first_layer_sparse ? (!calib->indptr || !calib->ids || !calib->vals) : !calib->dense)
            return SLONN_ERR_ARG;
        if (calib->dense && ((uintptr_t)calib->dense & 15u)) return SLONN_ERR_ALIGN;
    }

    slonn_model *m = new (std::nothrow) slonn_model;
    if (!m) return SLONN_ERR_NOMEM;
    memset(m, 0, sizeof(*m));
    m->magic = SLONN_MAGIC;
    cudaGetDevice(&m->device);
    m->n_layers = desc->n_layers;
    m->dtype = desc->dtype;
    m->K = desc->K; m->L = desc->L; m->H = desc->K * desc->L;
    m->list_cap = desc->list_cap;
    m->first_sparse = desc->first_layer_sparse ? 1u : 0u;
    m->free_hash = desc->free_hash_nodes ? 1u : 0u;
    for (uint32_t l = 0; l <= desc->n_layers; ++l) m->dims[l] = desc->dims[l];
    for (uint32_t l = 0; l < desc->n_layers; ++l) {
        slonn_layer &ly = m->layer[l];
        ly.W = W[l]; ly.bias = bias[l]; ly.D = desc->dims[l]; ly.N = desc->dims[l + 1];
        ly.has_act = desc->has_activator[l] ? 1u : 0u;
        if (ly.has_act) m->act_index[l] = m->n_act++;
    }

    cudaStream_t st = (cudaStream_t)stream;
    int rc = SLONN_OK;
    float *cur = nullptr, *A = nullptr;
    uint32_t *d_status = nullptr;
    uint32_t last_needed = 0;
    bool any = false;

    rc = make_transposed_copies(m, st, 0);
    if (rc) goto fail;
    for (uint32_t l = 0; l < m->n_layers; ++l)
        if (m->layer[l].has_act) { last_needed = l; any = true; }
    if (any) {
        const uint32_t n_cal = calib->n_rows;
        CK(cudaMalloc(&d_status, 4 * sizeof(uint32_t)));
        CK(cudaMemsetAsync(d_status, 0, 4 * sizeof(uint32_t), st));
        for (uint32_t l = 0; l <= last_needed; ++l) {
            const slonn_layer &ly = m->layer[l];
            const uint32_t relu = (l + 1 == m->n_layers) ? 0u : 1u;
            CK(cudaMalloc(&A, sizeof(float) * (uint64_t)n_cal * ly.N));
            if (l == 0 && m->first_sparse)
                rc = slonn_forward_sparse_first(m, calib->indptr, calib->ids, calib->vals, n_cal, A, relu, d_status, st);
            else
                rc = slonn_forward_all_rows(m, l, l == 0 ? calib->dense : cur, n_cal, A, relu, st);
            if (rc) goto fail;
            if (ly.has_act) {
                const uint32_t *ov = desc->hash_nodes_override ? desc->hash_nodes_override[l] : nullptr;
                if ((rc = train_layer(m, l, A, n_cal, desc->seed, ov, st))) goto fail;
            }
            CK(cudaStreamSynchronize(st));
            cudaFree(cur);
            cur = A;
            A = nullptr;
        }
        uint32_t hs[4];
        CK(cudaMemcpy(hs, d_status, sizeof(hs), cudaMemcpyDeviceToHost));
        if (hs[0]) { rc = -(int)hs[0]; goto fail; }
    }
    cudaFree(cur); cur = nullptr;
    rc = make_transposed_copies(m, st, 1);
    if (rc) goto fail;
    CK(cudaStreamSynchronize(st));
    cudaFree(cur); cudaFree(A); cudaFree(d_status);
    *out = m;
    return SLONN_OK;
fail:
    cudaFree(cur); cudaFree(A); cudaFree(d_status);
    slonn_free(m);
    return rc;
}

// ---------------------------------------------------------------------------
// Persisting a trained Node Activator.  The paper trains it "pre- or post-deployment"
// (Sec. 3.2), i.e. the tables are an artefact that outlives the process that made them.
// Blob (little endian): header, then per activator layer { L*K hash nodes, cap, id_bytes,
// table bytes }, then a 64-bit FNV-1a checksum of everything before it.  Weights are not part
// of the blob: the caller passes them again when loading, as for slonn_build.
// ---------------------------------------------------------------------------
namespace {

struct blob_header {
    uint32_t magic, version, n_layers, dtype, K, L, list_cap, first_sparse, free_hash;
    uint32_t dims[SLONN_MAX_LAYERS + 1];
    uint8_t has_act[SLONN_MAX_LAYERS];
};
constexpr uint32_t BLOB_MAGIC = 0x4e4e4c53u; // "SLNN"
constexpr uint32_t BLOB_VERSION = 2;

uint64_t fnv1a(const unsigned char *p, uint64_t n)
{
    uint64_t h = 0xcbf29ce484222325ull;
    for (uint64_t i = 0; i < n; ++i) { h ^= p[i]; h *= 0x100000001b3ull; }
    return h;
}

uint64_t blob_bytes(const slonn_model *m)
{
    uint64_t b = sizeof(blob_header);
    for (uint32_t l = 0; l < m->n_layers; ++l)
        if (m->layer[l].has_act) b += sizeof(uint32_t) * m->H + 2 * sizeof(uint32_t) + m->layer[l].table_bytes;
    return b + sizeof(uint64_t);
}

} // namespace

extern "C" int slonn_serialized_bytes(const slonn_model *m, uint64_t *bytes)
{
    if (!m || m->magic != SLONN_MAGIC || !bytes) return SLONN_ERR_ARG;
    *bytes = blob_bytes(m);
    return SLONN_OK;
}

extern "C" int slonn_serialize(const slonn_model *m, void *dst_host, uint64_t dst_bytes)
{
    if (!m || m->magic != SLONN_MAGIC || !dst_host) return SLONN_ERR_ARG;
    const uint64_t need = blob_bytes(m);
    if (dst_bytes < need) return SLONN_ERR_WORKSPACE;
    unsigned char *p = (unsigned char *)dst_host;
    blob_header h;
    memset(&h, 0, sizeof(h));
    h.magic = BLOB_MAGIC; h.version = BLOB_VERSION; h.n_layers = m->n_layers; h.dtype = (uint32_t)m->dtype;
    h.K = m->K; h.L = m->L; h.list_cap = m->list_cap; h.first_sparse = m->first_sparse; h.free_hash = m->free_hash;
    for (uint32_t l = 0; l <= m->n_layers; ++l) h.dims[l] = m->dims[l];
    for (uint32_t l = 0; l < m->n_layers; ++l) h.has_act[l] = (uint8_t)m->layer[l].has_act;
    memcpy(p, &h, sizeof(h));
    uint64_t o = sizeof(h);
    for (uint32_t l = 0; l < m->n_layers; ++l) {
        const slonn_layer &ly = m->layer[l];
        if (!ly.has_act) continue;
        memcpy(p + o, m->hash_nodes_host[l], sizeof(uint32_t) * m->H); o += sizeof(uint32_t) * m->H;
        memcpy(p + o, &ly.cap, 4); o += 4;
        memcpy(p + o, &ly.id_bytes, 4); o += 4;
        if (cudaMemcpy(p + o, ly.tables, ly.table_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return SLONN_ERR_CUDA;
        o += ly.table_bytes;
    }
    const uint64_t sum = fnv1a(p, o);
    memcpy(p + o, &sum, 8);
    return SLONN_OK;
}

extern "C" int slonn_deserialize(const void *src_host, uint64_t src_bytes, const void *const *W,
                                 const float *const *bias, void *stream, slonn_model **out)
{
    if (!src_host || !W || !bias || !out) return SLONN_ERR_ARG;
    if (src_bytes < sizeof(blob_header) + 8) return SLONN_ERR_ARG;
    const unsigned char *p = (const unsigned char *)src_host;
    blob_header h;
    memcpy(&h, p, sizeof(h));
    if (h.magic != BLOB_MAGIC || h.version != BLOB_VERSION) return SLONN_ERR_ARG;
    if (h.n_layers < 1 || h.n_layers > SLONN_MAX_LAYERS) return SLONN_ERR_DIM;
    if (h.dtype != SLONN_F32 && h.dtype != SLONN_BF16) return SLONN_ERR_DTYPE;
    if (h.K < 1 || h.K > 16 || h.L < 1 || h.L > 8) return SLONN_ERR_DIM;
    uint64_t sum_stored;
    memcpy(&sum_stored, p + src_bytes - 8, 8);
    if (fnv1a(p, src_bytes - 8) != sum_stored) return SLONN_ERR_ARG; // damaged or truncated blob
    const uint32_t esz = h.dtype == SLONN_BF16 ? 2u : 4u, H = h.K * h.L, nb = 1u << h.K;
    // walk the layer records once to validate sizes before anything is allocated
    {
        uint64_t o = sizeof(h);
        for (uint32_t l = 0; l < h.n_layers; ++l) {
            const uint32_t D = h.dims[l], N = h.dims[l + 1];
            if (D == 0 || N == 0) return SLONN_ERR_DIM;
            if (!widths_fit(D, N, h.has_act[l] != 0, l == 0 && h.first_sparse)) return SLONN_ERR_DIM;
            if (!W[l] || !bias[l]) return SLONN_ERR_ARG;
            if ((uintptr_t)W[l] & 15u) return SLONN_ERR_ALIGN;
            if (!(l == 0 && h.first_sparse) && (((uint64_t)D * esz) & 15u)) return SLONN_ERR_ALIGN;
            if (!h.has_act[l]) continue;
            if (H > N || (l == 0 && h.first_sparse)) return SLONN_ERR_DIM;
            if (o + sizeof(uint32_t) * H + 8 > src_bytes - 8) return SLONN_ERR_ARG;
            if (h.free_hash && H >= N) return SLONN_ERR_DIM;
            for (uint32_t k = 0; k < H; ++k) {
                uint32_t nd;
                memcpy(&nd, p + o + 4 * k, 4);
                if (nd >= N) return SLONN_ERR_ARG;
                for (uint32_t g = 0; g < k; ++g) { // hash nodes are distinct
                    uint32_t other;
                    memcpy(&other, p + o + 4 * g, 4);
                    if (other == nd) return SLONN_ERR_ARG;
                }
            }
            o += sizeof(uint32_t) * H;
            uint32_t cap, idb;
            memcpy(&cap, p + o, 4); memcpy(&idb, p + o + 4, 4); o += 8;
            if (cap < 1 || cap > (h.free_hash ? N - H : N) || idb != (N <= 65536u ? 2u : 4u)) return SLONN_ERR_ARG;
            const uint64_t tb = (uint64_t)h.L * nb * cap * idb;
            if (o + tb > src_bytes - 8) return SLONN_ERR_ARG;
            o += tb;
        }
        if (o != src_bytes - 8) return SLONN_ERR_ARG;
    }

    slonn_model *m = new (std::nothrow) slonn_model;
    if (!m) return SLONN_ERR_NOMEM;
    memset(m, 0, sizeof(*m));
    m->magic = SLONN_MAGIC;
    cudaGetDevice(&m->device);
    m->n_layers = h.n_layers; m->dtype = (int32_t)h.dtype; m->K = h.K; m->L = h.L; m->H = H;
    m->list_cap = h.list_cap; m->first_sparse = h.first_sparse ? 1u : 0u; m->free_hash = h.free_hash ? 1u : 0u;
    for (uint32_t l = 0; l <= h.n_layers; ++l) m->dims[l] = h.dims[l];
    cudaStream_t st = (cudaStream_t)stream;
    int rc = SLONN_OK;
    uint64_t o = sizeof(h);
    for (uint32_t l = 0; l < h.n_layers; ++l) {
        slonn_layer &ly = m->layer[l];
        ly.W = W[l]; ly.bias = bias[l]; ly.D = h.dims[l]; ly.N = h.dims[l + 1];
        ly.has_act = h.has_act[l] ? 1u : 0u;
        if (!ly.has_act) continue;
        m->act_index[l] = m->n_act++;
        memcpy(m->hash_nodes_host[l], p + o, sizeof(uint32_t) * H); o += sizeof(uint32_t) * H;
        memcpy(&ly.cap, p + o, 4); memcpy(&ly.id_bytes, p + o + 4, 4); o += 8;
        ly.table_bytes = (uint64_t)h.L * nb * ly.cap * ly.id_bytes;
        CK(cudaMalloc(&ly.hash_nodes, sizeof(uint32_t) * H));
        CK(cudaMemcpyAsync(ly.hash_nodes, m->hash_nodes_host[l], sizeof(uint32_t) * H, cudaMemcpyHostToDevice, st));
        CK(cudaMalloc(&ly.tables, ly.table_bytes));
        CK(cudaMemcpyAsync(ly.tables, p + o, ly.table_bytes, cudaMemcpyHostToDevice, st));
        o += ly.table_bytes;
    }
    rc = make_transposed_copies(m, st, 0);
    if (rc) goto fail;
    rc = make_transposed_copies(m, st, 1);
    if (rc) goto fail;
    CK(cudaStreamSynchronize(st));
    *out = m;
    return SLONN_OK;
fail:
    slonn_free(m);
    return rc;
}
