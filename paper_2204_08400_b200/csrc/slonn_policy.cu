// Accuracy-constrained budget choice (ACLO, Sec. 2.2 Eq. 2) and what it needs: the confidence
// measure c(k, x) (Sec. 2.1 Eq. 1), the Confidence LSH tables (Sec. 3.2 Eq. 4) trained on
// unlabelled rows with the network's own forward pass, and the per-query lookup that turns an
// accuracy target's confidence thresholds into a budget.
#include <cstring>
#include <new>

#include "slonn_common.cuh"

#define SLONN_THREADS 256
#define SLONN_ROWS_PER_WARP 4 // hash rows per warp pass (reduce_rows4)
#define SLONN_CONF_MAGIC 0x434f4e46u /* "CONF" */
#define SLONN_MAX_PROFILE 64

struct slonn_confidence {
    uint32_t magic;
    int device;
    uint32_t K, L, n_k;
    uint16_t profile_bp_host[SLONN_MAX_PROFILE];
    uint16_t *profile_bp; // device [n_k]
    double *sum;          // device [L][2^K][n_k]
    uint32_t *count;      // device [L][2^K]
};

namespace {

#define PCK(call) do { if ((call) != cudaSuccess) { rc = SLONN_ERR_CUDA; goto fail; } } while (0)

__global__ void fill_u16_kernel(uint16_t *dst, uint32_t n, uint16_t v)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = v;
}

// c(k, x) of one row per thread: sum_j softmax(z_full)_j * log softmax(z_k)_j in fp64, both
// softmaxes shifted by their maximum, terms added in index order without contraction.
__global__ void confidence_kernel(const float *z_full, const float *z_k, uint32_t n_rows, uint32_t n_out, double *c)
{
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= n_rows) return;
    const float *zf = z_full + (uint64_t)x * n_out, *zk = z_k + (uint64_t)x * n_out;
    double mf = (double)zf[0], mk = (double)zk[0];
    for (uint32_t j = 1; j < n_out; ++j) {
        if ((double)zf[j] > mf) mf = (double)zf[j];
        if ((double)zk[j] > mk) mk = (double)zk[j];
    }
    double sf = 0.0, sk = 0.0;
    for (uint32_t j = 0; j < n_out; ++j) {
        sf = __dadd_rn(sf, exp(__dsub_rn((double)zf[j], mf)));
        sk = __dadd_rn(sk, exp(__dsub_rn((double)zk[j], mk)));
    }
    const double lse_k = __dadd_rn(mk, log(sk));
    double acc = 0.0;
    for (uint32_t j = 0; j < n_out; ++j) {
        const double y = __ddiv_rn(exp(__dsub_rn((double)zf[j], mf)), sf);
        acc = __dadd_rn(acc, __dmul_rn(y, __dsub_rn((double)zk[j], lse_k)));
    }
    c[x] = acc;
}

// One thread per bucket (table b, key): rows of the first activator layer's codes that fall into it.
__global__ void confidence_count_kernel(const uint16_t *codes, uint32_t n_rows, uint32_t n_act, uint32_t L, uint32_t nb,
                                        uint32_t *count)
{
    const uint32_t bk = blockIdx.x * blockDim.x + threadIdx.x;
    if (bk >= L * nb) return;
    const uint32_t b = bk / nb, key = bk - b * nb;
    uint32_t n = 0;
    for (uint32_t x = 0; x < n_rows; ++x) n += (codes[((uint64_t)x * n_act) * L + b] == key) ? 1u : 0u;
    count[bk] = n;
}

// sum[b][key][i] = the bucket's rows' confidences added in row order (fp64).
__global__ void confidence_sum_kernel(const uint16_t *codes, const double *c, uint32_t n_rows, uint32_t n_act, uint32_t L,
                                      uint32_t nb, uint32_t i, uint32_t n_k, double *sum)
{
    const uint32_t bk = blockIdx.x * blockDim.x + threadIdx.x;
    if (bk >= L * nb) return;
    const uint32_t b = bk / nb, key = bk - b * nb;
    double s = 0.0;
    for (uint32_t x = 0; x < n_rows; ++x)
        if (codes[((uint64_t)x * n_act) * L + b] == key) s = __dadd_rn(s, c[x]);
    sum[(uint64_t)bk * n_k + i] = s;
}

struct slonn_aclo_params {
    const float *x;            // [n][D]
    const void *W;             // layer 0
    const float *bias;
    const uint32_t *hash_nodes;
    uint32_t D, nchunks, K, L, n_k;
    const double *sum;
    const uint32_t *count;
    const uint16_t *profile_bp;
    const float *threshold;    // [n_targets][n_k]
    const uint32_t *target;    // [n], nullable
    uint32_t n_targets;
    uint16_t *budget_bp;
    uint8_t *met;              // nullable
    double *estimate;          // [n][n_k], nullable
    uint32_t *status;          // nullable
};

// One block per query: the first layer's FreeHash keys of x (same fixed-order dot products as the
// forward pass), the pooled bucket means per profiled k, the smallest k that reaches its threshold.
template <bool BF16>
__global__ void __launch_bounds__(SLONN_THREADS) aclo_budget_kernel(slonn_aclo_params P)
{
    extern __shared__ float4 smem4[];
    __shared__ float zh[128];
    __shared__ uint32_t keys[8];
    __shared__ double est_s[SLONN_MAX_PROFILE];
    __shared__ uint32_t rows_s;
    const uint32_t q = blockIdx.x;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t H = P.K * P.L, nb = 1u << P.K;
    slonn_input in;
    in.kind = SLONN_IN_DENSE; in.dense = P.x; in.indptr = nullptr; in.ids = nullptr; in.vals = nullptr;
    in.ip_mul = in.ip_add = 0;
    stage_input<BF16>(in, q, P.D, P.nchunks, smem4);
    for (uint32_t h0 = warp * SLONN_ROWS_PER_WARP; h0 < H; h0 += nwarps * SLONN_ROWS_PER_WARP) {
        const uint4 *rows[SLONN_ROWS_PER_WARP];
#pragma unroll
        for (int r = 0; r < SLONN_ROWS_PER_WARP; ++r) {
            const uint32_t nd = __ldg(P.hash_nodes + min(h0 + r, H - 1));
            rows[r] = reinterpret_cast<const uint4 *>(P.W) + (uint64_t)nd * P.nchunks;
        }
        float acc[SLONN_ROWS_PER_WARP];
        warp_dot_rows<BF16, SLONN_ROWS_PER_WARP>(rows, smem4, P.nchunks, lane, acc);
        const float sum = reduce_rows4(acc, lane);
        const uint32_t h = h0 + (lane >> 3);
        if ((lane & 7u) == 0u && h < H) zh[h] = sum + __ldg(P.bias + __ldg(P.hash_nodes + h));
    }
    __syncthreads();
    if (threadIdx.x < P.L) {
        uint32_t key = 0;
        for (uint32_t j = 0; j < P.K; ++j)
            if (zh[threadIdx.x * P.K + j] > 0.0f) key |= (1u << j);
        keys[threadIdx.x] = key;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t rows = 0;
        for (uint32_t b = 0; b < P.L; ++b) rows += P.count[b * nb + keys[b]];
        rows_s = rows;
    }
    __syncthreads();
    if (threadIdx.x < P.n_k) {
        double s = 0.0;
        for (uint32_t b = 0; b < P.L; ++b) s = __dadd_rn(s, P.sum[((uint64_t)b * nb + keys[b]) * P.n_k + threadIdx.x]);
        const double est = rows_s ? __ddiv_rn(s, (double)rows_s) : 0.0;
        est_s[threadIdx.x] = est;
        if (P.estimate) P.estimate[(uint64_t)q * P.n_k + threadIdx.x] = est;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = P.target ? P.target[q] : 0u;
        if (t >= P.n_targets) {
            if (P.status) slonn_report(P.status, SLONN_ERR_ARG, q, 0);
            t = 0;
        }
        const float *thr = P.threshold + (uint64_t)t * P.n_k;
        uint16_t pick = 10000;
        uint8_t ok = 0;
        if (rows_s)
            for (uint32_t i = 0; i < P.n_k; ++i)
                if (est_s[i] >= (double)thr[i]) { pick = P.profile_bp[i]; ok = 1; break; }
        P.budget_bp[q] = pick;
        if (P.met) P.met[q] = ok;
    }
}

inline bool aclo_model_ok(const slonn_model *m)
{
    return m && m->magic == SLONN_MAGIC && m->layer[0].has_act && !m->first_sparse &&
           !m->layer[m->n_layers - 1].has_act;
}

} // namespace

extern "C" int slonn_confidence_build(const slonn_model *m, const slonn_rows *rows, const uint16_t *profile_bp,
                                      uint32_t n_k, void *stream, slonn_confidence **out)
{
    if (!m || m->magic != SLONN_MAGIC || !rows || !profile_bp || !out) return SLONN_ERR_ARG;
    if (!aclo_model_ok(m) || !rows->dense || rows->n_rows == 0) return SLONN_ERR_ARG;
    if ((uintptr_t)rows->dense & 15u) return SLONN_ERR_ALIGN;
    if (n_k < 1 || n_k > SLONN_MAX_PROFILE) return SLONN_ERR_DIM;
    for (uint32_t i = 0; i < n_k; ++i) {
        if (profile_bp[i] < 1 || profile_bp[i] > 10000) return SLONN_ERR_BUDGET;
        if (i && profile_bp[i] <= profile_bp[i - 1]) return SLONN_ERR_ARG; // ascending
    }
    slonn_confidence *c = new (std::nothrow) slonn_confidence;
    if (!c) return SLONN_ERR_NOMEM;
    memset(c, 0, sizeof(*c));
    c->magic = SLONN_CONF_MAGIC;
    cudaGetDevice(&c->device);
    c->K = m->K; c->L = m->L; c->n_k = n_k;
    memcpy(c->profile_bp_host, profile_bp, sizeof(uint16_t) * n_k);

    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t n = rows->n_rows, n_out = m->dims[m->n_layers], nb = 1u << m->K, nseg = nb * m->L;
    int rc = SLONN_OK;
    float *zf = nullptr, *zk = nullptr;
    uint16_t *codes = nullptr, *bp = nullptr;
    uint32_t *status = nullptr;
    double *conf = nullptr;
    void *ws = nullptr;
    uint64_t ws_bytes = 0;
    uint32_t hs[4];
    slonn_batch b;
    memset(&b, 0, sizeof(b));

    PCK(cudaMalloc(&c->profile_bp, sizeof(uint16_t) * n_k));
    PCK(cudaMalloc(&c->sum, sizeof(double) * (uint64_t)nseg * n_k));
    PCK(cudaMalloc(&c->count, sizeof(uint32_t) * nseg));
    PCK(cudaMemcpyAsync(c->profile_bp, c->profile_bp_host, sizeof(uint16_t) * n_k, cudaMemcpyHostToDevice, st));
    PCK(cudaMalloc(&zf, sizeof(float) * (uint64_t)n * n_out));
    PCK(cudaMalloc(&zk, sizeof(float) * (uint64_t)n * n_out));
    PCK(cudaMalloc(&codes, sizeof(uint16_t) * (uint64_t)n * m->n_act * m->L));
    PCK(cudaMalloc(&bp, sizeof(uint16_t) * n));
    PCK(cudaMalloc(&status, 4 * sizeof(uint32_t)));
    PCK(cudaMalloc(&conf, sizeof(double) * n));
    if ((rc = slonn_workspace_bytes(m, n, 10000, 0, &ws_bytes))) goto fail;
    PCK(cudaMalloc(&ws, ws_bytes));

    // the complete network: reference logits and the first layer's keys of every row
    b.n_queries = n; b.x_dense = rows->dense; b.budget_bp = bp; b.max_budget_bp = 10000;
    b.logits = zf; b.codes = codes; b.status = status;
    fill_u16_kernel<<<(n + 255) / 256, 256, 0, st>>>(bp, n, (uint16_t)10000);
    PCK(cudaGetLastError());
    if ((rc = slonn_run(m, &b, ws, ws_bytes, st))) goto fail;
    PCK(cudaMemcpyAsync(hs, status, sizeof(hs), cudaMemcpyDeviceToHost, st));
    PCK(cudaStreamSynchronize(st));
    if (hs[0]) { rc = -(int)hs[0]; goto fail; }
    confidence_count_kernel<<<(nseg + 127) / 128, 128, 0, st>>>(codes, n, m->n_act, m->L, nb, c->count);
    PCK(cudaGetLastError());

    // every profiled k: the k% network's logits, each row's confidence, the buckets' sums
    b.logits = zk; b.codes = nullptr;
    for (uint32_t i = 0; i < n_k; ++i) {
        fill_u16_kernel<<<(n + 255) / 256, 256, 0, st>>>(bp, n, profile_bp[i]);
        PCK(cudaGetLastError());
        b.max_budget_bp = profile_bp[i];
        if ((rc = slonn_run(m, &b, ws, ws_bytes, st))) goto fail;
        PCK(cudaMemcpyAsync(hs, status, sizeof(hs), cudaMemcpyDeviceToHost, st));
        confidence_kernel<<<(n + 127) / 128, 128, 0, st>>>(zf, zk, n, n_out, conf);
        confidence_sum_kernel<<<(nseg + 127) / 128, 128, 0, st>>>(codes, conf, n, m->n_act, m->L, nb, i, n_k, c->sum);
        PCK(cudaGetLastError());
        PCK(cudaStreamSynchronize(st));
        if (hs[0]) { rc = -(int)hs[0]; goto fail; }
    }
    cudaFree(zf); cudaFree(zk); cudaFree(codes); cudaFree(bp); cudaFree(status); cudaFree(conf); cudaFree(ws);
    *out = c;
    return SLONN_OK;
fail:
    cudaFree(zf); cudaFree(zk); cudaFree(codes); cudaFree(bp); cudaFree(status); cudaFree(conf); cudaFree(ws);
    slonn_confidence_free(c);
    return rc;
}

extern "C" void slonn_confidence_free(slonn_confidence *c)
{
    if (!c || c->magic != SLONN_CONF_MAGIC) return;
    cudaFree(c->profile_bp); cudaFree(c->sum); cudaFree(c->count);
    c->magic = 0;
    delete c;
}

extern "C" int slonn_confidence_to_host(const slonn_confidence *c, double *sum_host, uint64_t sum_entries,
                                        uint32_t *count_host, uint64_t count_entries)
{
    if (!c || c->magic != SLONN_CONF_MAGIC || !sum_host || !count_host) return SLONN_ERR_ARG;
    const uint64_t nseg = (uint64_t)c->L << c->K;
    if (sum_entries < nseg * c->n_k || count_entries < nseg) return SLONN_ERR_WORKSPACE;
    if (cudaMemcpy(sum_host, c->sum, sizeof(double) * nseg * c->n_k, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(count_host, c->count, sizeof(uint32_t) * nseg, cudaMemcpyDeviceToHost) != cudaSuccess)
        return SLONN_ERR_CUDA;
    return SLONN_OK;
}

extern "C" int slonn_aclo_budgets(const slonn_model *m, const slonn_confidence *c, const float *x_dense, uint32_t n,
                                  const float *threshold, uint32_t n_targets, const uint32_t *target,
                                  uint16_t *budget_bp, uint8_t *met, double *estimate, uint32_t *status, void *stream)
{
    if (!aclo_model_ok(m) || !c || c->magic != SLONN_CONF_MAGIC) return SLONN_ERR_ARG;
    if (c->K != m->K || c->L != m->L) return SLONN_ERR_ARG;
    if (!threshold || n_targets == 0 || !budget_bp) return SLONN_ERR_ARG;
    if (n == 0) return SLONN_OK;
    if (!x_dense) return SLONN_ERR_ARG;
    if ((uintptr_t)x_dense & 15u) return SLONN_ERR_ALIGN;
    const slonn_layer &l0 = m->layer[0];
    slonn_aclo_params P;
    memset(&P, 0, sizeof(P));
    P.x = x_dense; P.W = l0.W; P.bias = l0.bias; P.hash_nodes = l0.hash_nodes;
    P.D = l0.D; P.nchunks = l0.D * (m->dtype == SLONN_BF16 ? 2u : 4u) / 16u; P.K = m->K; P.L = m->L; P.n_k = c->n_k;
    P.sum = c->sum; P.count = c->count; P.profile_bp = c->profile_bp;
    P.threshold = threshold; P.target = target; P.n_targets = n_targets;
    P.budget_bp = budget_bp; P.met = met; P.estimate = estimate; P.status = status;
    const size_t smem = (size_t)l0.D * 4;
    cudaStream_t st = (cudaStream_t)stream;
    {
        const int rc = m->dtype == SLONN_BF16 ? slonn_allow_smem(reinterpret_cast<const void *>(aclo_budget_kernel<true>), smem)
                                              : slonn_allow_smem(reinterpret_cast<const void *>(aclo_budget_kernel<false>), smem);
        if (rc) return rc;
    }
    if (m->dtype == SLONN_BF16) aclo_budget_kernel<true><<<n, SLONN_THREADS, smem, st>>>(P);
    else aclo_budget_kernel<false><<<n, SLONN_THREADS, smem, st>>>(P);
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}
