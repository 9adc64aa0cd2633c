// Dense layer on the 5th-generation tensor cores: C = act(A * W^T + bias) with bf16
// operands and fp32 accumulation.  This is the "all nodes computed" case of the paper
// (Sec. 3.4: at a 100 % budget an SLO-NN is the full network), the one stage of the path that
// is a dense contraction.
//
// Persistent kernel, one block per SM, 128 x 256 output tiles, K in steps of 64 (one 128-byte
// swizzle atom), six warps with fixed roles:
//   warp 0 / one lane : TMA producer, cp.async.bulk.tensor 2-D tile loads into a 4-stage ring
//   warp 1 / one lane : tcgen05.mma issuer; two accumulators of 256 columns in tensor memory,
//                       so the MMAs of tile i+1 run while tile i is drained
//   warps 2-5         : epilogue, tcgen05.ld of one accumulator (32 rows per warp), bias,
//                       activation, shared-memory transpose, coalesced stores
// Hand-over through mbarriers: TMA -> MMA by transaction bytes, MMA -> TMA and MMA -> epilogue by
// tcgen05.commit, epilogue -> MMA by plain arrivals.  Every wait is bounded: when one runs out the
// block raises an abort flag, lets outstanding copies land, frees its tensor memory and reports
// SLONN_ERR_TIMEOUT through the status word.  No cluster launch, no multicast.
//
// Sums are not bit-compatible with the fixed-order fp32 kernels (the tensor core's accumulation
// order is not specified), so this path is only used where the caller asked for it.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>

#include "slonn_common.cuh"
#include "slonn_dense_tc.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int THREADS = 192, EPI_WARPS = 4;
constexpr uint32_t TMEM_COLS = 2 * BN; // two accumulators
constexpr uint32_t STAGE_A_BYTES = BM * BK * 2, STAGE_B_BYTES = BN * BK * 2;
constexpr uint32_t RING_BYTES = STAGES * (STAGE_A_BYTES + STAGE_B_BYTES);
// per epilogue warp: two 32-row x 128-byte output slabs (bf16 tiles on their way to a TMA store); the
// 32x33 fp32 transpose tile of the list-output path lives in the same bytes
constexpr uint32_t OUT_SLAB_BYTES = 32 * 128, OUT_STAGE_BYTES = EPI_WARPS * 2 * OUT_SLAB_BYTES;
constexpr uint32_t ROW_OFF_BYTES = EPI_WARPS * 32 * 8; // 32 row offsets per epilogue warp
constexpr uint32_t SMEM_BYTES = RING_BYTES + OUT_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */ + ROW_OFF_BYTES;
static_assert(2 * OUT_SLAB_BYTES >= 32 * 33 * 4, "the transpose tile must fit in a warp's slabs");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory per block");
constexpr uint32_t WAIT_LIMIT = 1u << 22;

// instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = bn (a multiple of 16)
__device__ __forceinline__ uint32_t umma_idesc(uint32_t bn)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait; false when it gave up or another role already raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t limit = WAIT_LIMIT)
{
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap *map, int32_t c0, int32_t c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst_smem), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

// one 2-D tile from shared memory to global memory (rows and columns outside the tensor are dropped)
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src_smem, int32_t c0, int32_t c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src_smem), "r"(c0), "r"(c1)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return ((uint64_t)hi << 32) | lo;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); // NaN stays NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// two fp32 -> two bf16 (round to nearest even) in one 32-bit word, `lo` in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&p);
}

__global__ void __launch_bounds__(THREADS, 1)
dense_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_out, uint32_t tma_out, const slonn_dense_epilogue E, uint32_t N,
                uint32_t K, uint32_t bn, uint32_t probe_limit)
{
    // probe_limit: 0 in normal use.  Otherwise (a test of the give-up path) the producer first waits, for at most
    // that many polls, on a barrier nobody arrives at -- before any copy or MMA has been issued.
    // map_out / tma_out: the bf16 output matrix as a tensor of 64-column x 32-row boxes (128-byte swizzle),
    // valid when tma_out != 0
    // bn: columns per tile, a multiple of 16 up to BN (narrow layers take a narrower MMA and B tile)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    // rows this launch must produce (a device-side count when the rows were compacted on the device)
    const uint32_t m_valid = E.row_count ? min(*E.row_count, E.M) : E.M;
    const uint32_t m_tiles = (m_valid + BM - 1) / BM, n_tiles = (N + bn - 1) / bn;
    const uint32_t tiles = m_tiles * n_tiles;
    if (blockIdx.x >= tiles) return; // uniform for the block: nothing allocated yet

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u; // swizzle atoms need 1024-byte alignment
    const uint32_t out_stage0 = base + RING_BYTES; // 1024-byte aligned
    const uint32_t bars = out_stage0 + OUT_STAGE_BYTES;
    const uint32_t full0 = bars, empty0 = bars + 8 * STAGES;
    const uint32_t tfull0 = bars + 16 * STAGES, tempty0 = tfull0 + 16;
    const uint32_t tmem_slot_addr = tempty0 + 16;
    const uint32_t probe_bar = tempty0 + 32;
    const uint32_t epi_addr = bars + 256;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot_addr - smem_u32(smem_raw)));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, EPI_WARPS); }
        mbar_init(probe_bar, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) { // one warp allocates the accumulator columns and gives the permit back
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot_addr), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t num_kb = (K + BK - 1) / BK;

    if (warp == 0) {
        // ---- TMA producer: runs ahead over this block's tiles ----
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            if (probe_limit) ok = mbar_wait(probe_bar, 0u, abort_flag, probe_limit); // never completes: runs out
            for (uint32_t t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
                const uint32_t m0 = (t / n_tiles) * BM, n0 = (t % n_tiles) * bn;
                for (uint32_t kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag))) break;
                    mbar_expect_tx(full0 + 8 * s, STAGE_A_BYTES + bn * BK * 2);
                    tma_load_2d(base + s * STAGE_A_BYTES, &map_a, (int32_t)(kb * BK), (int32_t)m0, full0 + 8 * s);
                    tma_load_2d(base + STAGES * STAGE_A_BYTES + s * STAGE_B_BYTES, &map_b, (int32_t)(kb * BK),
                                (int32_t)n0, full0 + 8 * s);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: alternates between the two accumulators ----
        if (lane == 0) {
            uint32_t it = 0, ti = 0;
            bool ok = true;
            const uint32_t idesc = umma_idesc(bn);
            for (uint32_t t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++ti) {
                const uint32_t acc = ti & 1u, aph = (ti >> 1) & 1u;
                if (!(ok = mbar_wait(tempty0 + 8 * acc, aph ^ 1u, abort_flag))) break; // drained by the epilogue
                tc_fence_after();
                const uint32_t d = tmem_base + acc * BN;
                for (uint32_t kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(full0 + 8 * s, ph, abort_flag))) break;
                    tc_fence_after();
                    const uint64_t da = umma_desc(base + s * STAGE_A_BYTES);
                    const uint64_t db = umma_desc(base + STAGES * STAGE_A_BYTES + s * STAGE_B_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) // 32 bytes further along K inside the swizzle atom
                        umma_bf16(d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | (uint32_t)k) != 0u);
                    umma_commit(empty0 + 8 * s); // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(tfull0 + 8 * acc); // accumulator complete
            }
        }
    } else {
        // ---- epilogue warps: TMEM lane = row of the tile, TMEM column = column of the tile ----
        const uint32_t ew = warp - 2;        // slice of the staging area
        const uint32_t quarter = warp & 3u;  // the TMEM lanes 32*quarter .. +31 this warp may read
        const uint32_t slab0 = out_stage0 + ew * 2 * OUT_SLAB_BYTES;
        float *tile = reinterpret_cast<float *>(smem_raw + (slab0 - smem_u32(smem_raw)));
        unsigned long long *row_off = reinterpret_cast<unsigned long long *>(smem_raw + (epi_addr - smem_u32(smem_raw))) + ew * 32;
        uint32_t slab_turn = 0; // alternates between the warp's two output slabs
        // Row-major outputs with 16-byte aligned rows (no fp32 output addressed through per-row list
        // offsets, no id output) can be written by the lane that holds the row.
        const bool direct = !(E.out_f32 && E.indptr) && !E.out_ids &&
                            (!E.bias || (reinterpret_cast<uintptr_t>(E.bias) & 15u) == 0u) &&
                            (!E.out_f32 || ((reinterpret_cast<uintptr_t>(E.out_f32) & 15u) == 0u && (E.f32_stride & 3u) == 0u)) &&
                            (!E.out_bf16 || ((reinterpret_cast<uintptr_t>(E.out_bf16) & 15u) == 0u && (E.ld_bf16 & 7u) == 0u));
        uint32_t ti = 0;
        for (uint32_t t = blockIdx.x; t < tiles; t += gridDim.x, ++ti) {
            const uint32_t m0 = (t / n_tiles) * BM, n0 = (t % n_tiles) * bn;
            const uint32_t acc = ti & 1u, aph = (ti >> 1) & 1u;
            // warp-uniform outcome of the wait
            if (!__all_sync(SLONN_FULL_MASK, mbar_wait(tfull0 + 8 * acc, aph, abort_flag))) break;
            tc_fence_after();
            const uint32_t mrow0 = m0 + quarter * 32;
            unsigned long long off = ~0ull; // ~0: row not present
            if (mrow0 + lane < m_valid) {
                const uint32_t src = E.row_map ? E.row_map[mrow0 + lane] : mrow0 + lane;
                off = E.indptr ? E.indptr[(uint64_t)src * E.ip_mul + E.ip_add] : (uint64_t)src * E.f32_stride;
            }
            row_off[lane] = off;
            __syncwarp();
            if (direct && tma_out) {
                // bf16 outputs through shared memory and a TMA store: the lane converts its row of the
                // tile, 64 columns (128 bytes) at a time, into a swizzled slab; one lane then sends the slab
                // as a single tiled copy, so global memory sees whole 128-byte lines.
                for (uint32_t c2 = 0; c2 < bn; c2 += 64) {
                    if (n0 + c2 >= N) break; // uniform
                    const uint32_t slab = slab0 + (slab_turn & 1u) * OUT_SLAB_BYTES;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); // the copy before last has read this slab
                    __syncwarp();
#pragma unroll
                    for (uint32_t half = 0; half < 2; ++half) {
                        const uint32_t c = c2 + 32u * half;
                        if (c >= bn || n0 + c >= N) continue; // uniform; the copy drops these columns
                        uint32_t r[32];
                        tmem_load32(tmem_base + ((quarter * 32u) << 16) + acc * BN + c, r);
                        float v[32];
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4) {
                            float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (E.bias && n0 + c + 4 * j4 + 3 < N) bb = __ldg(reinterpret_cast<const float4 *>(E.bias + n0 + c) + j4);
                            v[4 * j4 + 0] = __uint_as_float(r[4 * j4 + 0]) + bb.x;
                            v[4 * j4 + 1] = __uint_as_float(r[4 * j4 + 1]) + bb.y;
                            v[4 * j4 + 2] = __uint_as_float(r[4 * j4 + 2]) + bb.z;
                            v[4 * j4 + 3] = __uint_as_float(r[4 * j4 + 3]) + bb.w;
                        }
                        if (E.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = v[j] > 0.0f ? v[j] : 0.0f;
                        }
                        if (E.out_f32 && off != ~0ull && n0 + c + 32 <= N) {
                            float4 *dst = reinterpret_cast<float4 *>(E.out_f32 + off + n0 + c);
#pragma unroll
                            for (int j4 = 0; j4 < 8; ++j4)
                                dst[j4] = make_float4(v[4 * j4], v[4 * j4 + 1], v[4 * j4 + 2], v[4 * j4 + 3]);
                        } else if (E.out_f32 && off != ~0ull) {
                            for (int j = 0; j < 32; ++j)
                                if (n0 + c + j < N) E.out_f32[off + n0 + c + j] = v[j];
                        }
#pragma unroll
                        for (uint32_t j8 = 0; j8 < 4; ++j8) {
                            uint4 o;
                            o.x = pack_bf16x2(v[8 * j8 + 0], v[8 * j8 + 1]);
                            o.y = pack_bf16x2(v[8 * j8 + 2], v[8 * j8 + 3]);
                            o.z = pack_bf16x2(v[8 * j8 + 4], v[8 * j8 + 5]);
                            o.w = pack_bf16x2(v[8 * j8 + 6], v[8 * j8 + 7]);
                            // 128-byte swizzle: 16-byte unit u of row `lane` sits at unit u ^ (lane & 7)
                            const uint32_t unit = (half * 4u + j8) ^ (lane & 7u);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                         ::"r"(slab + lane * 128u + unit * 16u), "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w)
                                         : "memory");
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); // generic-proxy writes before the bulk copy reads
                    __syncwarp();
                    if (lane == 0 && mrow0 < E.M) tma_store_2d(&map_out, slab, (int32_t)(n0 + c2), (int32_t)mrow0);
                    ++slab_turn;
                }
            } else
            for (uint32_t c = 0; c < bn; c += 32) {
                if (n0 + c >= N) break; // columns past the layer width (uniform)
                uint32_t r[32];
                tmem_load32(tmem_base + ((quarter * 32u) << 16) + acc * BN + c, r); // whole warp takes part
                if (direct && n0 + c + 32 <= N) {
                    // plain row-major outputs, 32 whole columns: the lane owns a row of the tile and writes
                    // its 32 values itself with 16-byte stores, no trip through shared memory
                    const float4 *b4 = reinterpret_cast<const float4 *>(E.bias + n0 + c);
                    float v[32];
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const float4 bb = E.bias ? __ldg(b4 + j4) : make_float4(0.f, 0.f, 0.f, 0.f);
                        v[4 * j4 + 0] = __uint_as_float(r[4 * j4 + 0]) + bb.x;
                        v[4 * j4 + 1] = __uint_as_float(r[4 * j4 + 1]) + bb.y;
                        v[4 * j4 + 2] = __uint_as_float(r[4 * j4 + 2]) + bb.z;
                        v[4 * j4 + 3] = __uint_as_float(r[4 * j4 + 3]) + bb.w;
                    }
                    if (E.relu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = v[j] > 0.0f ? v[j] : 0.0f;
                    }
                    if (off != ~0ull) {
                        if (E.out_f32) {
                            float4 *dst = reinterpret_cast<float4 *>(E.out_f32 + off + n0 + c);
#pragma unroll
                            for (int j4 = 0; j4 < 8; ++j4)
                                dst[j4] = make_float4(v[4 * j4], v[4 * j4 + 1], v[4 * j4 + 2], v[4 * j4 + 3]);
                        }
                        if (E.out_bf16) {
                            uint4 *dst = reinterpret_cast<uint4 *>(E.out_bf16 + (uint64_t)(mrow0 + lane) * E.ld_bf16 + n0 + c);
#pragma unroll
                            for (int j8 = 0; j8 < 4; ++j8) {
                                uint4 o;
                                o.x = pack_bf16x2(v[8 * j8 + 0], v[8 * j8 + 1]);
                                o.y = pack_bf16x2(v[8 * j8 + 2], v[8 * j8 + 3]);
                                o.z = pack_bf16x2(v[8 * j8 + 4], v[8 * j8 + 5]);
                                o.w = pack_bf16x2(v[8 * j8 + 6], v[8 * j8 + 7]);
                                dst[j8] = o;
                            }
                        }
                    }
                    continue;
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) tile[lane * 33 + j] = __uint_as_float(r[j]);
                __syncwarp();
                const uint32_t n = n0 + c + lane;
                const float bias = (E.bias && n < N) ? __ldg(E.bias + n) : 0.0f;
#pragma unroll 4
                for (int rr = 0; rr < 32; ++rr) {
                    const unsigned long long ro = row_off[rr];
                    if (ro == ~0ull || n >= N) continue;
                    float v = tile[rr * 33 + lane] + bias;
                    if (E.relu) v = v > 0.0f ? v : 0.0f;
                    if (E.out_f32) E.out_f32[ro + n] = v;
                    if (E.out_ids) E.out_ids[ro + n] = n;
                    if (E.out_bf16) E.out_bf16[(uint64_t)(mrow0 + rr) * E.ld_bf16 + n] = f32_to_bf16_rne(v);
                }
                __syncwarp();
            }
            // this warp has read its part of the accumulator: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); // output copies done before the block may leave
    }
    __syncwarp();
    if (*abort_flag) {
        // a wait ran out: give copies that may still be in flight time to land before the block leaves
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        if (threadIdx.x == 0 && E.status) slonn_report(E.status, SLONN_ERR_TIMEOUT, blockIdx.x, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode()
{
    static std::mutex mu;
    static encode_tiled_fn fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (encode_tiled_fn)p;
    }
    return fn;
}

// bf16 matrix [rows][cols] row-major with rows `ld` elements apart, tiles of box_rows rows x 64 columns,
// 128-byte swizzle, zero fill outside
int make_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, uint64_t ld = 0)
{
    encode_tiled_fn enc = get_encode();
    if (!enc) return SLONN_ERR_CUDA;
    if (ld == 0) ld = cols;
    if (((uintptr_t)ptr & 15u) || ((ld * 2) & 15u)) return SLONN_ERR_ALIGN;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SLONN_OK : SLONN_ERR_CUDA;
}

constexpr int MAX_DEVICES = 64;
std::mutex g_dev_mu;
bool g_attr_set[MAX_DEVICES];
int g_sm_count[MAX_DEVICES];
std::atomic<uint32_t> g_probe_limit{0}; // slonn_test_tc_wait_limit

} // namespace

extern "C" int slonn_test_tc_wait_limit(uint32_t polls)
{
    g_probe_limit.store(polls);
    return SLONN_OK;
}

int slonn_dense_tc_launch(const void *A, const void *W, uint32_t N, uint32_t K, const slonn_dense_epilogue &E,
                          cudaStream_t st)
{
    if (!A || !W || E.M == 0 || N == 0 || K == 0) return SLONN_ERR_ARG;
    CUtensorMap ma, mb;
    int rc;
    if ((rc = make_map(&ma, A, E.M, K, BM))) return rc;
    const uint32_t bn = std::min<uint32_t>((uint32_t)BN, (N + 15u) / 16u * 16u);
    if ((rc = make_map(&mb, W, N, K, bn))) return rc;
    // the shared-memory opt-in and the SM count belong to a device: looked up once per device ordinal
    int dev = 0, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLONN_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(g_dev_mu);
        const bool cached = dev >= 0 && dev < MAX_DEVICES;
        if (!cached || !g_attr_set[dev]) {
            if (cudaFuncSetAttribute(dense_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
                return SLONN_ERR_CUDA;
            if (cached) g_attr_set[dev] = true;
        }
        sm_count = cached ? g_sm_count[dev] : 0;
        if (sm_count == 0) {
            if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count < 1)
                return SLONN_ERR_CUDA;
            if (cached) g_sm_count[dev] = sm_count;
        }
    }
    // bf16 outputs leave through a TMA store when nothing needs per-row list addressing
    CUtensorMap mo;
    memset(&mo, 0, sizeof(mo));
    uint32_t tma_out = 0;
    if (E.out_bf16 && !(E.out_f32 && E.indptr) && !E.out_ids && ((uintptr_t)E.out_bf16 & 15u) == 0 && (E.ld_bf16 & 7u) == 0 &&
        E.ld_bf16 >= N) {
        if ((rc = make_map(&mo, E.out_bf16, E.M, N, 32, E.ld_bf16))) return rc;
        tma_out = 1;
    }
    const uint64_t tiles = (uint64_t)((N + bn - 1) / bn) * ((E.M + BM - 1) / BM);
    const uint32_t grid = (uint32_t)std::min<uint64_t>(tiles, (uint64_t)sm_count); // one persistent block per SM
    dense_tc_kernel<<<grid, THREADS, SMEM_BYTES, st>>>(ma, mb, mo, tma_out, E, N, K, bn, g_probe_limit.load());
    return cudaGetLastError() == cudaSuccess ? SLONN_OK : SLONN_ERR_CUDA;
}

extern "C" int slonn_dense_layer(const void *x_bf16, const void *w_bf16, const float *bias, uint32_t M, uint32_t N,
                                 uint32_t D, uint32_t relu, float *out_f32, void *out_bf16, uint32_t *status,
                                 void *stream)
{
    if (!x_bf16 || !w_bf16 || (!out_f32 && !out_bf16)) return SLONN_ERR_ARG;
    if (M == 0 || N == 0 || D == 0) return SLONN_ERR_DIM;
    slonn_dense_epilogue E;
    memset(&E, 0, sizeof(E));
    E.M = M; E.bias = bias; E.relu = relu;
    E.out_f32 = out_f32; E.f32_stride = N;
    E.out_bf16 = (uint16_t *)out_bf16; E.ld_bf16 = N;
    E.status = status;
    if (status && cudaMemsetAsync(status, 0, 4 * sizeof(uint32_t), (cudaStream_t)stream) != cudaSuccess) return SLONN_ERR_CUDA;
    return slonn_dense_tc_launch(x_bf16, w_bf16, N, D, E, (cudaStream_t)stream);
}
