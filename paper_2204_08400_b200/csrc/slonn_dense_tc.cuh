// Interface of the tensor-core dense layer (slonn_dense_tc.cu) to the rest of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

// Where the rows of C = act(A * W^T + bias) go.  Row m of A is either row m of the outputs or,
// when the rows were gathered from a larger batch, the row named by row_map[m].
struct slonn_dense_epilogue {
    uint32_t M;                 // rows of A (upper bound when row_count is given)
    const uint32_t *row_count;  // device: rows actually present, nullable
    const uint32_t *row_map;    // device: source row (query) of each A row, nullable
    const float *bias;          // [N], nullable
    uint32_t relu;
    float *out_f32;             // nullable; row base = indptr[src * ip_mul + ip_add] or src * f32_stride
    uint32_t *out_ids;          // nullable; same addressing, receives the column index
    const uint64_t *indptr;     // nullable
    uint32_t ip_mul, ip_add;
    uint64_t f32_stride;
    uint16_t *out_bf16;         // nullable; dense [M][ld_bf16], row m (not remapped): the next layer's A
    uint32_t ld_bf16;
    uint32_t *status;           // nullable
};

// A: bf16 [M][K] row-major, W: bf16 [N][K] row-major; K * 2 bytes a multiple of 16.
int slonn_dense_tc_launch(const void *A, const void *W, uint32_t N, uint32_t K, const slonn_dense_epilogue &E,
                          cudaStream_t st);
