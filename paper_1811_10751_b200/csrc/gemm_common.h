// Parameters shared by the worker-product kernels (batched over the P nodes).
#pragma once

#include "gpd_internal.h"

namespace gpd {

// out[p] (M x N, row-major) = A[p] (M x K, row-major) * B[p]
//   b_kmajor == 0 : B[p] is K x N row-major   (forward: X~_p;  backward: W~_p)
//   b_kmajor == 1 : B[p] is N x K row-major   (update: X^_p, contraction over the batch)
// update == 1 : out[p] <- shrink * out[p] + eta * A[p] B[p]   (Eq. 10), skipped when the gate
//               result reports a decoding failure.
struct GemmParams {
    const void* A;
    const void* B;
    void* C;
    int64_t M, N, K;
    int P;
    int b_kmajor;
    int update;
    double shrink, eta;
    const gpd_locate_result* gate;
    int max_threshold;      // largest recovery threshold the result will be decoded with (0: unknown);
                            // the FP32 tensor-core path shortens its accumulation chains for large ones
    void* splitk_scratch;   // device scratch for the FP32 tensor-core path's split contraction (may be null)
    int64_t splitk_bytes;
};

gpd_status gemm_generic_launch(const GemmParams& prm, int elem_size, cudaStream_t st);
gpd_status gemv_launch(const GemmParams& prm, int elem_size, cudaStream_t st);
bool dgemm_mma_supported(const GemmParams& prm);
gpd_status dgemm_mma_launch(const GemmParams& prm, cudaStream_t st);
bool sgemm_3xtf32_supported(const GemmParams& prm);
gpd_status sgemm_3xtf32_launch(const GemmParams& prm, cudaStream_t st);
// Scratch the FP32 tensor-core path wants for cutting `pieces` parts out of its left-over tiles (pieces <= SM count).
int64_t sgemm_3xtf32_scratch_bytes(int64_t pieces);
gpd_status bounded_wait_selftest_launch(long long limit_cycles, cudaStream_t st);
int tf32_device_status_fetch_and_clear();   // synchronous read of the tensor-path status word

}  // namespace gpd
