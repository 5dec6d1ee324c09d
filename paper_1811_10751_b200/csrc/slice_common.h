// Integer-slice product paths (GPD_PREC_FP64_SLICED, _SLICED40, _SLICED_TRAIN): layout of the sliced
// share buffers and the entry points of their encoders (slice.cu) and of the tensor-core products
// (gemm_i8.cu).
#pragma once

#include "gpd_internal.h"

namespace gpd {

constexpr int kMaxSlices = 6;      // signed 8-bit digits kept per value: 6 (48 bits below the row scale) or 5 (40 bits)
constexpr int kDigitBits = 8;

// A sliced operand with R rows of K contiguous elements per node:
//   int8 planes [S][P][R][K], then (256-byte aligned) int32 exponents [P][R], then
//   (256-byte aligned) 4-byte encoder scratch [P][R].
// value(p, r, k) = 2^expo[p][r] * sum_t planes[t][p][r][k] * 2^(-8 (t + 1))
struct SlicedLayout {
    int64_t plane_bytes;   // P * R * K
    int64_t expo_offset;   // byte offset of the exponents
    int64_t amax_offset;   // byte offset of the encoder's scratch
    int64_t total_bytes;
};
SlicedLayout sliced_layout(int slices, int64_t P, int64_t rows, int64_t K);

// Share buffer of W in the training mode (GPD_PREC_FP64_SLICED_TRAIN), M = N1/m, K = N0/n:
//   [0, rows_offset)            FP64 shares [P][M][K]: what the update accumulates into and what audit,
//                               regeneration and share-error injection read and write
//   [rows_offset, cols_offset)  the same values as a sliced operand with rows = share rows (K contiguous):
//                               left operand of the forward product
//   [cols_offset, total)        and as a sliced operand with rows = share columns (M contiguous): right
//                               operand of the backward product
// The two sliced copies are cut anew from the FP64 shares whenever those change.
struct TrainLayout {
    int64_t rows_offset, cols_offset, total_bytes;
    SlicedLayout rows, cols;
};
TrainLayout train_layout(const gpd_plan_s* plan);

// Whether the plan's shapes fit this path (contraction lengths multiples of 16 and at most 16384, block
// counts the encoders are instantiated for, sliced buffers no larger than the FP64 buffers they replace).
bool sliced_supported(const gpd_plan_s* plan);

// Encoders.  operand: -1 = W (gpd_encode_A), else a gpd_operand.  dst: the caller's share buffer.
gpd_status encode_sliced_launch(gpd_plan_s* plan, int operand, const float* src, void* dst, cudaStream_t st);
// Training mode: cut both sliced copies of W's shares from the FP64 shares at the start of the buffer.
// gate (optional): a result whose decoding failure means the shares were left as they were: nothing is re-cut.
// cols_amax_ready: the column maxima already sit in the column copy's scratch (the update's epilogue met them).
gpd_status reslice_launch(gpd_plan_s* plan, void* W_shares, cudaStream_t st, const gpd_locate_result* gate = nullptr,
                          bool cols_amax_ready = false);

// One batched int8 digit-plane product with FP64 recombination:
//   C[p] (M x N, FP64, row-major) = A[p] (M x K) * B[p] (N x K)^T      for p = 0 .. P-1,
// both operands sliced with K contiguous; update: C[p] <- shrink * C[p] + eta * A[p] B[p]^T, skipped
// when gate reports a decoding failure.
struct I8Gemm {
    int slices, P;
    const void* A; const int* ea; int64_t M;
    const void* B; const int* eb; int64_t N;
    int64_t K;
    double* C;
    bool update;
    double shrink, eta;
    const gpd_locate_result* gate;
    unsigned int* colmax;       // update, optional: [P][N] largest |new C| per column (high words, zero on entry)
};
gpd_status gemm_i8_launch(const I8Gemm& g, cudaStream_t st);

// S~_p = W~_p X~_p (GPD_FWD) or C~^T_p = Delta~^T_p W~_p (GPD_BWD, training mode) from sliced operands.
gpd_status gemm_sliced_launch(gpd_plan_s* plan, gpd_product which, const void* W_shares, const void* other_sliced,
                              void* out, cudaStream_t st);
// Training mode: FP64 shares <- shrink * shares + eta * Delta^_p X^_p^T, then both sliced copies re-cut.
gpd_status update_sliced_launch(gpd_plan_s* plan, void* W_shares, const void* Dhat_sliced, const void* Xhat_sliced,
                                double shrink, double eta, const gpd_locate_result* gate, cudaStream_t st);
int i8_device_status_fetch_and_clear();

}  // namespace gpd
