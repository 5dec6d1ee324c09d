// Integer-slice product path (GPD_PREC_FP64_SLICED): layout of a sliced share buffer and the
// entry points of its encoder (slice.cu) and of its tensor-core product (gemm_i8.cu).
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

// Whether the plan's shapes fit this path (K = N0/n a multiple of 16, block counts the encoder
// is instantiated for, sliced buffers no larger than the FP64 share buffers they replace).
bool sliced_supported(const gpd_plan_s* plan);

// W~_p (is_A) or X~_p -> sliced operand (W: rows of the share; X: columns of the share).
gpd_status encode_sliced_launch(gpd_plan_s* plan, bool is_A, const float* src, void* dst, cudaStream_t st);

// S~_p = W~_p X~_p for all p from the two sliced operands, FP64 output [P][M][N].
gpd_status gemm_sliced_launch(gpd_plan_s* plan, const void* W_sliced, const void* X_sliced, void* out,
                              cudaStream_t st);
int i8_device_status_fetch_and_clear();

}  // namespace gpd
