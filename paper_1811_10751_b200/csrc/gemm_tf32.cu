// FP32-storage worker products on the tcgen05 tensor cores with 3xTF32 splitting.
#include "gemm_common.h"

namespace gpd {

bool sgemm_3xtf32_supported(const GemmParams&) { return false; }
gpd_status sgemm_3xtf32_launch(const GemmParams&, cudaStream_t) { return GPD_ERR_UNSUPPORTED; }

}  // namespace gpd
