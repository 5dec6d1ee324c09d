// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "gpd.h"

namespace gpd {

constexpr int kMaxNodes = GPD_MAX_NODES;
constexpr int kMaxQ = GPD_MAX_THRESHOLD;
constexpr int kMaxR = GPD_MAX_PARITY;
constexpr int kMaxBlocks = 64;   // blocks combined by one encoding polynomial (m*n, n*d1, d2*m)
constexpr int kMaxWanted = 64;   // wanted coefficients of one product (m*d1, d2*n, m*n)

// Zero tests of the locator in floating point (engineering constants, chosen from the noise
// floor of each storage type; the paper works in exact real arithmetic).
constexpr double kTauColFp32 = 1.220703125e-4;           // 2^-13
constexpr double kTauInFp32 = 3.0517578125e-5;           // 2^-15
constexpr double kTauColFp64 = 9.5367431640625e-7;       // 2^-20
constexpr double kTauInFp64 = 9.313225746154785e-10;     // 2^-30

// A worker output of magnitude >= kHuge is handled like a non-finite one (zeroed, its node flagged):
// the squared norms of the zero test stay inside the FP64 range for up to 64 values below it.
constexpr double kHuge = 3.273390607896142e150;          // 2^500
constexpr double kHugeSquared = 1.0715086071862673e301;  // 2^1000

// Geometry of one decodable product (forward, backward or audit).
struct ProductInfo {
    int Q = 0;             // recovery threshold = number of polynomial coefficients
    int R = 0;             // P - Q parity checks
    int grid_rows = 0;     // wanted block grid (m x d1, d2 x n, m x n)
    int grid_cols = 0;
    int64_t br = 0;        // rows / cols of one worker output = one result block
    int64_t bc = 0;
    int wanted[kMaxWanted] = {0};   // exponent of block (r, c), row-major over the grid
    std::vector<double> H;          // R x P, orthonormal rows, H * Vandermonde(points, Q) = 0
    std::vector<double> Hg;         // R x P, row j = w_p b_p^j (w the barycentric weights of the points,
                                    // largest magnitude 1): the same null space in power-sum form
    // offsets (in doubles) into the device table buffer
    int64_t off_H = 0, off_Hg = 0;
};

// Device-resident tables of a plan (one allocation).
struct DeviceTables {
    double* base = nullptr;
    int64_t n_doubles = 0;
    int64_t off_points = 0;
    int64_t off_coefW = 0, off_coefX = 0, off_coefDT = 0, off_coefDup = 0, off_coefXup = 0;
    // FP32 plans: scratch behind the tables (same allocation) in which the tensor-core products add up the
    // parts of a split contraction; one product launch of a plan uses it at a time
    void* splitk = nullptr;
    int64_t splitk_bytes = 0;
    // decoding matrices of the error-free case (every node in use), one per product, computed once at
    // upload by the kernel that otherwise computes them per call: [wanted][P] doubles at these offsets
    // (in doubles from base; -1: none), and one int of scratch for that kernel's gate
    int64_t off_dcache[4] = {-1, -1, -1, -1};
    int64_t off_dcache_gate = -1;
};

}  // namespace gpd

struct gpd_plan_s {
    gpd_shape shape;
    gpd_split split;
    int P = 0;
    int Qf = 0, Qb = 0, Qw = 0;  // thresholds under the plan's substitution
    gpd_precision prec = GPD_PREC_FP32;
    int elem_size = 4;
    bool sliced = false;         // GPD_PREC_FP64_SLICED / _SLICED40: shares are int8 digit planes, outputs double
    int slices = 0;              // digit planes per operand (6 or 5) when sliced
    bool train = false;          // GPD_PREC_FP64_SLICED_TRAIN: W's buffer holds FP64 shares and two sliced copies
    double tau_col = 0, tau_in = 0;
    std::vector<double> points;
    bool points_symmetric = false;   // b_{P-1-p} = -b_p exactly (always so for the built-in Chebyshev points)
    bool alt_subst = false;          // GPD_SUBST_V_EQ_UM: the exponent of W's block (i, j) is i + m j instead of n i + j
    std::vector<double> coefW, coefX, coefDT, coefDup, coefXup;   // [P][blocks]
    gpd::ProductInfo prod[4];    // indexed by gpd_product (GPD_UPD unused)
    // device side
    std::mutex mu;
    bool uploaded = false;
    int device = -1;
    gpd::DeviceTables dev;
};

namespace gpd {

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// Uploads the plan's tables on first use (cudaMalloc + cudaMemcpy on the current device).
gpd_status ensure_device(gpd_plan_s* plan);

// Number of SMs of the current device (cached per device; 148 if the query fails).
inline int sm_count() {
    static int cache[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cache[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cache[dev] = n;
    }
    return cache[dev];
}

inline gpd_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? GPD_OK : GPD_ERR_CUDA; }
inline gpd_status launch_ok() { return cuda_ok(cudaGetLastError()); }

// Workspace layout for locate / decode (bytes, 256-aligned sections).
struct WorkspaceLayout {
    int64_t off_gram;      // double[kMaxR * kMaxR]   syndrome Gram matrix
    int64_t off_counts;    // unsigned long long[4]   n_active, nonfinite mask, spare
    int64_t off_decode;    // double[kMaxWanted * kMaxNodes] decode matrix D
    int64_t off_flags;     // int[8] decode gate, number of regenerated nodes
    int64_t off_regen;     // double[kMaxNodes * kMaxNodes] regeneration matrix
    int64_t total;
};
WorkspaceLayout workspace_layout();

// Entry points used by coded_layer_step and by the public wrappers (all asynchronous).
gpd_status encode_launch(gpd_plan_s* plan, int operand_or_A, const float* src, void* dst, cudaStream_t st);
gpd_status worker_gemm_launch(gpd_plan_s* plan, gpd_product which, const void* W_sh, const void* other,
                              void* out, cudaStream_t st);
gpd_status update_launch(gpd_plan_s* plan, void* W_sh, const void* Dhat, const void* Xhat, float eta,
                         float lambda, const gpd_locate_result* gate, cudaStream_t st);
gpd_status inject_launch(gpd_plan_s* plan, gpd_product which, void* outputs, uint64_t seed, int mode,
                         double prob, uint64_t node_mask, int count, double scale, uint64_t* hit_mask,
                         cudaStream_t st);
gpd_status locate_launch(gpd_plan_s* plan, gpd_product which, const void* outputs, uint64_t erased_mask,
                         gpd_locate_result* result, void* workspace, cudaStream_t st);
gpd_status locate_static_launch(gpd_plan_s* plan, gpd_product which, const void* outputs,
                                uint64_t erased_mask, gpd_locate_result* result, cudaStream_t st);
gpd_status regenerate_launch(gpd_plan_s* plan, void* shares, const gpd_locate_result* result, void* workspace,
                             cudaStream_t st);
gpd_status correct_positions_launch(gpd_plan_s* plan, gpd_product which, void* outputs, gpd_position_result* result,
                                    void* workspace, cudaStream_t st);
int64_t position_workspace_bytes(const gpd_plan_s* plan);
// Fills the plan's cache of error-free decoding matrices (called once, from the upload, on the default stream).
gpd_status decode_cache_fill(gpd_plan_s* plan);
gpd_status decode_launch(gpd_plan_s* plan, gpd_product which, const void* outputs, bool have_mask,
                         uint64_t use_mask, const gpd_locate_result* result, float* out, float* act_out,
                         int activation, void* workspace, cudaStream_t st);

}  // namespace gpd
