// Encoding: every share is a small linear combination of the blocks of the source matrix,
// share_p = sum_blocks coef[p][blk] * M_blk  (Eq. 1 / Eq. 3, Theorem 2's X~, the backpropagation
// and update encodings).  Bandwidth-bound: each source element is read once, all P shares of
// that element are produced from registers and streamed out with 16-byte stores.
#include "gpd_internal.h"
#include "slice_common.h"

namespace gpd {

namespace {

struct EncodeParams {
    const float* src;      // rows x cols, row-major
    void* dst;             // [P][br][bc]
    const double* coef;    // [P][nblk]
    int64_t cols;          // leading dimension of src
    int64_t br, bc;        // block rows / cols
    int gc;                // blocks per row of the grid
    int nblk;              // gr * gc
    int P;
};

template <typename T>
__device__ __forceinline__ void store4(T* p, double a, double b, double c, double d);
template <>
__device__ __forceinline__ void store4<float>(float* p, double a, double b, double c, double d) {
    __stcs(reinterpret_cast<float4*>(p), make_float4((float)a, (float)b, (float)c, (float)d));
}
template <>
__device__ __forceinline__ void store4<double>(double* p, double a, double b, double c, double d) {
    __stcs(reinterpret_cast<double2*>(p), make_double2(a, b));
    __stcs(reinterpret_cast<double2*>(p) + 1, make_double2(c, d));
}

// One thread: one group of 4 consecutive columns at one in-block position, all blocks, all shares.
template <typename T, int NBLK>
__global__ void __launch_bounds__(256) encode_vec4_kernel(EncodeParams prm) {
    extern __shared__ double s_coef[];                     // [P][NBLK]
    for (int i = threadIdx.x; i < prm.P * NBLK; i += blockDim.x) s_coef[i] = prm.coef[i];
    __syncthreads();
    const int64_t bc4 = prm.bc >> 2;
    const int64_t total = prm.br * bc4;
    const int64_t block_elems = prm.br * prm.bc;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = t / bc4;
        const int64_t c = (t - r * bc4) << 2;
        float4 x[NBLK];
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const int gi = b / prm.gc, gj = b - gi * prm.gc;
            const float* s = prm.src + (gi * prm.br + r) * prm.cols + gj * prm.bc + c;
            x[b] = __ldg(reinterpret_cast<const float4*>(s));
        }
        T* out = reinterpret_cast<T*>(prm.dst) + r * prm.bc + c;
        for (int p = 0; p < prm.P; ++p) {
            const double* cf = s_coef + p * NBLK;
            double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll
            for (int b = 0; b < NBLK; ++b) {
                const double k = cf[b];
                a0 = fma(k, (double)x[b].x, a0);
                a1 = fma(k, (double)x[b].y, a1);
                a2 = fma(k, (double)x[b].z, a2);
                a3 = fma(k, (double)x[b].w, a3);
            }
            store4<T>(out + p * block_elems, a0, a1, a2, a3);
        }
    }
}

// Fallback for block widths that are not a multiple of 4 or unusual block counts: one element
// per thread, coefficients from shared memory, blocks re-read per share (served by L1/L2).
template <typename T>
__global__ void __launch_bounds__(256) encode_scalar_kernel(EncodeParams prm) {
    extern __shared__ double s_coef[];
    for (int i = threadIdx.x; i < prm.P * prm.nblk; i += blockDim.x) s_coef[i] = prm.coef[i];
    __syncthreads();
    const int64_t total = prm.br * prm.bc;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = t / prm.bc;
        const int64_t c = t - r * prm.bc;
        T* out = reinterpret_cast<T*>(prm.dst) + t;
        for (int p = 0; p < prm.P; ++p) {
            double acc = 0.0;
            for (int b = 0; b < prm.nblk; ++b) {
                const int gi = b / prm.gc, gj = b - gi * prm.gc;
                acc = fma(s_coef[p * prm.nblk + b],
                          (double)__ldg(prm.src + (gi * prm.br + r) * prm.cols + gj * prm.bc + c), acc);
            }
            out[p * total] = (T)acc;
        }
    }
}

template <typename T, int NBLK>
void launch_vec4(const EncodeParams& prm, int grid, cudaStream_t st) {
    encode_vec4_kernel<T, NBLK><<<grid, 256, sizeof(double) * prm.P * NBLK, st>>>(prm);
}

template <typename T>
gpd_status dispatch(const EncodeParams& prm, cudaStream_t st) {
    const bool vec_ok = (prm.bc % 4 == 0) && (prm.cols % 4 == 0) &&
                        (reinterpret_cast<uintptr_t>(prm.src) % 16 == 0) &&
                        (reinterpret_cast<uintptr_t>(prm.dst) % 16 == 0);
    const int64_t work = vec_ok ? prm.br * (prm.bc / 4) : prm.br * prm.bc;
    int grid = (int)std::min<int64_t>((work + 255) / 256, sm_count() * 16);
    if (grid < 1) grid = 1;
    if (vec_ok) {
        switch (prm.nblk) {
            case 1: launch_vec4<T, 1>(prm, grid, st); return launch_ok();
            case 2: launch_vec4<T, 2>(prm, grid, st); return launch_ok();
            case 3: launch_vec4<T, 3>(prm, grid, st); return launch_ok();
            case 4: launch_vec4<T, 4>(prm, grid, st); return launch_ok();
            case 6: launch_vec4<T, 6>(prm, grid, st); return launch_ok();
            case 8: launch_vec4<T, 8>(prm, grid, st); return launch_ok();
            case 9: launch_vec4<T, 9>(prm, grid, st); return launch_ok();
            case 12: launch_vec4<T, 12>(prm, grid, st); return launch_ok();
            case 16: launch_vec4<T, 16>(prm, grid, st); return launch_ok();
            default: break;
        }
    }
    encode_scalar_kernel<T><<<grid, 256, sizeof(double) * prm.P * prm.nblk, st>>>(prm);
    return launch_ok();
}

}  // namespace

gpd_status encode_launch(gpd_plan_s* plan, int operand_or_A, const float* src, void* dst,
                         cudaStream_t st) {
    // digit-plane modes: operands are cut into planes by slice.cu; in the training mode W's shares are
    // first evaluated to FP64 at the start of their buffer (below), then both sliced copies are cut
    if (plan->sliced && !(plan->train && operand_or_A == -1)) return encode_sliced_launch(plan, operand_or_A, src, dst, st);
    gpd_status rc = ensure_device(plan);
    if (rc != GPD_OK) return rc;
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    EncodeParams prm{};
    prm.src = src;
    prm.dst = dst;
    prm.P = plan->P;
    int gr = 1;
    switch (operand_or_A) {
        case -1:                                            // W: m x n blocks
            gr = c.m; prm.gc = c.n; prm.cols = s.N0; prm.br = s.N1 / c.m; prm.bc = s.N0 / c.n;
            prm.coef = plan->dev.base + plan->dev.off_coefW; break;
        case GPD_OPERAND_X_FWD:                             // X: n x d1 blocks
            gr = c.n; prm.gc = c.d1; prm.cols = s.B; prm.br = s.N0 / c.n; prm.bc = s.B / c.d1;
            prm.coef = plan->dev.base + plan->dev.off_coefX; break;
        case GPD_OPERAND_DELTAT_BWD:                        // Delta^T: d2 x m blocks
            gr = c.d2; prm.gc = c.m; prm.cols = s.N1; prm.br = s.B / c.d2; prm.bc = s.N1 / c.m;
            prm.coef = plan->dev.base + plan->dev.off_coefDT; break;
        case GPD_OPERAND_DELTA_UPD:                         // Delta: m x 1 blocks
            gr = c.m; prm.gc = 1; prm.cols = s.B; prm.br = s.N1 / c.m; prm.bc = s.B;
            prm.coef = plan->dev.base + plan->dev.off_coefDup; break;
        case GPD_OPERAND_X_UPD:                             // X: n x 1 blocks
            gr = c.n; prm.gc = 1; prm.cols = s.B; prm.br = s.N0 / c.n; prm.bc = s.B;
            prm.coef = plan->dev.base + plan->dev.off_coefXup; break;
        default: return GPD_ERR_ARG;
    }
    prm.nblk = gr * prm.gc;
    rc = plan->elem_size == 4 ? dispatch<float>(prm, st) : dispatch<double>(prm, st);
    if (rc == GPD_OK && plan->train && operand_or_A == -1) rc = reslice_launch(plan, dst, st);
    return rc;
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_encode_A(gpd_plan_t plan, const float* W_dev, void* W_shares_dev,
                                   void* stream) {
    if (!plan || !W_dev || !W_shares_dev) return GPD_ERR_ARG;
    return encode_launch(plan, -1, W_dev, W_shares_dev, as_stream(stream));
}

extern "C" gpd_status gpd_encode_B(gpd_plan_t plan, gpd_operand operand, const float* src_dev,
                                   void* shares_dev, void* stream) {
    if (!plan || !src_dev || !shares_dev) return GPD_ERR_ARG;
    if (operand == GPD_OPERAND_DELTAT_BWD && plan->prod[GPD_BWD].Q == 0) return GPD_ERR_P_TOO_SMALL;
    return encode_launch(plan, (int)operand, src_dev, shares_dev, as_stream(stream));
}
