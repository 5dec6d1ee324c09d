// Worker products (steps O1, O2) and the coded update (step O3, Eq. 10): dispatch, plus the
// shape-agnostic CUDA-core kernels used for blocks the tensor-core paths do not take
// (matrix-vector products, 5-row blocks, dimensions that break 16-byte alignment).
#include "gemm_common.h"
#include "slice_common.h"

namespace gpd {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

// 64x64 output tile per CTA, 16x16 threads, 4x4 outputs per thread; FP32 data accumulates in
// FP32, FP64 data in FP64.  Every load and store is bounds-checked.
template <typename T>
__global__ void __launch_bounds__(256) gemm_generic_kernel(GemmParams prm) {
    if (prm.update && prm.gate && prm.gate->outcome == GPD_DECODE_FAILURE) return;
    __shared__ T As[TK][TM + 1];
    __shared__ T Bs[TK][TN + 1];
    const int p = blockIdx.z;
    const T* A = reinterpret_cast<const T*>(prm.A) + (int64_t)p * prm.M * prm.K;
    const T* B = reinterpret_cast<const T*>(prm.B) + (int64_t)p * prm.K * prm.N;
    T* C = reinterpret_cast<T*>(prm.C) + (int64_t)p * prm.M * prm.N;
    const int64_t m0 = (int64_t)blockIdx.y * TM, n0 = (int64_t)blockIdx.x * TN;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    T acc[4][4] = {};
    for (int64_t k0 = 0; k0 < prm.K; k0 += TK) {
        for (int i = threadIdx.x; i < TM * TK; i += 256) {          // A tile: k fastest in memory
            const int kk = i % TK, mm = i / TK;
            const int64_t gm = m0 + mm, gk = k0 + kk;
            As[kk][mm] = (gm < prm.M && gk < prm.K) ? A[gm * prm.K + gk] : T(0);
        }
        if (prm.b_kmajor) {
            for (int i = threadIdx.x; i < TN * TK; i += 256) {
                const int kk = i % TK, nn = i / TK;
                const int64_t gn = n0 + nn, gk = k0 + kk;
                Bs[kk][nn] = (gn < prm.N && gk < prm.K) ? B[gn * prm.K + gk] : T(0);
            }
        } else {
            for (int i = threadIdx.x; i < TN * TK; i += 256) {
                const int nn = i % TN, kk = i / TN;
                const int64_t gn = n0 + nn, gk = k0 + kk;
                Bs[kk][nn] = (gn < prm.N && gk < prm.K) ? B[gk * prm.N + gn] : T(0);
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            T a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t gm = m0 + ty * 4 + i;
        if (gm >= prm.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t gn = n0 + tx * 4 + j;
            if (gn >= prm.N) continue;
            T* c = C + gm * prm.N + gn;
            *c = prm.update ? (T)(prm.shrink * (double)*c + prm.eta * (double)acc[i][j]) : acc[i][j];
        }
    }
}

// Matrix-vector worker product (mini-batch 1): one warp per output row, FP64 accumulation,
// the node's coded vector is read through L1/L2.  Bandwidth-bound on the shares.
template <typename T>
__global__ void __launch_bounds__(256) gemv_kernel(GemmParams prm) {
    const int p = blockIdx.y;
    const T* A = reinterpret_cast<const T*>(prm.A) + (int64_t)p * prm.M * prm.K;
    const T* x = reinterpret_cast<const T*>(prm.B) + (int64_t)p * prm.K;
    T* y = reinterpret_cast<T*>(prm.C) + (int64_t)p * prm.M;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    constexpr int V = 16 / sizeof(T);
    const bool vec = (prm.K % V == 0) && (reinterpret_cast<uintptr_t>(A) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(x) % 16 == 0);
    for (int64_t row = warp; row < prm.M; row += nwarps) {
        const T* a = A + row * prm.K;
        double acc = 0.0;
        if (vec) {
            for (int64_t k = (int64_t)lane * V; k < prm.K; k += 32 * V) {
                if constexpr (sizeof(T) == 4) {
                    const float4 av = __ldcs(reinterpret_cast<const float4*>(a + k));
                    const float4 xv = __ldg(reinterpret_cast<const float4*>(x + k));
                    acc = fma((double)av.x, (double)xv.x, acc);
                    acc = fma((double)av.y, (double)xv.y, acc);
                    acc = fma((double)av.z, (double)xv.z, acc);
                    acc = fma((double)av.w, (double)xv.w, acc);
                } else {
                    const double2 av = __ldcs(reinterpret_cast<const double2*>(a + k));
                    const double2 xv = __ldg(reinterpret_cast<const double2*>(x + k));
                    acc = fma(av.x, xv.x, acc);
                    acc = fma(av.y, xv.y, acc);
                }
            }
        } else {
            for (int64_t k = lane; k < prm.K; k += 32) acc = fma((double)a[k], (double)x[k], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) y[row] = (T)acc;
    }
}

}  // namespace

gpd_status gemm_generic_launch(const GemmParams& prm, int elem_size, cudaStream_t st) {
    dim3 grid((unsigned)((prm.N + TN - 1) / TN), (unsigned)((prm.M + TM - 1) / TM), (unsigned)prm.P);
    if (elem_size == 4)
        gemm_generic_kernel<float><<<grid, 256, 0, st>>>(prm);
    else
        gemm_generic_kernel<double><<<grid, 256, 0, st>>>(prm);
    return launch_ok();
}

gpd_status gemv_launch(const GemmParams& prm, int elem_size, cudaStream_t st) {
    const int64_t warps_needed = prm.M;
    int blocks = (int)std::min<int64_t>((warps_needed + 7) / 8, sm_count() * 8 / std::max(1, std::min(prm.P, 8)));
    if (blocks < 1) blocks = 1;
    dim3 grid((unsigned)blocks, (unsigned)prm.P);
    if (elem_size == 4)
        gemv_kernel<float><<<grid, 256, 0, st>>>(prm);
    else
        gemv_kernel<double><<<grid, 256, 0, st>>>(prm);
    return launch_ok();
}

gpd_status worker_gemm_launch(gpd_plan_s* plan, gpd_product which, const void* W_sh, const void* other,
                              void* out, cudaStream_t st) {
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    if (plan->sliced) return gemm_sliced_launch(plan, which, W_sh, other, out, st);
    GemmParams prm{};
    prm.P = plan->P;
    prm.C = out;
    prm.shrink = 0.0;
    prm.eta = 1.0;
    if (which == GPD_FWD) {                     // S~_p = W~_p X~_p
        prm.A = W_sh; prm.B = other;
        prm.M = s.N1 / c.m; prm.K = s.N0 / c.n; prm.N = s.B / c.d1;
    } else if (which == GPD_BWD) {              // C~^T_p = Delta~^T_p W~_p
        if (plan->prod[GPD_BWD].Q == 0) return GPD_ERR_P_TOO_SMALL;
        prm.A = other; prm.B = W_sh;
        prm.M = s.B / c.d2; prm.K = s.N1 / c.m; prm.N = s.N0 / c.n;
    } else {
        return GPD_ERR_ARG;
    }
    prm.max_threshold = plan->prod[which].Q;
    if (prm.N == 1) return gemv_launch(prm, plan->elem_size, st);
    if (plan->elem_size == 8 && dgemm_mma_supported(prm)) return dgemm_mma_launch(prm, st);
    if (plan->elem_size == 4 && sgemm_3xtf32_supported(prm)) {
        const gpd_status rc = ensure_device(plan);       // the plan's allocation carries the split-contraction scratch
        if (rc != GPD_OK) return rc;
        prm.splitk_scratch = plan->dev.splitk;
        prm.splitk_bytes = plan->dev.splitk_bytes;
        return sgemm_3xtf32_launch(prm, st);
    }
    return gemm_generic_launch(prm, plan->elem_size, st);
}

gpd_status update_launch(gpd_plan_s* plan, void* W_sh, const void* Dhat, const void* Xhat, float eta,
                         float lambda, const gpd_locate_result* gate, cudaStream_t st) {
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    if (plan->sliced)
        return update_sliced_launch(plan, W_sh, Dhat, Xhat, 1.0 - (double)eta * (double)lambda, (double)eta, gate, st);
    GemmParams prm{};
    prm.P = plan->P;
    prm.A = Dhat; prm.B = Xhat; prm.C = W_sh;
    prm.M = s.N1 / c.m; prm.N = s.N0 / c.n; prm.K = s.B;
    prm.b_kmajor = 1;
    prm.update = 1;
    prm.shrink = 1.0 - (double)eta * (double)lambda;
    prm.eta = (double)eta;
    prm.gate = gate;
    if (plan->elem_size == 8 && dgemm_mma_supported(prm)) return dgemm_mma_launch(prm, st);
    if (plan->elem_size == 4 && sgemm_3xtf32_supported(prm)) return sgemm_3xtf32_launch(prm, st);
    return gemm_generic_launch(prm, plan->elem_size, st);
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_worker_gemm(gpd_plan_t plan, gpd_product which, const void* W_shares_dev,
                                      const void* other_shares_dev, void* outputs_dev, void* stream) {
    if (!plan || !W_shares_dev || !other_shares_dev || !outputs_dev) return GPD_ERR_ARG;
    return worker_gemm_launch(plan, which, W_shares_dev, other_shares_dev, outputs_dev, as_stream(stream));
}

extern "C" gpd_status gpd_update_shares(gpd_plan_t plan, void* W_shares_dev, const void* Dhat_dev,
                                        const void* Xhat_dev, float eta, float lambda,
                                        const gpd_locate_result* gate_dev, void* stream) {
    if (!plan || !W_shares_dev || !Dhat_dev || !Xhat_dev) return GPD_ERR_ARG;
    return update_launch(plan, W_shares_dev, Dhat_dev, Xhat_dev, eta, lambda, gate_dev, as_stream(stream));
}

extern "C" gpd_status gpd_selftest_bounded_wait(int64_t limit_cycles, void* stream) {
    const long long limit = std::max<long long>(1000, std::min<long long>(limit_cycles, 100000000LL));
    return bounded_wait_selftest_launch(limit, as_stream(stream));
}

extern "C" gpd_status gpd_device_status(int32_t* status_host) {
    if (!status_host) return GPD_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return GPD_ERR_CUDA;
    const int a = tf32_device_status_fetch_and_clear(), b = i8_device_status_fetch_and_clear();
    *status_host = a != 0 ? a : b;
    return GPD_OK;
}
