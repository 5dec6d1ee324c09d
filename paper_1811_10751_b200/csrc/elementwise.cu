// Element-wise steps of the training iteration (Section II-B: C1 activation, C2 Hadamard product
// with g(X), the last-layer transition; Section IX: the sparse-autoencoder terms).  All Theta(N B)
// work, done once on the GPU instead of redundantly at every node.
#include "gpd_internal.h"

namespace gpd {

namespace {

__device__ __forceinline__ float act(float v, int kind) {
    if (kind == GPD_ACT_RELU) return v > 0.f ? v : 0.f;
    if (kind == GPD_ACT_SIGMOID) return 1.f / (1.f + __expf(-v));
    return v;
}
// g with g(f(u)) = f'(u), evaluated on the activation output x = f(u)
__device__ __forceinline__ float act_g(float x, int kind) {
    if (kind == GPD_ACT_RELU) return x > 0.f ? 1.f : 0.f;
    if (kind == GPD_ACT_SIGMOID) return x * (1.f - x);
    return 1.f;
}

__global__ void activation_kernel(const float* in, float* out, int64_t n, int kind) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = act(in[i], kind);
}

__device__ __forceinline__ double block_sum(double v, double* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (warp == 0) {
        t = lane < (int)(blockDim.x >> 5) ? scratch[lane] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    }
    __syncthreads();
    return t;                                          // valid in warp 0
}

// One CTA; thread per sample column.  S is C x B (a column is one sample).
__global__ void __launch_bounds__(256) softmax_xent_kernel(const float* S, const int* labels, float* Delta,
                                                           float* DeltaT, float* loss, int64_t C, int64_t B) {
    __shared__ double scratch[8];
    double local = 0.0;
    const double invB = 1.0 / (double)B;
    for (int64_t b = threadIdx.x; b < B; b += blockDim.x) {
        double mx = -1e300;
        for (int64_t c = 0; c < C; ++c) mx = fmax(mx, (double)S[c * B + b]);
        double sum = 0.0;
        for (int64_t c = 0; c < C; ++c) sum += exp((double)S[c * B + b] - mx);
        const int y = labels[b];
        for (int64_t c = 0; c < C; ++c) {
            const double pr = exp((double)S[c * B + b] - mx) / sum;
            const float d = (float)(((c == y ? 1.0 : 0.0) - pr) * invB);
            if (Delta) Delta[c * B + b] = d;
            if (DeltaT) DeltaT[b * C + c] = d;
        }
        local += -((double)S[(int64_t)y * B + b] - mx - log(sum));
    }
    const double tot = block_sum(local, scratch);
    if (threadIdx.x == 0 && loss) *loss = (float)(tot * invB);
}

// Delta_prev[j][b] = CT[b][j] * g(X[j][b]); 32 x 32 tiles through shared memory so that both the
// N x B and the B x N outputs are written coalesced.
__global__ void __launch_bounds__(256) hadamard_kernel(const float* CT, const float* X, float* Delta,
                                                       float* DeltaT, int64_t N, int64_t B, int kind) {
    __shared__ float tile[32][33];
    const int64_t j0 = (int64_t)blockIdx.x * 32, b0 = (int64_t)blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;     // 32 x 8
    for (int r = ty; r < 32; r += 8) {                           // read CT[b0+r][j0+tx]
        const int64_t b = b0 + r, j = j0 + tx;
        tile[r][tx] = (b < B && j < N) ? CT[b * N + j] : 0.f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {                           // element (j0+r, b0+tx)
        const int64_t j = j0 + r, b = b0 + tx;
        if (j < N && b < B) {
            const float d = tile[tx][r] * act_g(X[j * B + b], kind);
            if (Delta) Delta[j * B + b] = d;
            tile[tx][r] = d;
        }
    }
    __syncthreads();
    if (DeltaT)
        for (int r = ty; r < 32; r += 8) {
            const int64_t b = b0 + r, j = j0 + tx;
            if (b < B && j < N) DeltaT[b * N + j] = tile[r][tx];
        }
}

// Delta2 = (2/B)(X - S2), its transpose, and (1/B) sum (S2 - X)^2 accumulated into *loss.
__global__ void __launch_bounds__(256) sae_output_kernel(const float* S2, const float* X, float* Delta,
                                                         float* DeltaT, float* loss, int64_t N, int64_t B) {
    __shared__ float tile[32][33];
    __shared__ double scratch[8];
    const int64_t i0 = (int64_t)blockIdx.x * 32, b0 = (int64_t)blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float k = 2.f / (float)B;
    double local = 0.0;
    for (int r = ty; r < 32; r += 8) {
        const int64_t i = i0 + r, b = b0 + tx;
        float d = 0.f;
        if (i < N && b < B) {
            const float diff = X[i * B + b] - S2[i * B + b];
            d = k * diff;
            local += (double)diff * (double)diff;
            if (Delta) Delta[i * B + b] = d;
        }
        tile[r][tx] = d;
    }
    __syncthreads();
    if (DeltaT)
        for (int r = ty; r < 32; r += 8) {
            const int64_t b = b0 + r, i = i0 + tx;
            if (b < B && i < N) DeltaT[b * N + i] = tile[tx][r];
        }
    const double tot = block_sum(local, scratch);
    if (threadIdx.x == 0 && loss) atomicAdd(loss, (float)(tot / (double)B));
}

// One CTA per 32 hidden units: rho_hat (row means of Y1), then
// Delta1[i][b] = (C2T[b][i] - (beta/B) Q(rho_hat_i)) * Y1 (1 - Y1), and the KL penalty.
__global__ void __launch_bounds__(256) sae_hidden_kernel(const float* C2T, const float* Y1, float rho,
                                                         float beta, float* Delta, float* DeltaT,
                                                         float* kl_loss, int64_t N, int64_t B) {
    __shared__ float tile[32][33];
    __shared__ double s_q[32];
    __shared__ double scratch[8];
    const int64_t i0 = (int64_t)blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    double kl_local = 0.0;
    for (int r = ty; r < 32; r += 8) {                           // warp ty sums rows r
        const int64_t i = i0 + r;
        double s = 0.0;
        if (i < N)
            for (int64_t b = tx; b < B; b += 32) s += (double)Y1[i * B + b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (tx == 0) {
            double rh = s / (double)B;
            rh = fmin(fmax(rh, 1e-7), 1.0 - 1e-7);
            s_q[r] = -(double)rho / rh + (1.0 - (double)rho) / (1.0 - rh);
            if (i < N)
                kl_local += (double)rho * log((double)rho / rh) +
                            (1.0 - (double)rho) * log((1.0 - (double)rho) / (1.0 - rh));
        }
    }
    __syncthreads();
    const double kb = (double)beta / (double)B;
    for (int64_t b0 = 0; b0 < B; b0 += 32) {
        for (int r = ty; r < 32; r += 8) {                       // C2T[b0+r][i0+tx]
            const int64_t b = b0 + r, i = i0 + tx;
            tile[r][tx] = (b < B && i < N) ? C2T[b * N + i] : 0.f;
        }
        __syncthreads();
        for (int r = ty; r < 32; r += 8) {                       // element (i0+r, b0+tx)
            const int64_t i = i0 + r, b = b0 + tx;
            if (i < N && b < B) {
                const float y = Y1[i * B + b];
                const float d = (float)(((double)tile[tx][r] - kb * s_q[r]) * (double)y * (1.0 - (double)y));
                if (Delta) Delta[i * B + b] = d;
                tile[tx][r] = d;
            }
        }
        __syncthreads();
        if (DeltaT)
            for (int r = ty; r < 32; r += 8) {
                const int64_t b = b0 + r, i = i0 + tx;
                if (b < B && i < N) DeltaT[b * N + i] = tile[r][tx];
            }
        __syncthreads();
    }
    const double tot = block_sum(kl_local, scratch);
    if (threadIdx.x == 0 && kl_loss) atomicAdd(kl_loss, (float)((double)beta * tot));
}

}  // namespace

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_activation(gpd_activation_kind kind, const float* S_dev, float* X_next_dev,
                                     int64_t count, void* stream) {
    if (!S_dev || !X_next_dev || count < 0) return GPD_ERR_ARG;
    if (count == 0) return GPD_OK;
    const int grid = (int)std::min<int64_t>((count + 255) / 256, sm_count() * 8);
    activation_kernel<<<grid, 256, 0, as_stream(stream)>>>(S_dev, X_next_dev, count, (int)kind);
    return launch_ok();
}

extern "C" gpd_status gpd_softmax_xent_delta(const float* S_dev, const int32_t* labels_dev, float* Delta_dev,
                                             float* DeltaT_dev, float* loss_dev, int64_t C, int64_t B,
                                             void* stream) {
    if (!S_dev || !labels_dev || C <= 0 || B <= 0) return GPD_ERR_ARG;
    softmax_xent_kernel<<<1, 256, 0, as_stream(stream)>>>(S_dev, labels_dev, Delta_dev, DeltaT_dev, loss_dev, C, B);
    return launch_ok();
}

extern "C" gpd_status gpd_backprop_hadamard(gpd_activation_kind kind, const float* CT_dev, const float* X_dev,
                                            float* Delta_dev, float* DeltaT_dev, int64_t N, int64_t B,
                                            void* stream) {
    if (!CT_dev || !X_dev || N <= 0 || B <= 0) return GPD_ERR_ARG;
    dim3 grid((unsigned)((N + 31) / 32), (unsigned)((B + 31) / 32));
    hadamard_kernel<<<grid, 256, 0, as_stream(stream)>>>(CT_dev, X_dev, Delta_dev, DeltaT_dev, N, B, (int)kind);
    return launch_ok();
}

extern "C" gpd_status gpd_sae_output_delta(const float* S2_dev, const float* X_dev, float* Delta2_dev,
                                           float* Delta2T_dev, float* loss_dev, int64_t N, int64_t B,
                                           void* stream) {
    if (!S2_dev || !X_dev || N <= 0 || B <= 0) return GPD_ERR_ARG;
    if (loss_dev && cudaMemsetAsync(loss_dev, 0, sizeof(float), as_stream(stream)) != cudaSuccess)
        return GPD_ERR_CUDA;
    dim3 grid((unsigned)((N + 31) / 32), (unsigned)((B + 31) / 32));
    sae_output_kernel<<<grid, 256, 0, as_stream(stream)>>>(S2_dev, X_dev, Delta2_dev, Delta2T_dev, loss_dev, N, B);
    return launch_ok();
}

extern "C" gpd_status gpd_sae_hidden_delta(const float* C2T_dev, const float* Y1_dev, float rho, float beta,
                                           float* Delta1_dev, float* Delta1T_dev, float* kl_loss_dev,
                                           int64_t N, int64_t B, void* stream) {
    if (!C2T_dev || !Y1_dev || N <= 0 || B <= 0) return GPD_ERR_ARG;
    if (kl_loss_dev && cudaMemsetAsync(kl_loss_dev, 0, sizeof(float), as_stream(stream)) != cudaSuccess)
        return GPD_ERR_CUDA;
    sae_hidden_kernel<<<(unsigned)((N + 31) / 32), 256, 0, as_stream(stream)>>>(
        C2T_dev, Y1_dev, rho, beta, Delta1_dev, Delta1T_dev, kl_loss_dev, N, B);
    return launch_ok();
}
