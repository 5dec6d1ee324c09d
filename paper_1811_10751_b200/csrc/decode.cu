// Decoding: interpolate the product polynomial from the evaluations of the nodes in use and
// keep the wanted coefficients (Theorem 2's proof; the Vandermonde system of the decoding
// appendix).  Done as one small FP64 factorisation followed by a bandwidth-bound streaming pass:
//
//   1. decode_matrix_kernel (one CTA): Householder QR of the |S| x Q Vandermonde matrix of the
//      nodes in use; row w of D = e_w^T R^-1 Q^T is the linear functional that reads coefficient
//      w of the least-squares polynomial off the node values.  Normal equations are never
//      formed (the Vandermonde matrix is too ill-conditioned for that at thresholds near 30).
//   2. decode_stream_kernel: out_block(w)[pos] = sum_p D[w][p] * Z[p][pos], each worker output
//      read once with 16-byte loads, FP64 accumulation, FP32 store into the right block of the
//      result; optional fused activation (step C1).
#include "gpd_internal.h"
#include "slice_common.h"

namespace gpd {

namespace {

struct MatrixParams {
    const double* points;            // [P]
    double* D;                       // [n_wanted][P]
    int* gate;                       // [0] = 1 if the stream kernel may run
    const gpd_locate_result* result; // used when have_mask == 0
    unsigned long long use_mask;
    int have_mask;
    int P, Q, n_wanted;
    int wanted[kMaxWanted];
    double* regen;                   // optional [n_flagged][P]: re-evaluation of the interpolated
                                     // polynomial at the flagged nodes' points (share regeneration)
    const double* cached;            // optional [n_wanted][P]: this kernel's D for "every node in use"
};

constexpr int kMatrixThreads = 256;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One CTA of 8 warps.  Factorisation: eight lanes per column (see the loop).  Rows of the
// pseudo-inverse: one warp per wanted coefficient, lanes over the entries of y (Q <= 32) and of x
// (rows <= 64, two per lane).
__global__ void __launch_bounds__(kMatrixThreads) decode_matrix_kernel(MatrixParams prm) {
    __shared__ double A[kMaxNodes][kMaxQ + 1];       // Vandermonde rows of the nodes in use -> R
    __shared__ double Vh[kMaxNodes][kMaxQ + 1];      // Householder vectors (column k = reflector k)
    __shared__ int node_of[kMaxNodes];
    __shared__ int s_rows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = prm.P, Q = prm.Q;
    if (tid < 32) {                                  // nodes in use, in increasing order (one warp, two ballots)
        bool ok = prm.have_mask ? true : prm.result->outcome != GPD_DECODE_FAILURE;
        int rows = 0;
        for (int base = 0; base < P; base += 32) {
            const int p = base + tid;
            bool use = false;
            if (p < P) use = prm.have_mask ? ((prm.use_mask >> p) & 1ULL) != 0ULL : prm.result->flagged[p] == 0;
            const unsigned int m = __ballot_sync(0xffffffffu, use);
            if (use) node_of[rows + __popc(m & ((1u << tid) - 1u))] = p;
            rows += __popc(m);
        }
        if (rows < Q) ok = false;                    // fewer clean nodes than the threshold
        if (tid == 0) {
            s_rows = ok ? rows : 0;
            prm.gate[0] = ok ? 1 : 0;
        }
    }
    __syncthreads();
    const int rows = s_rows;
    if (rows == P && prm.cached && !prm.regen) {     // the error-free case: the matrix was computed at upload
        for (int i = tid; i < prm.n_wanted * P; i += kMatrixThreads) prm.D[i] = prm.cached[i];
        return;
    }
    for (int i = tid; i < prm.n_wanted * P; i += kMatrixThreads) prm.D[i] = 0.0;
    if (rows == 0) return;
    for (int r = tid; r < rows; r += kMatrixThreads) {
        const double b = prm.points[node_of[r]];
        if (prm.regen) {
            // regeneration only needs the polynomial's values, not its monomial coefficients: the
            // Chebyshev basis T_c keeps this least-squares system well conditioned on [-1,1]
            double t0 = 1.0, t1 = b;
            for (int c = 0; c < Q; ++c) { A[r][c] = t0; const double t2 = 2.0 * b * t1 - t0; t0 = t1; t1 = t2; }
        } else {
            double acc = 1.0;
            for (int c = 0; c < Q; ++c) { A[r][c] = acc; acc *= b; }
        }
    }
    __syncthreads();
    // Householder triangularisation.  Eight lanes share a column (column = k + tid / 8, rows strided
    // by eight between them, partial sums met by three shuffles inside the group), so that a step
    // costs rows / 8 dependent operations instead of rows.  Within a step column k is only read:
    // the last warp stores the unit reflector (its own columns k + 28 .. k + 31 rarely exist, and
    // the first warp, which holds the columns every step has, is left with one branch), and R's
    // diagonal entry is put in after the barrier.  Row loops are unrolled to the largest trip
    // count (64 rows / 8 lanes) so that their loads go out together.
    const int part = tid & 7, colg = tid >> 3;           // kMatrixThreads / 8 = 32 >= Q columns
    constexpr int kTrips = kMaxNodes / 8;
    for (int k = 0; k < Q; ++k) {
        double vk[kTrips];                               // this lane's entries of column k (rows k + part + 8 j)
        double sigma = 0.0;
#pragma unroll
        for (int j = 0; j < kTrips; ++j) {
            const int r = k + part + 8 * j;
            vk[j] = r < rows ? A[r][k] : 0.0;
            sigma = fma(vk[j], vk[j], sigma);
        }
        sigma += __shfl_xor_sync(0xffffffffu, sigma, 1);
        sigma += __shfl_xor_sync(0xffffffffu, sigma, 2);
        sigma += __shfl_xor_sync(0xffffffffu, sigma, 4);     // same value in every group (same order of additions)
        const double akk = A[k][k];
        const double alpha = akk >= 0.0 ? -sqrt(sigma) : sqrt(sigma);
        const double inv_vnorm = rsqrt(fmax(sigma - 2.0 * alpha * akk + alpha * alpha, 1e-300));
        if (part == 0) vk[0] -= alpha;                   // v = a_k - alpha e_k (row k sits in lane 0, trip 0)
        const int c = k + colg;
        if (colg > 0 && c < Q) {
            double ac[kTrips];
            double dot = 0.0;
#pragma unroll
            for (int j = 0; j < kTrips; ++j) {
                const int r = k + part + 8 * j;
                ac[j] = r < rows ? A[r][c] : 0.0;
                dot = fma(vk[j], ac[j], dot);
            }
            const unsigned int gmask = 0xffu << (8 * (colg & 3));
            dot += __shfl_xor_sync(gmask, dot, 1);
            dot += __shfl_xor_sync(gmask, dot, 2);
            dot += __shfl_xor_sync(gmask, dot, 4);
            const double f = 2.0 * dot * inv_vnorm * inv_vnorm;
#pragma unroll
            for (int j = 0; j < kTrips; ++j) {
                const int r = k + part + 8 * j;
                if (r < rows) A[r][c] = fma(-f, vk[j], ac[j]);
            }
        }
        if (warp == kMatrixThreads / 32 - 1) {           // unit reflector, 32 lanes over the rows
#pragma unroll
            for (int j = 0; j < kMaxNodes / 32; ++j) {
                const int r = k + lane + 32 * j;
                if (r < rows) Vh[r][k] = (A[r][k] - (r == k ? alpha : 0.0)) * inv_vnorm;
            }
        }
        __syncthreads();
        if (tid == 0) A[k][k] = alpha;               // R's diagonal; nothing below reads column k again
    }
    __syncthreads();                                 // the last diagonal entry
    // row w of the pseudo-inverse: solve R^T y = e_w, then x = H_0 H_1 ... H_{Q-1} [y; 0]
    for (int wi = warp; wi < prm.n_wanted; wi += kMatrixThreads / 32) {
        const int w = prm.wanted[wi];
        double y = 0.0;                              // lane i keeps y_i
        const double rdiag = lane < Q ? 1.0 / A[lane][lane] : 0.0;
        for (int i = w; i < Q; ++i) {                // y_i = 0 for i < w
            const double s = warp_sum(lane < i ? A[lane][i] * y : 0.0);
            if (lane == i) y = ((i == w ? 1.0 : 0.0) - s) * rdiag;
        }
        double x0 = lane < Q ? y : 0.0, x1 = 0.0;    // x[lane], x[lane + 32]
        const bool in0 = lane < rows, in1 = lane + 32 < rows;
        for (int k = Q - 1; k >= 0; --k) {
            const double v0 = (in0 && lane >= k) ? Vh[lane][k] : 0.0, v1 = in1 ? Vh[lane + 32][k] : 0.0;
            const double dot2 = 2.0 * warp_sum(v0 * x0 + v1 * x1);
            x0 -= dot2 * v0;
            x1 -= dot2 * v1;
        }
        if (in0) prm.D[wi * P + node_of[lane]] = x0;
        if (in1) prm.D[wi * P + node_of[lane + 32]] = x1;
    }
    if (prm.regen) {
        // Regeneration (Section VI): node f's share is a polynomial of degree Q-1 evaluated at b_f.
        // With D[c][q] the functional giving its c-th Chebyshev coefficient from the clean nodes q,
        // share_f = sum_q (sum_c T_c(b_f) D[c][q]) share_q.  Needs n_wanted == Q, wanted[c] == c.
        __syncthreads();                             // D was written by other warps of this CTA
        int nf = 0;
        for (int f = 0; f < P; ++f) {
            if (!prm.result->flagged[f]) continue;
            const double b = prm.points[f];
            for (int q = tid; q < P; q += kMatrixThreads) {
                double acc = 0.0, t0 = 1.0, t1 = b;
                for (int c = 0; c < Q; ++c) {
                    acc = fma(t0, prm.D[c * P + q], acc);
                    const double t2 = 2.0 * b * t1 - t0; t0 = t1; t1 = t2;
                }
                prm.regen[nf * P + q] = acc;
            }
            ++nf;
        }
        if (tid == 0) prm.gate[1] = nf;
    }
}

struct StreamParams {
    const void* Z;             // [P][br*bc]
    const double* D;           // [n_wanted][P]
    const int* gate;
    float* out;                // result matrix, leading dimension ldo
    float* act_out;            // optional
    int64_t br, bc, ldo;
    int P, n_wanted, grid_cols;
    int activation;
};

__device__ __forceinline__ float apply_act(float v, int kind) {
    if (kind == GPD_ACT_RELU) return v > 0.f ? v : 0.f;
    if (kind == GPD_ACT_SIGMOID) return 1.f / (1.f + __expf(-v));
    return v;
}

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, double (&v)[4]) {
        const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};
template <> struct Vec<double> {
    static constexpr int N = 2;
    __device__ static void load(const double* p, double (&v)[2]) {
        const double2 t = __ldcs(reinterpret_cast<const double2*>(p));
        v[0] = t.x; v[1] = t.y;
    }
};

// NW wanted coefficients per pass over the inputs; VECTOR: 16-byte loads of N positions.
// Shared memory: the columns of D of the nodes in use, compacted and transposed to [node][wanted]
// (padded to a multiple of NW) so that a node's NW coefficients come with 16-byte loads, and the
// nodes' element offsets into Z.
template <typename T, int NW, bool VECTOR>
__global__ void __launch_bounds__(256) decode_stream_kernel(StreamParams prm) {
    if (prm.gate[0] == 0) return;
    extern __shared__ __align__(16) double sD[];     // [n_used][WP]
    __shared__ int64_t s_off[kMaxNodes];             // node * L for the nodes in use
    __shared__ int s_nodes[kMaxNodes];
    __shared__ int s_nused;
    const int64_t L = prm.br * prm.bc;
    const int WP = (prm.n_wanted + NW - 1) / NW * NW;
    if (threadIdx.x < 32) {                          // nodes with an all-zero column of D are not read
        int n = 0;
        for (int base = 0; base < prm.P; base += 32) {
            const int p = base + (int)threadIdx.x;
            bool used = false;
            if (p < prm.P)
                for (int w = 0; w < prm.n_wanted; ++w) used |= prm.D[w * prm.P + p] != 0.0;
            const unsigned int m = __ballot_sync(0xffffffffu, used);
            if (used) {
                const int slot = n + __popc(m & ((1u << threadIdx.x) - 1u));
                s_nodes[slot] = p;
                s_off[slot] = (int64_t)p * L;
            }
            n += __popc(m);
        }
        if (threadIdx.x == 0) s_nused = n;
    }
    __syncthreads();
    const int nused = s_nused;
    for (int i = threadIdx.x; i < nused * WP; i += blockDim.x) {
        const int node = i / WP, w = i - node * WP;
        sD[i] = w < prm.n_wanted ? prm.D[w * prm.P + s_nodes[node]] : 0.0;
    }
    __syncthreads();
    constexpr int N = VECTOR ? Vec<T>::N : 1;
    constexpr int U = 6;                             // nodes per trip, loads issued first
    const T* Z = reinterpret_cast<const T*>(prm.Z);
    const int64_t groups = VECTOR ? L / N : L;
    for (int64_t gidx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; gidx < groups;
         gidx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t pos = gidx * N;
        const int64_t row = pos / prm.bc, col = pos - row * prm.bc;
        const T* zpos = Z + pos;
        for (int w0 = 0; w0 < prm.n_wanted; w0 += NW) {
            double acc[NW][N];
#pragma unroll
            for (int w = 0; w < NW; ++w)
#pragma unroll
                for (int v = 0; v < N; ++v) acc[w][v] = 0.0;
            auto fetch = [&](int i, double (&z)[N]) {
                if constexpr (VECTOR) Vec<T>::load(zpos + s_off[i], z);
                else z[0] = (double)__ldcs(zpos + s_off[i]);
            };
            auto absorb = [&](int i, const double (&z)[N]) {
                const double* d = sD + i * WP + w0;  // NW coefficients, 16-byte aligned (NW is even)
#pragma unroll
                for (int w = 0; w < NW; w += 2) {
                    const double2 dv = *reinterpret_cast<const double2*>(d + w);
#pragma unroll
                    for (int v = 0; v < N; ++v) {
                        acc[w][v] = fma(dv.x, z[v], acc[w][v]);
                        acc[w + 1][v] = fma(dv.y, z[v], acc[w + 1][v]);
                    }
                }
            };
            int i0 = 0;
            for (; i0 + U <= nused; i0 += U) {
                double z[U][N];
#pragma unroll
                for (int u = 0; u < U; ++u) fetch(i0 + u, z[u]);
#pragma unroll
                for (int u = 0; u < U; ++u) absorb(i0 + u, z[u]);
            }
            if (i0 < nused) {                        // the last n_used mod U nodes
                double z[U][N];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (i0 + u < nused) fetch(i0 + u, z[u]);
                    else
#pragma unroll
                        for (int v = 0; v < N; ++v) z[u][v] = 0.0;
                }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (i0 + u < nused) absorb(i0 + u, z[u]);
            }
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const int wi = w0 + w;
                if (wi >= prm.n_wanted) break;
                const int gr = wi / prm.grid_cols, gc = wi - gr * prm.grid_cols;
                const int64_t o = (gr * prm.br + row) * prm.ldo + gc * prm.bc + col;
                if constexpr (VECTOR && N == 4) {
                    const float4 v = make_float4((float)acc[w][0], (float)acc[w][1], (float)acc[w][2], (float)acc[w][3]);
                    *reinterpret_cast<float4*>(prm.out + o) = v;
                    if (prm.act_out)
                        *reinterpret_cast<float4*>(prm.act_out + o) =
                            make_float4(apply_act(v.x, prm.activation), apply_act(v.y, prm.activation),
                                        apply_act(v.z, prm.activation), apply_act(v.w, prm.activation));
                } else if constexpr (VECTOR && N == 2) {
                    const float2 v = make_float2((float)acc[w][0], (float)acc[w][1]);
                    *reinterpret_cast<float2*>(prm.out + o) = v;
                    if (prm.act_out)
                        *reinterpret_cast<float2*>(prm.act_out + o) =
                            make_float2(apply_act(v.x, prm.activation), apply_act(v.y, prm.activation));
                } else {
                    prm.out[o] = (float)acc[w][0];
                    if (prm.act_out) prm.act_out[o] = apply_act((float)acc[w][0], prm.activation);
                }
            }
        }
    }
}

template <typename T, int NW, bool VECTOR>
void launch_stream(const StreamParams& prm, cudaStream_t st) {
    constexpr int N = VECTOR ? Vec<T>::N : 1;
    const int64_t groups = prm.br * prm.bc / N;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((groups + 255) / 256, sm_count() * 4));
    const int WP = (prm.n_wanted + NW - 1) / NW * NW;
    decode_stream_kernel<T, NW, VECTOR><<<grid, 256, sizeof(double) * WP * prm.P, st>>>(prm);
}

template <typename T>
gpd_status dispatch_stream(const StreamParams& prm, cudaStream_t st) {
    constexpr int N = Vec<T>::N;
    const bool vec = (prm.bc % N == 0) && (prm.ldo % N == 0) &&
                     (reinterpret_cast<uintptr_t>(prm.Z) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(prm.out) % 16 == 0) &&
                     (!prm.act_out || reinterpret_cast<uintptr_t>(prm.act_out) % 16 == 0) &&
                     ((prm.br * prm.bc) % N == 0);
    if (vec) {
        if (prm.n_wanted <= 4) launch_stream<T, 4, true>(prm, st);
        else if (prm.n_wanted <= 8) launch_stream<T, 8, true>(prm, st);
        else launch_stream<T, 16, true>(prm, st);
    } else {
        if (prm.n_wanted <= 4) launch_stream<T, 4, false>(prm, st);
        else launch_stream<T, 16, false>(prm, st);
    }
    return launch_ok();
}

}  // namespace

gpd_status decode_cache_fill(gpd_plan_s* plan) {
    for (int w : {GPD_FWD, GPD_BWD, GPD_AUDIT}) {
        const ProductInfo& pi = plan->prod[w];
        if (pi.Q == 0 || plan->dev.off_dcache[w] < 0) continue;
        MatrixParams mp{};
        mp.points = plan->dev.base + plan->dev.off_points;
        mp.D = plan->dev.base + plan->dev.off_dcache[w];
        mp.gate = reinterpret_cast<int*>(plan->dev.base + plan->dev.off_dcache_gate);
        mp.use_mask = plan->P >= 64 ? ~0ULL : ((1ULL << plan->P) - 1ULL);
        mp.have_mask = 1;
        mp.P = plan->P; mp.Q = pi.Q; mp.n_wanted = pi.grid_rows * pi.grid_cols;
        for (int i = 0; i < mp.n_wanted; ++i) mp.wanted[i] = pi.wanted[i];
        decode_matrix_kernel<<<1, kMatrixThreads>>>(mp);
        if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
    }
    return GPD_OK;
}

gpd_status decode_launch(gpd_plan_s* plan, gpd_product which, const void* outputs, bool have_mask,
                         uint64_t use_mask, const gpd_locate_result* result, float* out, float* act_out,
                         int activation, void* workspace, cudaStream_t st) {
    if (which != GPD_FWD && which != GPD_BWD && which != GPD_AUDIT) return GPD_ERR_ARG;
    // digit-plane shares: forward product only, except in the training mode (its backward outputs and the
    // FP64 shares that lead W's buffer are plain doubles)
    if (plan->sliced && !plan->train && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;
    const ProductInfo& pi = plan->prod[which];
    if (pi.Q == 0) return GPD_ERR_P_TOO_SMALL;
    gpd_status rc = ensure_device(plan);
    if (rc != GPD_OK) return rc;
    const WorkspaceLayout wl = workspace_layout();
    char* ws = reinterpret_cast<char*>(workspace);
    MatrixParams mp{};
    mp.points = plan->dev.base + plan->dev.off_points;
    mp.D = reinterpret_cast<double*>(ws + wl.off_decode);
    mp.gate = reinterpret_cast<int*>(ws + wl.off_flags);
    mp.result = result;
    mp.use_mask = use_mask;
    mp.have_mask = have_mask ? 1 : 0;
    mp.P = plan->P; mp.Q = pi.Q; mp.n_wanted = pi.grid_rows * pi.grid_cols;
    for (int i = 0; i < mp.n_wanted; ++i) mp.wanted[i] = pi.wanted[i];
    mp.cached = plan->dev.off_dcache[which] >= 0 ? plan->dev.base + plan->dev.off_dcache[which] : nullptr;
    decode_matrix_kernel<<<1, kMatrixThreads, 0, st>>>(mp);
    rc = launch_ok();
    if (rc != GPD_OK) return rc;
    StreamParams sp{};
    sp.Z = outputs; sp.D = mp.D; sp.gate = mp.gate; sp.out = out; sp.act_out = act_out;
    sp.br = pi.br; sp.bc = pi.bc; sp.ldo = pi.bc * pi.grid_cols;
    sp.P = plan->P; sp.n_wanted = mp.n_wanted; sp.grid_cols = pi.grid_cols;
    sp.activation = activation;
    return plan->elem_size == 4 ? dispatch_stream<float>(sp, st) : dispatch_stream<double>(sp, st);
}

namespace {

struct RegenParams {
    void* shares;                    // [P][L] in/out
    const double* Rg;                // [n_flagged][P], zero columns for flagged nodes
    const int* gate;                 // [0] run?, [1] n_flagged
    const gpd_locate_result* result;
    int64_t L;
    int P;
};

// share_f[pos] = sum over clean q of Rg[f][q] * share_q[pos]; clean shares are read once, flagged
// shares are overwritten in place (the two sets are disjoint, so in-place is safe).
template <typename T>
__global__ void __launch_bounds__(256) regen_stream_kernel(RegenParams prm) {
    if (prm.gate[0] == 0 || prm.gate[1] == 0) return;
    extern __shared__ double sR[];                   // [n_flagged][P]
    __shared__ int s_flag[kMaxNodes], s_clean[kMaxNodes];
    __shared__ int s_nf, s_nc;
    if (threadIdx.x == 0) {
        int nf = 0, nc = 0;
        for (int p = 0; p < prm.P; ++p) {
            if (prm.result->flagged[p]) s_flag[nf++] = p; else s_clean[nc++] = p;
        }
        s_nf = nf; s_nc = nc;
    }
    __syncthreads();
    const int nf = s_nf, nc = s_nc;
    for (int i = threadIdx.x; i < nf * prm.P; i += blockDim.x) sR[i] = prm.Rg[i];
    __syncthreads();
    T* S = reinterpret_cast<T*>(prm.shares);
    for (int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; pos < prm.L;
         pos += (int64_t)gridDim.x * blockDim.x) {
        for (int f0 = 0; f0 < nf; f0 += 4) {
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            for (int i = 0; i < nc; ++i) {
                const int q = s_clean[i];
                const double z = (double)__ldcs(S + (int64_t)q * prm.L + pos);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (f0 + u < nf) acc[u] = fma(sR[(f0 + u) * prm.P + q], z, acc[u]);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (f0 + u < nf) S[(int64_t)s_flag[f0 + u] * prm.L + pos] = (T)acc[u];
        }
    }
}

}  // namespace

gpd_status regenerate_launch(gpd_plan_s* plan, void* shares, const gpd_locate_result* result, void* workspace,
                             cudaStream_t st) {
    const ProductInfo& pi = plan->prod[GPD_AUDIT];
    if (pi.Q == 0 || (plan->sliced && !plan->train)) return GPD_ERR_UNSUPPORTED;
    gpd_status rc = ensure_device(plan);
    if (rc != GPD_OK) return rc;
    const WorkspaceLayout wl = workspace_layout();
    char* ws = reinterpret_cast<char*>(workspace);
    MatrixParams mp{};
    mp.points = plan->dev.base + plan->dev.off_points;
    mp.D = reinterpret_cast<double*>(ws + wl.off_decode);
    mp.gate = reinterpret_cast<int*>(ws + wl.off_flags);
    mp.result = result;
    mp.have_mask = 0;
    mp.P = plan->P; mp.Q = pi.Q; mp.n_wanted = pi.Q;
    for (int c = 0; c < pi.Q; ++c) mp.wanted[c] = c;
    mp.regen = reinterpret_cast<double*>(ws + wl.off_regen);
    decode_matrix_kernel<<<1, kMatrixThreads, 0, st>>>(mp);
    if ((rc = launch_ok()) != GPD_OK) return rc;
    RegenParams rp{};
    rp.shares = shares; rp.Rg = mp.regen; rp.gate = mp.gate; rp.result = result;
    rp.L = pi.br * pi.bc; rp.P = plan->P;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((rp.L + 255) / 256, sm_count() * 8));
    const size_t smem = sizeof(double) * (size_t)plan->P * plan->P;
    if (plan->elem_size == 4) regen_stream_kernel<float><<<grid, 256, smem, st>>>(rp);
    else regen_stream_kernel<double><<<grid, 256, smem, st>>>(rp);
    if ((rc = launch_ok()) != GPD_OK) return rc;
    // training mode: the regenerated FP64 shares lead the buffer; the sliced copies follow them
    return plan->train ? reslice_launch(plan, shares, st) : GPD_OK;
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_decode(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                                 const uint8_t* use_mask_host, const gpd_locate_result* result_dev,
                                 float* out_dev, float* act_out_dev, gpd_activation_kind activation,
                                 void* workspace_dev, void* stream) {
    if (!plan || !outputs_dev || !out_dev) return GPD_ERR_ARG;
    if (!use_mask_host && !result_dev) return GPD_ERR_ARG;
    if (!workspace_dev) return GPD_ERR_WORKSPACE;
    uint64_t mask = 0;
    if (use_mask_host) {
        int n = 0;
        for (int p = 0; p < plan->P; ++p)
            if (use_mask_host[p]) { mask |= 1ULL << p; ++n; }
        if (which >= 0 && which <= GPD_AUDIT && which != GPD_UPD && n < plan->prod[which].Q)
            return GPD_ERR_P_TOO_SMALL;
    }
    return decode_launch(plan, which, outputs_dev, use_mask_host != nullptr, mask, result_dev, out_dev,
                         act_out_dev, (int)activation, workspace_dev, as_stream(stream));
}

extern "C" gpd_status gpd_regenerate_shares(gpd_plan_t plan, void* W_shares_dev, const gpd_locate_result* result_dev,
                                            void* workspace_dev, void* stream) {
    if (!plan || !W_shares_dev || !result_dev) return GPD_ERR_ARG;
    if (!workspace_dev) return GPD_ERR_WORKSPACE;
    return regenerate_launch(plan, W_shares_dev, result_dev, workspace_dev, as_stream(stream));
}
