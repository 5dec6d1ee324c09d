// Encoding for the integer-slice product paths (GPD_PREC_FP64_SLICED, GPD_PREC_FP64_SLICED40).
//
// The shares W~_p (Eq. 1) and X~_p (Theorem 2) are evaluated in FP64 exactly as in encode.cu, but
// instead of being stored as doubles each value a is stored as S = 6 (or 5) signed 8-bit digits:
//     a = 2^e * sum_{t=0..S-1} d_t * 256^-(t+1)  (+ remainder below 2^(e - 8 S - 1)),   d_t in [-128, 127],
// with one exponent e per row of W~_p (per column of X~_p) chosen so that |a| < 0.4923 * 2^e (from
// a bound of the row's magnitudes for W~_p, from the column's largest magnitude for X~_p).  The
// digits of one operand form S int8 planes; products of planes are exact in int32 on the tensor
// cores (gemm_i8.cu), which gives FP64-class worker products at integer-tensor-core speed.
// Both operands are written K-major: W planes [S][P][M][K], X planes [S][P][N][K] (transposed).
// Layout of a sliced share buffer: planes, then the int32 exponents, then encoder scratch.
#include <cmath>

#include "gpd_internal.h"
#include "slice_common.h"

namespace gpd {

namespace {

struct SliceParams {
    const float* src;      // source matrix, row-major, leading dimension ld
    const double* coef;    // [P][nblk]
    int8_t* planes;        // [S][P][R][K]   (R = rows of the K-major operand)
    int* expo;             // [P][R]
    unsigned int* amax;    // [P][R] scratch of the X side: largest |value| per operand row (high word)
    int64_t ld;            // leading dimension of src
    int64_t br, bc;        // block rows / cols of src
    int gc, nblk, P;
    // W only: the share of node p is a polynomial of degree nblk - 1 in its point b_p, and the points come
    // in pairs b_{P-1-p} = -b_p.  blk_of_exp[e] is the block whose coefficient is b_p^e.
    bool poly;
    int blk_of_exp[16];
};

// Largest magnitudes are tracked as the high 32 bits of |a| (non-negative doubles order like
// their bit patterns); hi + 1 with a zero low word is an upper bound within 2^-20 relative.
__device__ __forceinline__ unsigned int abs_hi(double a) { return (unsigned int)__double2hiint(a) & 0x7FFFFFFFu; }
__device__ __forceinline__ unsigned int abs_hi_max4(const double (&a)[4]) {
    return max(max(abs_hi(a[0]), abs_hi(a[1])), max(abs_hi(a[2]), abs_hi(a[3])));
}

// Exponent e such that every |a| <= amax has |a| 2^-e < 0.4923, which keeps the biased fixed-point
// value of digits4() inside 8 S bits; amax is given by its high word as above.  Magnitudes below
// 2^-900 (and non-finite ones) get the marker -1000: all digits zero.
__device__ __forceinline__ int slice_exponent(unsigned int amax_hi) {
    if (amax_hi < 0x07B00000u || amax_hi >= 0x7FF00000u) return -1000;
    const double amax = __hiloint2double((int)(amax_hi + 1u), 0);
    int x;
    frexp(amax * 1.015625, &x);   // amax (1 + 1/64) = f 2^x, f in [0.5, 1)
    return x + 1;
}
// 2^(8 S - e) as a double, 0 for the all-zero marker
template <int S>
__device__ __forceinline__ double slice_scale(int e) {
    if (e <= -1000) return 0.0;
    return __longlong_as_double((long long)(8 * S - e + 1023) << 52);
}

// Digits of four values at once.  U = rint(a 2^(8S-e)) + sum_i 128 * 256^i lies in [0, 2^(8S));
// its bytes minus 128 (= bytes with the top bit flipped) are the digits, most significant first.
// U is read from the mantissa of a 2^(8S-e) + 2^52 + bias (one FMA); word[t] holds digit t of
// values 0..3 in bytes 0..3.  A zero scale gives zero digits for finite a.
template <int S>
__device__ __forceinline__ void digits4(const double (&a)[4], double scale, unsigned int (&word)[S]) {
    // 2^52 + 128 (256^S - 1) / 255
    const double magic = S == 6 ? 4503599627370496.0 + 141289400074368.0 : 4503599627370496.0 + 551911719040.0;
    unsigned int lo[4], hi[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const double t = fma(a[v], scale, magic);
        lo[v] = (unsigned int)__double2loint(t);
        hi[v] = (unsigned int)__double2hiint(t);
    }
    // 4 x 4 byte transposes in two rounds of permutes: pairs of values first, then pairs of pairs
    unsigned int byte_of[8];                                          // byte i of U for values 0..3
    const unsigned int l01a = __byte_perm(lo[0], lo[1], 0x5140), l23a = __byte_perm(lo[2], lo[3], 0x5140);
    const unsigned int l01b = __byte_perm(lo[0], lo[1], 0x7362), l23b = __byte_perm(lo[2], lo[3], 0x7362);
    byte_of[0] = __byte_perm(l01a, l23a, 0x5410); byte_of[1] = __byte_perm(l01a, l23a, 0x7632);
    byte_of[2] = __byte_perm(l01b, l23b, 0x5410); byte_of[3] = __byte_perm(l01b, l23b, 0x7632);
    const unsigned int h01 = __byte_perm(hi[0], hi[1], 0x5140), h23 = __byte_perm(hi[2], hi[3], 0x5140);
    byte_of[4] = __byte_perm(h01, h23, 0x5410); byte_of[5] = __byte_perm(h01, h23, 0x7632);
    byte_of[6] = byte_of[7] = 0u;                                     // S <= 6
#pragma unroll
    for (int t = 0; t < S; ++t) word[t] = byte_of[S - 1 - t] ^ 0x80808080u;   // digit t sits in byte S-1-t
}

// ---- W side: operand rows are rows of the share (K = block columns, contiguous in the source) ----
// Pass 1: one CTA per share row r.  The scale of W~_p[r][:] comes from the bound
//     max_c |W~_p[r][c]| <= sum_b |coef_pb| max_c |W_b[r][c]|,
// which needs one streaming pass over W and no evaluation of the shares; it overestimates the true
// maximum by the cancellation between blocks (a factor below the number of blocks, about 3 for
// eight Gaussian blocks), i.e. it spends one to two of the 8 S bits.
template <int NBLK>
__global__ void __launch_bounds__(256) rowscale_kernel(SliceParams prm) {
    __shared__ unsigned int sBlk[NBLK];          // bit patterns of non-negative floats order like integers
    if (threadIdx.x < NBLK) sBlk[threadIdx.x] = 0u;
    __syncthreads();
    const int64_t r = blockIdx.x;
    const int lane = threadIdx.x & 31;
    unsigned int m[NBLK];
#pragma unroll
    for (int b = 0; b < NBLK; ++b) m[b] = 0u;
    for (int64_t c = (int64_t)threadIdx.x * 4; c < prm.bc; c += 1024) {
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const int gi = b / prm.gc, gj = b - gi * prm.gc;
            const float4 v = __ldg(reinterpret_cast<const float4*>(prm.src + (gi * prm.br + r) * prm.ld + gj * prm.bc + c));
            m[b] = max(m[b], max(max(__float_as_uint(fabsf(v.x)), __float_as_uint(fabsf(v.y))),
                                 max(__float_as_uint(fabsf(v.z)), __float_as_uint(fabsf(v.w)))));
        }
    }
#pragma unroll
    for (int b = 0; b < NBLK; ++b) {             // all 32 lanes are here: the column loop has ended
        const unsigned int w = __reduce_max_sync(0xffffffffu, m[b]);
        if (lane == 0) atomicMax(&sBlk[b], w);
    }
    __syncthreads();
    for (int p = threadIdx.x; p < prm.P; p += 256) {
        double bound = 0.0;
        for (int b = 0; b < NBLK; ++b) bound += fabs(prm.coef[p * NBLK + b]) * (double)__uint_as_float(sBlk[b]);
        prm.expo[(int64_t)p * prm.br + r] = slice_exponent(abs_hi(bound));
    }
}

// Pass 2: one thread per 4 consecutive columns of a share row: recompute the share values in FP64,
// cut them into digits with the row's exponent, store 4 digits (one 32-bit word) per plane.
template <int NBLK, int S>
__global__ void __launch_bounds__(256) rowslice_kernel(SliceParams prm) {
    extern __shared__ double s_coef[];
    for (int i = threadIdx.x; i < prm.P * NBLK; i += 256) s_coef[i] = prm.coef[i];
    __syncthreads();
    const int64_t bc4 = prm.bc >> 2, total = prm.br * bc4;
    const int64_t plane_stride = (int64_t)prm.P * prm.br * prm.bc, node_stride = prm.br * prm.bc;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < total; t += (int64_t)gridDim.x * 256) {
        const int64_t r = t / bc4, c = (t - r * bc4) << 2;
        double x[NBLK][4];                       // converted once, used by every node
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const int gi = b / prm.gc, gj = b - gi * prm.gc;
            const float4 v = __ldg(reinterpret_cast<const float4*>(prm.src + (gi * prm.br + r) * prm.ld + gj * prm.bc + c));
            x[b][0] = v.x; x[b][1] = v.y; x[b][2] = v.z; x[b][3] = v.w;
        }
        int8_t* dst = prm.planes + r * prm.bc + c;
        const int* ex = prm.expo + r;
#pragma unroll 2
        for (int p = 0; p < prm.P; ++p, dst += node_stride, ex += prm.br) {
            const double* cf = s_coef + p * NBLK;
            double a[4] = {0, 0, 0, 0};
#pragma unroll
            for (int b = 0; b < NBLK; ++b) {
                const double k = cf[b];
                a[0] = fma(k, x[b][0], a[0]); a[1] = fma(k, x[b][1], a[1]);
                a[2] = fma(k, x[b][2], a[2]); a[3] = fma(k, x[b][3], a[3]);
            }
            unsigned int word[S];
            digits4<S>(a, slice_scale<S>(__ldg(ex)), word);
#pragma unroll
            for (int s = 0; s < S; ++s)
                __stcs(reinterpret_cast<unsigned int*>(dst + s * plane_stride), word[s]);
        }
    }
}

// Both passes in one kernel, for share rows whose source values (NBLK block rows of bc floats) fit
// in shared memory twice.  A persistent CTA walks share rows r; while it works on row r the source
// values of its next row arrive through asynchronous 16-byte copies, so that no thread waits on
// global memory inside the node loop and W is read from DRAM once.  Per row: block maxima from
// shared memory -> the P exponents of the row (same bound as rowscale_kernel) -> digits.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const unsigned int s = (unsigned int)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;\n" ::: "memory"); }

constexpr int kFusedMaxThreads = 512;
// shared memory of the fused kernel: coefficients, per-node scales, block maxima (two sets), two row buffers
inline size_t fused_smem_bytes(int P, int nblk, int64_t bc) {
    const size_t head = (sizeof(double) * ((size_t)P * nblk + P) + sizeof(unsigned int) * 2 * nblk + 15) / 16 * 16;
    return head + 2 * sizeof(float) * (size_t)nblk * (size_t)bc;
}

template <int NBLK, int S, bool POLY>
__global__ void __launch_bounds__(kFusedMaxThreads, 1) rowslice_fused_kernel(SliceParams prm) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    const int P = prm.P, tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
    double* s_cf = reinterpret_cast<double*>(s_raw);                       // [P][NBLK]
    double* s_scale = s_cf + P * NBLK;                                     // [P]  2^(8S - e_p) of the current row
    unsigned int* s_blk = reinterpret_cast<unsigned int*>(s_scale + P);    // [2][NBLK] largest |W_b[r][:]| as float bits
    const int64_t bc = prm.bc;
    const int bc4 = (int)(bc >> 2);
    float* stage = reinterpret_cast<float*>(s_raw + (sizeof(double) * ((size_t)P * NBLK + P) +
                                                     sizeof(unsigned int) * 2 * NBLK + 15) / 16 * 16);   // [2][NBLK][bc]
    for (int i = tid; i < P * NBLK; i += nthr) s_cf[i] = prm.coef[i];
    if (tid < 2 * NBLK) s_blk[tid] = 0u;

    auto fetch = [&](int64_t r, int buf) {
        float* d = stage + (size_t)buf * NBLK * bc;
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const int gi = b / prm.gc, gj = b - gi * prm.gc;
            const float* srow = prm.src + (gi * prm.br + r) * prm.ld + gj * bc;
            for (int it = tid; it < bc4; it += nthr) cp_async16(d + b * bc + 4 * it, srow + 4 * it);
        }
    };
    // 32-bit word offsets into the planes (the launcher checks that all S planes stay below 2^32 words)
    unsigned int* planes_w = reinterpret_cast<unsigned int*>(prm.planes);
    const unsigned int node_words = (unsigned int)((prm.br * bc) >> 2), plane_words = (unsigned int)P * node_words;
    int64_t r = blockIdx.x;
    if (r < prm.br) fetch(r, 0);
    cp_async_commit();
    for (int buf = 0; r < prm.br; r += gridDim.x, buf ^= 1) {
        if (r + gridDim.x < prm.br) fetch(r + gridDim.x, buf ^ 1);
        cp_async_commit();
        cp_async_wait_all_but_one();                 // this thread's copies of row r have landed ...
        __syncthreads();                             // ... and so have everyone else's
        const float* xb = stage + (size_t)buf * NBLK * bc;
        unsigned int* blk = s_blk + buf * NBLK;
        {
            unsigned int m[NBLK];
#pragma unroll
            for (int b = 0; b < NBLK; ++b) m[b] = 0u;
            for (int it = tid; it < bc4; it += nthr) {
#pragma unroll
                for (int b = 0; b < NBLK; ++b) {
                    const float4 v = *reinterpret_cast<const float4*>(xb + b * bc + 4 * it);
                    m[b] = max(m[b], max(max(__float_as_uint(fabsf(v.x)), __float_as_uint(fabsf(v.y))),
                                         max(__float_as_uint(fabsf(v.z)), __float_as_uint(fabsf(v.w)))));
                }
            }
#pragma unroll
            for (int b = 0; b < NBLK; ++b) {         // every lane is here: the item loop has ended
                const unsigned int w = __reduce_max_sync(0xffffffffu, m[b]);
                if (lane == 0 && w) atomicMax(&blk[b], w);
            }
        }
        __syncthreads();
        for (int p = tid; p < P; p += nthr) {
            double bound = 0.0;
            for (int b = 0; b < NBLK; ++b) bound += fabs(s_cf[p * NBLK + b]) * (double)__uint_as_float(blk[b]);
            const int e = slice_exponent(abs_hi(bound));
            prm.expo[(int64_t)p * prm.br + r] = e;
            s_scale[p] = slice_scale<S>(e);
        }
        __syncthreads();
        if (tid < NBLK) blk[tid] = 0u;               // next read two rows from now, barriers in between
        for (int it = tid; it < bc4; it += nthr) {
            double x[NBLK][4];                       // POLY: indexed by the exponent, else by the block
#pragma unroll
            for (int b = 0; b < NBLK; ++b) {
                const int blk = POLY ? prm.blk_of_exp[b] : b;
                const float4 v = *reinterpret_cast<const float4*>(xb + blk * bc + 4 * it);
                x[b][0] = v.x; x[b][1] = v.y; x[b][2] = v.z; x[b][3] = v.w;
            }
            unsigned int off = (unsigned int)((r * bc) >> 2) + (unsigned int)it;   // word offset inside plane 0, node 0
            if constexpr (POLY) {
                // sum_e x_e b^e = E(b^2) + b O(b^2) with E, O the even and odd halves: nodes p and P-1-p
                // (b and -b) share E and O, which halves the FP64 work of the evaluation
                constexpr int LE = (NBLK - 1) & ~1, LO = ((NBLK - 2) & ~1) + 1;
                const int blk1 = prm.blk_of_exp[1];
                for (int p = 0; 2 * p < P; ++p) {
                    const int p2 = P - 1 - p;
                    const double b1 = s_cf[p * NBLK + blk1], b2 = s_cf[p2 * NBLK + blk1], y = b1 * b1;
                    double E[4], O[4], a[4];
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        E[v] = x[LE][v];
                        O[v] = x[LO][v];
#pragma unroll
                        for (int e = LE - 2; e >= 0; e -= 2) E[v] = fma(E[v], y, x[e][v]);
#pragma unroll
                        for (int e = LO - 2; e >= 1; e -= 2) O[v] = fma(O[v], y, x[e][v]);
                        a[v] = fma(b1, O[v], E[v]);
                    }
                    unsigned int word[S];
                    digits4<S>(a, s_scale[p], word);
                    const unsigned int o1 = off + (unsigned int)p * node_words;
#pragma unroll
                    for (int s = 0; s < S; ++s) __stcs(planes_w + (o1 + (unsigned int)s * plane_words), word[s]);
                    if (p2 != p) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) a[v] = fma(b2, O[v], E[v]);
                        digits4<S>(a, s_scale[p2], word);
                        const unsigned int o2 = off + (unsigned int)p2 * node_words;
#pragma unroll
                        for (int s = 0; s < S; ++s) __stcs(planes_w + (o2 + (unsigned int)s * plane_words), word[s]);
                    }
                }
            } else {
#pragma unroll 2
                for (int p = 0; p < P; ++p, off += node_words) {
                    const double* cf = s_cf + p * NBLK;
                    double a[4] = {0, 0, 0, 0};
#pragma unroll
                    for (int b = 0; b < NBLK; ++b) {
                        const double k = cf[b];
                        a[0] = fma(k, x[b][0], a[0]); a[1] = fma(k, x[b][1], a[1]);
                        a[2] = fma(k, x[b][2], a[2]); a[3] = fma(k, x[b][3], a[3]);
                    }
                    unsigned int word[S];
                    digits4<S>(a, s_scale[p], word);
#pragma unroll
                    for (int s = 0; s < S; ++s) __stcs(planes_w + (off + (unsigned int)s * plane_words), word[s]);
                }
            }
        }
        __syncthreads();                             // row buffer `buf` is refilled by the next trip's copies
    }
}

// ---- X side: operand rows are columns of the share (K = block rows, strided in the source) ----
// A CTA stages the source values of a tile (128 rows kk x 8 columns n of every block) in shared
// memory, transposed, so that a thread owns 4 consecutive kk of one column (warp = column,
// lane = kk / 4): it converts its values once and runs over the nodes.
//   S = 0    : largest |X~_p[kk][n]| over kk, met in amax[p][n] (high words, zeroed before the launch)
//   S = 5, 6 : S digits with the column's exponent, written K-major (128 bytes per warp and plane);
//              the CTAs of the first row slab also publish the exponents.
constexpr int XT_K = 128, XT_N = 8, XT_PITCH = XT_K + 4;

template <int NBLK, int S>
__global__ void __launch_bounds__(256) colpass_kernel(SliceParams prm) {
    extern __shared__ double s_coef[];                             // [P][NBLK], then the tile
    float* xs = reinterpret_cast<float*>(s_coef + prm.P * NBLK);   // [NBLK][XT_N][XT_PITCH]
    for (int i = threadIdx.x; i < prm.P * NBLK; i += 256) s_coef[i] = prm.coef[i];
    const int64_t n0 = (int64_t)blockIdx.x * XT_N, k0 = (int64_t)blockIdx.y * XT_K;
    {   // stage the tile: thread = (column nn, rows kq + 32 j); all loads issued before the stores
        const int nn = threadIdx.x % XT_N, kq = threadIdx.x / XT_N;
        const int64_t gn = n0 + nn;
        float v[NBLK][XT_K / 32];
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const int gi = b / prm.gc, gj = b - gi * prm.gc;
#pragma unroll
            for (int j = 0; j < XT_K / 32; ++j) {
                const int64_t gk = k0 + kq + 32 * j;
                v[b][j] = (gk < prm.br && gn < prm.bc) ? __ldg(prm.src + (gi * prm.br + gk) * prm.ld + gj * prm.bc + gn) : 0.f;
            }
        }
#pragma unroll
        for (int b = 0; b < NBLK; ++b)
#pragma unroll
            for (int j = 0; j < XT_K / 32; ++j) xs[(b * XT_N + nn) * XT_PITCH + kq + 32 * j] = v[b][j];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t gn = n0 + warp, gk = k0 + 4 * lane;
    if (gn >= prm.bc) return;                                      // whole warp
    double x[NBLK][4];
#pragma unroll
    for (int b = 0; b < NBLK; ++b) {
        const float4 v = *reinterpret_cast<const float4*>(xs + (b * XT_N + warp) * XT_PITCH + 4 * lane);
        x[b][0] = v.x; x[b][1] = v.y; x[b][2] = v.z; x[b][3] = v.w;
    }
    const int64_t plane_stride = (int64_t)prm.P * prm.bc * prm.br;
#pragma unroll 2
    for (int p = 0; p < prm.P; ++p) {
        const double* cf = s_coef + p * NBLK;
        double a[4] = {0, 0, 0, 0};
#pragma unroll
        for (int b = 0; b < NBLK; ++b) {
            const double k = cf[b];
            a[0] = fma(k, x[b][0], a[0]); a[1] = fma(k, x[b][1], a[1]);
            a[2] = fma(k, x[b][2], a[2]); a[3] = fma(k, x[b][3], a[3]);
        }
        if (S == 0) {
            const unsigned int mx = __reduce_max_sync(0xffffffffu, abs_hi_max4(a));
            if (lane == 0) atomicMax(prm.amax + (int64_t)p * prm.bc + gn, mx);
        } else {
            const int e = slice_exponent(prm.amax[(int64_t)p * prm.bc + gn]);
            if (blockIdx.y == 0 && lane == 0) prm.expo[(int64_t)p * prm.bc + gn] = e;
            constexpr int SS = S > 0 ? S : 1;
            unsigned int word[SS];
            digits4<SS>(a, slice_scale<SS>(e), word);
            if (gk < prm.br) {                                     // br is a multiple of 16: whole words
                int8_t* dst = prm.planes + ((int64_t)p * prm.bc + gn) * prm.br + gk;
#pragma unroll
                for (int s = 0; s < SS; ++s) *reinterpret_cast<unsigned int*>(dst + s * plane_stride) = word[s];
            }
        }
    }
}

// ---- training mode: the sliced copies of W's shares, cut from the FP64 shares ----------------------
// Rows: one warp per row (node p, share row r) of K doubles: largest magnitude (exact), exponent,
// digits; a lane owns four consecutive values per trip, so a warp reads 1 KB and writes 128 bytes
// per plane at a time.
template <int S>
__global__ void __launch_bounds__(256) reslice_rows_kernel(const double* __restrict__ master, int8_t* planes, int* expo,
                                                          int64_t n_rows, int64_t K, int64_t plane_stride,
                                                          const gpd_locate_result* gate) {
    if (gate && gate->outcome == GPD_DECODE_FAILURE) return;      // the update was skipped: the copies still hold the shares
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= n_rows) return;                                     // whole warp
    const double* src = master + row * K;
    unsigned int mx = 0u;
    for (int64_t k = 4 * lane; k < K; k += 128) {
        const double2 v0 = *reinterpret_cast<const double2*>(src + k), v1 = *reinterpret_cast<const double2*>(src + k + 2);
        mx = max(mx, max(max(abs_hi(v0.x), abs_hi(v0.y)), max(abs_hi(v1.x), abs_hi(v1.y))));
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    const int e = slice_exponent(mx);
    if (lane == 0) expo[row] = e;
    const double scale = slice_scale<S>(e);
    int8_t* dst = planes + row * K;
    for (int64_t k = 4 * lane; k < K; k += 128) {                  // second read of the row: from L1 / L2
        const double2 v0 = *reinterpret_cast<const double2*>(src + k), v1 = *reinterpret_cast<const double2*>(src + k + 2);
        const double a[4] = {v0.x, v0.y, v1.x, v1.y};
        unsigned int word[S];
        digits4<S>(a, scale, word);
#pragma unroll
        for (int t = 0; t < S; ++t) *reinterpret_cast<unsigned int*>(dst + t * plane_stride + k) = word[t];
    }
}

// Columns, pass 1: largest magnitude of every column of every node's share (M x K), met in
// amax[p][c] (high words, zeroed before the launch).  Thread = column, CTA = slab of 64 rows.
__global__ void __launch_bounds__(256) colmax_kernel(const double* __restrict__ master, unsigned int* amax, int64_t M, int64_t K) {
    const int64_t c = (int64_t)blockIdx.x * 256 + threadIdx.x, r0 = (int64_t)blockIdx.y * 64, p = blockIdx.z;
    if (c >= K) return;
    const double* src = master + (p * M + r0) * K + c;
    const int64_t rows = min((int64_t)64, M - r0);
    unsigned int mx = 0u;
    for (int64_t r = 0; r < rows; ++r) mx = max(mx, abs_hi(src[r * K]));
    if (mx) atomicMax(amax + p * K + c, mx);
}

// Columns, pass 2: a CTA stages a tile of 128 rows x 32 columns of one node's share in shared memory
// (read along the rows of the share, 256-byte segments), then every thread takes four consecutive
// rows of one column (warp = column, four columns per warp in turn), cuts them into digits with the
// column's exponent and writes them with the share's row index contiguous: [S][P][K][M].
constexpr int RC_ROWS = 128, RC_COLS = 32, RC_PITCH = RC_ROWS + 1;
template <int S>
__global__ void __launch_bounds__(256) reslice_cols_kernel(const double* __restrict__ master, const unsigned int* amax,
                                                          int8_t* planes, int* expo, int64_t M, int64_t K,
                                                          int64_t plane_stride, const gpd_locate_result* gate) {
    __shared__ double xs[RC_COLS * RC_PITCH];
    if (gate && gate->outcome == GPD_DECODE_FAILURE) return;      // the update was skipped: the copies still hold the shares
    const int64_t c0 = (int64_t)blockIdx.x * RC_COLS, r0 = (int64_t)blockIdx.y * RC_ROWS, p = blockIdx.z;
    const double* src = master + p * M * K;
    for (int idx = threadIdx.x; idx < RC_ROWS * RC_COLS; idx += 256) {
        const int cc = idx % RC_COLS, rr = idx / RC_COLS;
        const int64_t gr = r0 + rr, gc = c0 + cc;
        xs[cc * RC_PITCH + rr] = (gr < M && gc < K) ? src[gr * K + gc] : 0.0;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t gr = r0 + 4 * lane;
    for (int cc = warp; cc < RC_COLS; cc += 8) {
        const int64_t gc = c0 + cc;
        if (gc >= K) break;
        const int e = slice_exponent(amax[p * K + gc]);
        if (blockIdx.y == 0 && lane == 0) expo[p * K + gc] = e;
        const double* col = xs + cc * RC_PITCH + 4 * lane;
        const double a[4] = {col[0], col[1], col[2], col[3]};
        unsigned int word[S];
        digits4<S>(a, slice_scale<S>(e), word);
        if (gr < M) {                                              // M is a multiple of 16: whole words
            int8_t* dst = planes + (p * K + gc) * M + gr;
#pragma unroll
            for (int t = 0; t < S; ++t) *reinterpret_cast<unsigned int*>(dst + t * plane_stride) = word[t];
        }
    }
}

template <int NBLK>
gpd_status launch_rows_fused(const SliceParams& prm, int slices, size_t smem, cudaStream_t st) {
    // CTA size follows the row length (one thread per four columns, at most 512); shorter rows run
    // more CTAs per SM on the same register and shared-memory budget
    const int threads = (int)std::min<int64_t>(kFusedMaxThreads, ((prm.bc >> 2) + 31) / 32 * 32);
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(kFusedMaxThreads / threads, (200 * 1024) / smem));
    const int grid = (int)std::min<int64_t>(prm.br, (int64_t)sm_count() * per_sm);
    auto go = [&](auto kernel) -> gpd_status {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return GPD_ERR_CUDA;
        kernel<<<grid, threads, smem, st>>>(prm);
        return launch_ok();
    };
    if constexpr (NBLK >= 2) {
        if (prm.poly) return slices == 6 ? go(rowslice_fused_kernel<NBLK, 6, true>) : go(rowslice_fused_kernel<NBLK, 5, true>);
    }
    return slices == 6 ? go(rowslice_fused_kernel<NBLK, 6, false>) : go(rowslice_fused_kernel<NBLK, 5, false>);
}

template <int NBLK>
gpd_status launch_rows(const SliceParams& prm, int slices, cudaStream_t st) {
    if constexpr (NBLK <= 8) {       // beyond eight blocks the fused kernel's source values spill
        const size_t fused = fused_smem_bytes(prm.P, NBLK, prm.bc);
        const bool small_offsets = (int64_t)kMaxSlices * prm.P * prm.br * prm.bc < (int64_t)4 << 32;
        if (fused <= 200 * 1024 && small_offsets) return launch_rows_fused<NBLK>(prm, slices, fused, st);
    }
    // many blocks, or rows too long to stage: scale pass, then slice pass from global memory
    rowscale_kernel<NBLK><<<(unsigned)prm.br, 256, 0, st>>>(prm);
    if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
    const int64_t work = prm.br * (prm.bc / 4);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, sm_count() * 16));
    const size_t smem = sizeof(double) * prm.P * NBLK;
    if (slices == 6) rowslice_kernel<NBLK, 6><<<grid, 256, smem, st>>>(prm);
    else rowslice_kernel<NBLK, 5><<<grid, 256, smem, st>>>(prm);
    return launch_ok();
}

template <int NBLK, int S>
gpd_status launch_colpass(const SliceParams& prm, cudaStream_t st) {
    const size_t smem = sizeof(double) * prm.P * NBLK + sizeof(float) * NBLK * XT_N * XT_PITCH;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(colpass_kernel<NBLK, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return GPD_ERR_CUDA;
    dim3 grid((unsigned)((prm.bc + XT_N - 1) / XT_N), (unsigned)((prm.br + XT_K - 1) / XT_K));
    colpass_kernel<NBLK, S><<<grid, 256, smem, st>>>(prm);
    return launch_ok();
}

template <int NBLK>
gpd_status launch_cols(const SliceParams& prm, int slices, cudaStream_t st) {
    if (cudaMemsetAsync(prm.amax, 0, sizeof(unsigned int) * prm.P * prm.bc, st) != cudaSuccess) return GPD_ERR_CUDA;
    gpd_status rc = launch_colpass<NBLK, 0>(prm, st);
    if (rc != GPD_OK) return rc;
    return slices == 6 ? launch_colpass<NBLK, 6>(prm, st) : launch_colpass<NBLK, 5>(prm, st);
}

}  // namespace

bool sliced_supported(const gpd_plan_s* plan) {
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int64_t K = s.N0 / c.n;
    const int64_t M = s.N1 / c.m, N = s.B / c.d1;
    const int nb_w = c.m * c.n, nb_x = c.n * c.d1;
    auto ok_blk = [](int n) {
        return n == 1 || n == 2 || n == 3 || n == 4 || n == 6 || n == 8 || n == 9 || n == 12 || n == 16;
    };
    auto ok_k = [](int64_t k) { return k % 16 == 0 && k <= 16384; };   // TMA rows of whole 16 bytes; int32 accumulation of
                                                                        // up to 6 plane pairs of |digit| <= 128 over K terms
    if (!ok_k(K) || !ok_blk(nb_w) || !ok_blk(nb_x)) return false;
    // scales are tracked through FP32 magnitudes of the inputs times the coefficients
    for (double c : plan->coefW) if (!(std::fabs(c) < 1e30)) return false;
    for (double c : plan->coefX) if (!(std::fabs(c) < 1e30)) return false;
    // the sliced operands live in buffers sized for the FP64 shares they replace
    auto fits = [&](int64_t rows, int64_t k) {
        return sliced_layout(plan->slices, plan->P, rows, k).total_bytes <= 8 * (int64_t)plan->P * rows * k;
    };
    if (!fits(M, K) || !fits(N, K)) return false;
    if (plan->train) {
        // backward product: contraction over N1/m, Delta~^T_p rows of B/d2; update: contraction over B
        if (plan->prod[GPD_BWD].Q == 0 || plan->prod[GPD_AUDIT].Q == 0) return false;
        if (!ok_k(M) || !ok_k(s.B) || !ok_k(s.B / c.d2) || !ok_k(N) || !ok_blk(c.d2 * c.m) || !ok_blk(c.m) || !ok_blk(c.n))
            return false;
        for (double c : plan->coefDT) if (!(std::fabs(c) < 1e30)) return false;
        if (!fits(s.B / c.d2, M) || !fits(M, s.B) || !fits(K, s.B) || !fits(K, M)) return false;
    }
    return true;
}

TrainLayout train_layout(const gpd_plan_s* plan) {
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int64_t M = s.N1 / c.m, K = s.N0 / c.n, P = plan->P;
    TrainLayout t;
    t.rows = sliced_layout(plan->slices, P, M, K);
    t.cols = sliced_layout(plan->slices, P, K, M);
    t.rows_offset = (8 * P * M * K + 255) / 256 * 256;
    t.cols_offset = (t.rows_offset + t.rows.total_bytes + 255) / 256 * 256;
    t.total_bytes = t.cols_offset + t.cols.total_bytes;
    return t;
}

SlicedLayout sliced_layout(int slices, int64_t P, int64_t rows, int64_t K) {
    SlicedLayout l;
    l.plane_bytes = P * rows * K;
    l.expo_offset = (slices * l.plane_bytes + 255) / 256 * 256;
    l.amax_offset = (l.expo_offset + P * rows * 4 + 255) / 256 * 256;
    l.total_bytes = l.amax_offset + P * rows * 4;
    return l;
}

gpd_status reslice_launch(gpd_plan_s* plan, void* W_shares, cudaStream_t st, const gpd_locate_result* gate,
                          bool cols_amax_ready) {
    if (!plan->train) return GPD_ERR_UNSUPPORTED;
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int64_t M = s.N1 / c.m, K = s.N0 / c.n, P = plan->P;
    const TrainLayout tl = train_layout(plan);
    char* base = reinterpret_cast<char*>(W_shares);
    const double* master = reinterpret_cast<const double*>(base);
    {   // rows of the shares
        int8_t* planes = reinterpret_cast<int8_t*>(base + tl.rows_offset);
        int* expo = reinterpret_cast<int*>(base + tl.rows_offset + tl.rows.expo_offset);
        const int64_t n_rows = P * M;
        reslice_rows_kernel<6><<<(unsigned)((n_rows + 7) / 8), 256, 0, st>>>(master, planes, expo, n_rows, K, P * M * K, gate);
        if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
    }
    {   // columns of the shares
        int8_t* planes = reinterpret_cast<int8_t*>(base + tl.cols_offset);
        int* expo = reinterpret_cast<int*>(base + tl.cols_offset + tl.cols.expo_offset);
        unsigned int* amax = reinterpret_cast<unsigned int*>(base + tl.cols_offset + tl.cols.amax_offset);
        if (!cols_amax_ready) {
            if (cudaMemsetAsync(amax, 0, sizeof(unsigned int) * P * K, st) != cudaSuccess) return GPD_ERR_CUDA;
            colmax_kernel<<<dim3((unsigned)((K + 255) / 256), (unsigned)((M + 63) / 64), (unsigned)P), 256, 0, st>>>(master, amax, M, K);
            if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
        }
        reslice_cols_kernel<6><<<dim3((unsigned)((K + RC_COLS - 1) / RC_COLS), (unsigned)((M + RC_ROWS - 1) / RC_ROWS), (unsigned)P),
                                 256, 0, st>>>(master, amax, planes, expo, M, K, P * M * K, gate);
    }
    return launch_ok();
}

gpd_status encode_sliced_launch(gpd_plan_s* plan, int operand, const float* src, void* dst, cudaStream_t st) {
    // 16-byte loads of the source rows, word stores into the planes, aligned exponent tables
    if (reinterpret_cast<uintptr_t>(src) % 16 != 0 || reinterpret_cast<uintptr_t>(dst) % 16 != 0) return GPD_ERR_ARG;
    gpd_status rc = ensure_device(plan);
    if (rc != GPD_OK) return rc;
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    SliceParams prm{};
    prm.src = src;
    prm.P = plan->P;
    int gr;
    bool by_rows = true;          // operand rows = rows of the share (else: its columns, written transposed)
    switch (operand) {
        case -1:                  // W: m x n blocks of (N1/m) x (N0/n); operand rows = share rows, K = N0/n
            gr = c.m; prm.gc = c.n; prm.ld = s.N0; prm.br = s.N1 / c.m; prm.bc = s.N0 / c.n;
            prm.coef = plan->dev.base + plan->dev.off_coefW;
            prm.poly = c.m * c.n <= 16 && plan->points_symmetric;
            for (int i = 0; i < c.m; ++i)
                for (int j = 0; j < c.n; ++j)
                    if (prm.poly) prm.blk_of_exp[plan->alt_subst ? i + c.m * j : c.n * i + j] = i * c.n + j;
            break;
        case GPD_OPERAND_X_FWD:   // X: n x d1 blocks of (N0/n) x (B/d1); operand rows = share columns, K = N0/n
            gr = c.n; prm.gc = c.d1; prm.ld = s.B; prm.br = s.N0 / c.n; prm.bc = s.B / c.d1;
            prm.coef = plan->dev.base + plan->dev.off_coefX; by_rows = false; break;
        case GPD_OPERAND_DELTAT_BWD:   // Delta^T: d2 x m blocks of (B/d2) x (N1/m); operand rows = share rows, K = N1/m
            gr = c.d2; prm.gc = c.m; prm.ld = s.N1; prm.br = s.B / c.d2; prm.bc = s.N1 / c.m;
            prm.coef = plan->dev.base + plan->dev.off_coefDT; break;
        case GPD_OPERAND_DELTA_UPD:    // Delta: m x 1 blocks of (N1/m) x B; operand rows = share rows, K = B
            gr = c.m; prm.gc = 1; prm.ld = s.B; prm.br = s.N1 / c.m; prm.bc = s.B;
            prm.coef = plan->dev.base + plan->dev.off_coefDup; break;
        case GPD_OPERAND_X_UPD:        // X: n x 1 blocks of (N0/n) x B; operand rows = share rows, K = B
            gr = c.n; prm.gc = 1; prm.ld = s.B; prm.br = s.N0 / c.n; prm.bc = s.B;
            prm.coef = plan->dev.base + plan->dev.off_coefXup; break;
        default: return GPD_ERR_ARG;
    }
    if (operand != -1 && operand != GPD_OPERAND_X_FWD && !plan->train) return GPD_ERR_UNSUPPORTED;
    prm.nblk = gr * prm.gc;
    const SlicedLayout lay = by_rows ? sliced_layout(plan->slices, plan->P, prm.br, prm.bc)
                                     : sliced_layout(plan->slices, plan->P, prm.bc, prm.br);
    prm.planes = reinterpret_cast<int8_t*>(dst);
    prm.expo = reinterpret_cast<int*>(reinterpret_cast<char*>(dst) + lay.expo_offset);
    prm.amax = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(dst) + lay.amax_offset);
#define GPD_SLICE_CASE(NB) \
    case NB: return by_rows ? launch_rows<NB>(prm, plan->slices, st) : launch_cols<NB>(prm, plan->slices, st)
    switch (prm.nblk) {
        GPD_SLICE_CASE(1); GPD_SLICE_CASE(2); GPD_SLICE_CASE(3); GPD_SLICE_CASE(4); GPD_SLICE_CASE(6);
        GPD_SLICE_CASE(8); GPD_SLICE_CASE(9); GPD_SLICE_CASE(12); GPD_SLICE_CASE(16);
        default: return GPD_ERR_UNSUPPORTED;
    }
#undef GPD_SLICE_CASE
}

}  // namespace gpd
