// FP64-class worker products (steps O1, O2) and the coded update (O3, Eq. 10) on the integer tensor
// cores.  The kernel multiplies two sliced operands, C[p] = A[p] B[p]^T; the forward product takes
// A = W~_p (rows), B = X~_p^T, the backward product A = Delta~^T_p, B = W~_p^T (the column-sliced
// copy of the shares), the update A = Delta^_p, B = X^_p and adds into the FP64 shares.
//
// Both operands arrive cut into S = 6 (or 5) signed 8-bit digit planes (slice.cu):
//     W~_p[i][k] = 2^ea[i] * sum_s A_s[i][k] 256^-(s+1),   X~_p[k][j] = 2^eb[j] * sum_t B_t[j][k] 256^-(t+1).
// A digit-plane product A_s B_t^T is an int8 x int8 -> int32 contraction, exact on the tensor
// cores (|digit| <= 128, so six summed pairs cannot overflow for K <= 21845).  Pairs with
// s + t <= S - 1 (weight >= 256^-(S+1)) are kept: 21 of 36 (15 of 25), the rest lie below
// 2^-(8 S + 2) of the row/column scales.  Pairs of equal weight share one accumulator, so a 128 x 64
// output tile owns S 128 x 64 int32 accumulators in tensor memory, group g = s + t at columns
// 64 g.  For a fixed s the planes t = 0 .. S-1-s are adjacent in shared memory and their
// accumulators are adjacent in tensor memory, so one tcgen05.mma of N = 64 (S - s) columns
// (two when that exceeds 256) covers all pairs of plane s: 8 (6) instructions per 32 elements of K.
//
// One CTA per SM walks the output tiles.  Warp roles: warp 0 one lane issues the TMA copies (two per
// 64-element k-block: the planes are a 4-d tensor [S][P][rows][K] and one box holds all S planes of an
// operand; 3-stage ring that runs on across tiles), warp 1 allocates tensor memory and
// one lane issues the MMAs, warps 2..9 read the accumulators back and combine them in FP64
// (sum_g acc_g 2^-8g), release tensor memory to the next tile's MMAs, then apply the row and column
// powers of two and store while that tile's main loop is already running.
// Every mbarrier wait is bounded; on expiry the CTA raises a status word, drains its copies,
// frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>

#include "slice_common.h"
#include "tc_common.h"

namespace gpd {

namespace {

// Output tiles are 128 x 64: S accumulator groups of 64 columns fill 384 of the 512 tensor-memory columns.
// (Tiles of 128 x 32 with two alternating accumulator sets, which hide the epilogue's read of tensor
// memory, were measured and are slower at every contraction length: the A planes are then fetched per
// 32 instead of per 64 output columns.)
constexpr int BM = 128, BN = 64, BK = 64, STAGES = 3;
constexpr int UMMA_K = 32;                            // int8 elements per MMA along K
constexpr int A_PLANE_BYTES = BM * BK;                // 8 KB, rows of 64 B
constexpr int B_PLANE_BYTES = BN * BK;                // 4 KB
__host__ __device__ constexpr int stage_bytes(int S) { return S * (A_PLANE_BYTES + B_PLANE_BYTES); }   // 72 KB (60 KB)
__host__ __device__ constexpr int smem_bytes(int S) { return STAGES * stage_bytes(S) + 1024; }
constexpr int TMEM_COLS = 512;                        // allocations are powers of two
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + kEpiWarps * 32;

__device__ int g_i8_status = 0;                       // GPD_ERR_TIMEOUT if a bounded wait expired

using tc::kWaitCycles;
using tc::mbar_arrive;
using tc::mbar_expect_tx;
using tc::mbar_init;
using tc::mbar_try_wait;
using tc::smem_u32;
using tc::tma_load_4d;
using tc::umma_commit;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    return tc::mbar_wait(bar, parity, abort_flag, &g_i8_status);
}
// K-major tile with rows of 64 bytes under the 64-byte swizzle: 8-row groups 512 bytes apart
// (descriptor version 1, layout type 4).
__device__ __forceinline__ uint64_t desc_sw64(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(16 >> 4) << 16;
    d |= (uint64_t)(512 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)4 << 61;
    return d;
}
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor: int32 accumulator, signed 8-bit A and B, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t idesc_i8(int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
// 2^e as a double (0 below the normal range: only the all-zero marker gets there)
__device__ __forceinline__ double exp2i(int e) {
    if (e < -1022) return 0.0;
    if (e > 1023) e = 1023;
    return __longlong_as_double((long long)(e + 1023) << 52);
}
// int32 -> double without the conversion unit: 2^52 + 2^31 + x has x ^ 0x80000000 as its low word
__device__ __forceinline__ double i2d(uint32_t x) {
    return __hiloint2double(0x43300000, (int)(x ^ 0x80000000u)) - 4503601774854144.0;
}

struct I8Params {
    const int* ea;     // [P][M]
    const int* eb;     // [P][N]
    double* C;         // [P][M][N]
    int64_t M, N, K;
    int P;
    double shrink, eta;                  // update: C <- shrink * C + eta * A B^T
    const gpd_locate_result* gate;       // update: skipped when this reports a decoding failure
    unsigned int* colmax;                // update, optional: [P][N] largest |new C| per column (high words)
};

// One warp reads 16 lanes x 32 consecutive 32-bit columns of tensor memory in the 16 x 256-bit shape:
// thread t gets, for each block k of 8 columns, registers 4k + 2i + e = (lane 8i + t / 4, column 8k + 2 (t % 4) + e),
// lanes counted from the lane base of taddr.
__device__ __forceinline__ void tmem_ld_16x256(uint32_t (&r)[16], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
template <int S, bool UPDATE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_i8_sliced_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, I8Params prm,
                      int tiles_m, int tiles_n, int tiles) {
    if (UPDATE && prm.gate && prm.gate->outcome == GPD_DECODE_FAILURE) return;
    constexpr int STAGE_BYTES = stage_bytes(S);
    constexpr int CW = BN / 2;                        // columns an epilogue warp reads (two warps per lane quarter)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // full/empty: operand ring (runs on across the tiles of this CTA); acc_full: a tile's accumulators
    // are complete; acc_empty: the epilogue warps have read them, the next tile may overwrite them
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full, acc_empty;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (int)((prm.K + BK - 1) / BK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&acc_full, 1);
        mbar_init(&acc_empty, kEpiWarps);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    volatile int* abort_p = &abort_flag;

    auto A_plane = [&](int s, int t) { return smem + s * STAGE_BYTES + t * A_PLANE_BYTES; };
    auto B_plane = [&](int s, int t) { return smem + s * STAGE_BYTES + S * A_PLANE_BYTES + t * B_PLANE_BYTES; };
    // tile -> (node p, row tile, column tile); consecutive CTAs take consecutive tiles of one round
    auto tile_origin = [&](int tile, int& p, int& m0, int& n0) {
        const int tn = tile % tiles_n, tm = (tile / tiles_n) % tiles_m;
        p = tile / (tiles_n * tiles_m);
        m0 = tm * BM;
        n0 = tn * BN;
    };

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int it = 0;                          // k-blocks issued so far, over all tiles
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                int p, m0, n0;
                tile_origin(tile, p, m0, n0);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_p)) { ok = false; break; }
                    mbar_expect_tx(&full_bar[s], STAGE_BYTES);
                    // one copy per operand brings all S digit planes of the block (box K x rows x 1 node x S)
                    tma_load_4d(A_plane(s, 0), &tmA, kb * BK, m0, p, 0, &full_bar[s]);
                    tma_load_4d(B_plane(s, 0), &tmB, kb * BK, n0, p, 0, &full_bar[s]);
                }
            }
            if (*abort_p) {                      // let copies still in flight land before the CTA exits
                for (int j = it > STAGES ? it - STAGES : 0; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full_bar[j % STAGES], (j / STAGES) & 1) && clock64() - t0 < kWaitCycles) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            int it = 0, ti = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++ti) {
                // the previous tile's accumulators must have been read
                if (!mbar_wait(&acc_empty, (ti & 1) ^ 1, abort_p)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(&full_bar[s], ph, abort_p)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a0 = smem_u32(A_plane(s, 0)), b0 = smem_u32(B_plane(s, 0));
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
#pragma unroll
                        for (int ta = 0; ta < S; ++ta) {
                            // planes tb = 0 .. S-1-ta of B in one operand of 64 (S - ta) rows, at most 256 per MMA;
                            // the pair (ta, tb) lands in accumulator group ta + tb = columns 64 (ta + tb)
                            const uint64_t da = desc_sw64(a0 + ta * A_PLANE_BYTES + k * UMMA_K);
                            const int n_total = BN * (S - ta);
                            const int n_first = n_total > 256 ? 256 : n_total;
                            // the plane-0 instruction of a tile's first k-step overwrites every group
                            const uint32_t acc = (kb > 0 || k > 0 || ta > 0) ? 1u : 0u;
                            umma_i8(tmem_base + BN * ta, da, desc_sw64(b0 + k * UMMA_K), idesc_i8(n_first), acc);
                            if (n_total > 256)
                                umma_i8(tmem_base + BN * ta + 256, da, desc_sw64(b0 + (256 / BN) * B_PLANE_BYTES + k * UMMA_K),
                                        idesc_i8(n_total - 256), acc);
                        }
                    }
                    umma_commit(&empty_bar[s]);      // stage reusable once these MMAs have read it
                }
                if (ok) umma_commit(&acc_full);      // this tile's accumulators complete
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        // Tensor memory is read in the 16 x 256-bit shape: a row of 8 columns is spread over 4 adjacent
        // lanes, 2 columns each, so that a 16-byte store per lane writes 64 contiguous bytes of each of
        // 8 rows (whole 32-byte sectors) instead of 16 bytes of each of 32 rows.
        constexpr int NK = CW / 8;                   // 8-column blocks per warp
        const int q = warp & 3;                      // this warp may touch TMEM lanes 32q .. 32q+31
        const int c0 = ((warp - 2) >> 2) * CW;       // two warps per lane quarter: CW columns each
        const int rq = lane >> 2, cq = lane & 3;     // row within a block of 8 rows, column pair within 8 columns
        int ti = 0;
        for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++ti) {
            int p, m0, n0;
            tile_origin(tile, p, m0, n0);
            // this thread's outputs: rows r_base + 8 ri (ri = 0..3), columns c_base + 8 k + {0, 1} (k = 0..NK-1)
            const int64_t r_base = (int64_t)m0 + q * 32 + rq;
            const int64_t c_base = (int64_t)n0 + c0 + 2 * cq;
            int era[4], ecb[NK][2];                  // exponents of the rows' and the columns' scales
#pragma unroll
            for (int ri = 0; ri < 4; ++ri)
                era[ri] = r_base + 8 * ri < prm.M ? prm.ea[(int64_t)p * prm.M + r_base + 8 * ri] - 2 * kDigitBits : 0;
#pragma unroll
            for (int k = 0; k < NK; ++k)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    ecb[k][e] = c_base + 8 * k + e < prm.N ? prm.eb[(int64_t)p * prm.N + c_base + 8 * k + e] : 0;
            const bool acc_ready = mbar_wait(&acc_full, ti & 1, abort_p);
            __syncwarp();
            if (!__all_sync(0xffffffffu, acc_ready)) break;   // tcgen05.ld is warp-collective: all lanes or none
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            double v[4][NK][2];
#pragma unroll
            for (int ri = 0; ri < 4; ++ri)
#pragma unroll
                for (int k = 0; k < NK; ++k) v[ri][k][0] = v[ri][k][1] = 0.0;
            // lanes 32q + 16h .. + 15 of group g; register 4k + 2i + e = (row 8i + rq, column 8k + 2cq + e)
            auto group_addr = [&](int g, int h) {
                return tmem_base + ((uint32_t)(q * 32 + 16 * h) << 16) + (uint32_t)(BN * g + c0);
            };
            // smallest weight first; two groups are in flight per wait (one for the odd one out).
            // (Summing the groups as 64-bit integers first, to spare the FP64 pipe, was measured: slower.)
#pragma unroll
            for (int g = S - 1; g >= 0; g -= 2) {
                uint32_t r[2][2][4 * NK];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    tmem_ld_16x256(r[0][h], group_addr(g, h));
                    if (g >= 1) tmem_ld_16x256(r[1][h], group_addr(g - 1, h));
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if (u == 1 && g < 1) break;
                    const double w = exp2i(-kDigitBits * (g - u));
#pragma unroll
                    for (int ri = 0; ri < 4; ++ri)
#pragma unroll
                        for (int k = 0; k < NK; ++k)
#pragma unroll
                            for (int e = 0; e < 2; ++e)
                                v[ri][k][e] = fma(i2d(r[u][ri >> 1][4 * k + 2 * (ri & 1) + e]), w, v[ri][k][e]);
                }
            }
            // the accumulators are in registers: hand tensor memory back to the MMA warp, then scale
            // and store while the next tile's main loop runs
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty);
            double* cbase = prm.C + (int64_t)p * prm.M * prm.N + r_base * prm.N + c_base;
            const bool vec = (prm.N & 1) == 0;       // 16-byte stores: pairs start at even columns
            unsigned int cmax[NK][2];                // update: largest |new value| of this thread's rows, per column
#pragma unroll
            for (int k = 0; k < NK; ++k) cmax[k][0] = cmax[k][1] = 0u;
#pragma unroll
            for (int ri = 0; ri < 4; ++ri) {
                if (r_base + 8 * ri >= prm.M) continue;
                double* crow = cbase + (int64_t)(8 * ri) * prm.N;
                double2 old[NK];                     // update: the stored shares this thread adds into
                if (UPDATE && vec) {
#pragma unroll
                    for (int k = 0; k < NK; ++k)
                        if (c_base + 8 * k + 1 < prm.N) old[k] = *reinterpret_cast<const double2*>(crow + 8 * k);
                }
#pragma unroll
                for (int k = 0; k < NK; ++k) {
                    double2 o;
                    o.x = v[ri][k][0] * exp2i(era[ri] + ecb[k][0]);
                    o.y = v[ri][k][1] * exp2i(era[ri] + ecb[k][1]);
                    if (vec && c_base + 8 * k + 1 < prm.N) {
                        if (UPDATE) {
                            o.x = fma(prm.eta, o.x, prm.shrink * old[k].x);
                            o.y = fma(prm.eta, o.y, prm.shrink * old[k].y);
                            cmax[k][0] = max(cmax[k][0], (unsigned int)__double2hiint(o.x) & 0x7FFFFFFFu);
                            cmax[k][1] = max(cmax[k][1], (unsigned int)__double2hiint(o.y) & 0x7FFFFFFFu);
                            *reinterpret_cast<double2*>(crow + 8 * k) = o;      // read again soon: no streaming hint
                        } else {
                            __stcs(reinterpret_cast<double2*>(crow + 8 * k), o);
                        }
                    } else {
                        if (c_base + 8 * k < prm.N) {
                            const double nx = UPDATE ? fma(prm.eta, o.x, prm.shrink * crow[8 * k]) : o.x;
                            if (UPDATE) cmax[k][0] = max(cmax[k][0], (unsigned int)__double2hiint(nx) & 0x7FFFFFFFu);
                            crow[8 * k] = nx;
                        }
                        if (c_base + 8 * k + 1 < prm.N) {
                            const double ny = UPDATE ? fma(prm.eta, o.y, prm.shrink * crow[8 * k + 1]) : o.y;
                            if (UPDATE) cmax[k][1] = max(cmax[k][1], (unsigned int)__double2hiint(ny) & 0x7FFFFFFFu);
                            crow[8 * k + 1] = ny;
                        }
                    }
                }
            }
            if (UPDATE && prm.colmax) {
                // column maxima of the new shares for the column-sliced copy: over this thread's four rows
                // (above), then over the eight lanes that hold the same columns, one atomic per column
#pragma unroll
                for (int k = 0; k < NK; ++k)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        unsigned int v = cmax[k][e];
                        v = max(v, __shfl_xor_sync(0xffffffffu, v, 4));
                        v = max(v, __shfl_xor_sync(0xffffffffu, v, 8));
                        v = max(v, __shfl_xor_sync(0xffffffffu, v, 16));
                        if (rq == 0 && v && c_base + 8 * k + e < prm.N)
                            atomicMax(prm.colmax + (int64_t)p * prm.N + c_base + 8 * k + e, v);
                    }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side -------------------------------------------------------------------------------------
// 3-D byte tensor [batch][rows][K] (K contiguous), box {BK, box_rows, 1}, 64-byte swizzle,
// out-of-range elements read as zero.
// planes [S][P][rows][K] as a 4-d tensor; one box = a K-block of box_rows rows of one node in all S planes
bool make_map(CUtensorMap* map, const void* base, int S, int64_t P, int64_t rows, int64_t K, int box_rows) {
    return tc::make_map_4d(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base, S, P, rows, K, BK, box_rows, 1, S,
                           CU_TENSOR_MAP_SWIZZLE_64B);
}

template <int S, bool UPDATE>
gpd_status launch_i8(const I8Gemm& g, const I8Params& prm, cudaStream_t st) {
    CUtensorMap tmA, tmB;
    if (!make_map(&tmA, g.A, S, g.P, g.M, g.K, BM)) return GPD_ERR_CUDA;
    if (!make_map(&tmB, g.B, S, g.P, g.N, g.K, BN)) return GPD_ERR_CUDA;
    auto kernel = gemm_i8_sliced_kernel<S, UPDATE>;
    constexpr int smem = smem_bytes(S);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GPD_ERR_CUDA;
    const int tiles_n = (int)((g.N + BN - 1) / BN), tiles_m = (int)((g.M + BM - 1) / BM);
    const int64_t tiles = (int64_t)tiles_n * tiles_m * g.P;
    const unsigned grid = (unsigned)std::min<int64_t>(tiles, sm_count());     // persistent: one CTA per SM walks the tiles
    kernel<<<grid, kThreads, smem, st>>>(tmA, tmB, prm, tiles_m, tiles_n, (int)tiles);
    return launch_ok();
}

}  // namespace

gpd_status gemm_i8_launch(const I8Gemm& g, cudaStream_t st) {
    if (g.K % 16 != 0 || g.K > 16384 || (g.slices != 5 && g.slices != 6)) return GPD_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(g.A) % 16 || reinterpret_cast<uintptr_t>(g.B) % 16 ||
        reinterpret_cast<uintptr_t>(g.C) % 16)
        return GPD_ERR_ARG;
    I8Params prm{};
    prm.P = g.P; prm.M = g.M; prm.N = g.N; prm.K = g.K;
    prm.ea = g.ea; prm.eb = g.eb; prm.C = g.C;
    prm.shrink = g.shrink; prm.eta = g.eta; prm.gate = g.gate; prm.colmax = g.colmax;
    if (g.update) return g.slices == 6 ? launch_i8<6, true>(g, prm, st) : GPD_ERR_UNSUPPORTED;
    return g.slices == 6 ? launch_i8<6, false>(g, prm, st) : launch_i8<5, false>(g, prm, st);
}

gpd_status gemm_sliced_launch(gpd_plan_s* plan, gpd_product which, const void* W_shares, const void* other_sliced,
                              void* out, cudaStream_t st) {
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int S = plan->slices;
    const char* wbase = reinterpret_cast<const char*>(W_shares);
    const char* obase = reinterpret_cast<const char*>(other_sliced);
    I8Gemm g{};
    g.slices = S; g.P = plan->P; g.C = reinterpret_cast<double*>(out);
    g.update = false; g.shrink = 0.0; g.eta = 1.0; g.gate = nullptr;
    if (which == GPD_FWD) {                       // S~_p = W~_p X~_p: A = rows of W~_p, B = columns of X~_p
        g.M = s.N1 / c.m; g.K = s.N0 / c.n; g.N = s.B / c.d1;
        const SlicedLayout lb = sliced_layout(S, g.P, g.N, g.K);
        if (plan->train) {
            const TrainLayout tl = train_layout(plan);
            g.A = wbase + tl.rows_offset;
            g.ea = reinterpret_cast<const int*>(wbase + tl.rows_offset + tl.rows.expo_offset);
        } else {
            const SlicedLayout la = sliced_layout(S, g.P, g.M, g.K);
            g.A = wbase;
            g.ea = reinterpret_cast<const int*>(wbase + la.expo_offset);
        }
        g.B = obase;
        g.eb = reinterpret_cast<const int*>(obase + lb.expo_offset);
    } else if (which == GPD_BWD) {                // C~^T_p = Delta~^T_p W~_p: A = rows of Delta~^T_p, B = columns of W~_p
        if (!plan->train) return GPD_ERR_UNSUPPORTED;
        if (plan->prod[GPD_BWD].Q == 0) return GPD_ERR_P_TOO_SMALL;
        g.M = s.B / c.d2; g.K = s.N1 / c.m; g.N = s.N0 / c.n;
        const TrainLayout tl = train_layout(plan);
        const SlicedLayout la = sliced_layout(S, g.P, g.M, g.K);
        g.A = obase;
        g.ea = reinterpret_cast<const int*>(obase + la.expo_offset);
        g.B = wbase + tl.cols_offset;
        g.eb = reinterpret_cast<const int*>(wbase + tl.cols_offset + tl.cols.expo_offset);
    } else {
        return GPD_ERR_ARG;
    }
    return gemm_i8_launch(g, st);
}

gpd_status update_sliced_launch(gpd_plan_s* plan, void* W_shares, const void* Dhat_sliced, const void* Xhat_sliced,
                                double shrink, double eta, const gpd_locate_result* gate, cudaStream_t st) {
    if (!plan->train) return GPD_ERR_UNSUPPORTED;
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int S = plan->slices;
    I8Gemm g{};
    g.slices = S; g.P = plan->P;
    g.M = s.N1 / c.m; g.N = s.N0 / c.n; g.K = s.B;                 // Delta^_p (M x B) X^_p^T (B x N)
    const SlicedLayout la = sliced_layout(S, g.P, g.M, g.K), lb = sliced_layout(S, g.P, g.N, g.K);
    g.A = Dhat_sliced;
    g.ea = reinterpret_cast<const int*>(reinterpret_cast<const char*>(Dhat_sliced) + la.expo_offset);
    g.B = Xhat_sliced;
    g.eb = reinterpret_cast<const int*>(reinterpret_cast<const char*>(Xhat_sliced) + lb.expo_offset);
    g.C = reinterpret_cast<double*>(W_shares);                     // the FP64 shares lead the buffer
    g.update = true; g.shrink = shrink; g.eta = eta; g.gate = gate;
    // the epilogue meets the column maxima of the new shares, which the re-cut of the column copy needs
    const TrainLayout tl = train_layout(plan);
    g.colmax = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(W_shares) + tl.cols_offset + tl.cols.amax_offset);
    if (cudaMemsetAsync(g.colmax, 0, sizeof(unsigned int) * g.P * g.N, st) != cudaSuccess) return GPD_ERR_CUDA;
    gpd_status rc = gemm_i8_launch(g, st);
    if (rc != GPD_OK) return rc;
    return reslice_launch(plan, W_shares, st, gate, true);
}

int i8_device_status_fetch_and_clear() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_i8_status, sizeof(int)) != cudaSuccess) return (int)GPD_ERR_CUDA;
    if (v != 0) cudaMemcpyToSymbol(g_i8_status, &zero, sizeof(int));
    return v;
}

}  // namespace gpd
