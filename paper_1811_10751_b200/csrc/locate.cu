// Error detection and location over the P worker outputs: Algorithm 1 (Section V-A) taken at
// node level, in the polynomial-time form the decoding appendix allows.
//
// Pass 1 (streaming, bandwidth-bound): every output position l holds one codeword z_l (the P
// values the nodes produced there).  Its syndrome s_l = H z_l is formed in FP64 from H held in
// shared memory; the codeword passes Algorithm 1's zero test when ||s_l||^2 <= tau^2 ||z_l||^2.
// Failing ("active") codewords contribute s_l s_l^T / ||z_l||^2 to a Gram matrix G, reduced per
// CTA through a shared-memory SYRK and added to global memory with one atomic per entry.
// Non-finite values and erased nodes count as zero and their node is flagged up front.
//
// Pass 2 (one warp): pivoted Cholesky factorisation of G: numerical rank rho (pivots above the
// eigenvalue threshold) and range (its leading rho columns); the error
// support is the set of nodes whose parity-check column H_p lies in that range (any P-Q columns of H are independent, so for at most P-Q-1 erroneous nodes no
// other column does); the support is verified by the syndrome energy left outside span(H_A).
// A rank-deficient error matrix (fewer columns of H in that span than its rank) is handled by
// Algorithm 1's search over the supersets of the columns found, bounded in the number of supports.
// More than P-Q-1 nodes or an ambiguous geometry end in a declared decoding failure (Theorem 3,
// third claim).
#include "gpd_internal.h"

namespace gpd {

namespace {

constexpr int kThreads = 256;
constexpr long long kMaxFallbackSupports = 4096;   // supports the superset search of the finish kernel may try

struct SyndromeParams {
    const void* Z;              // [P][L]
    const double* H;            // [R][P]
    int64_t L;
    int P, R;
    double tau2;                // tau_col^2
    unsigned long long erased;  // bit p set: node p is ignored (treated as zero)
    double* gram;               // [R][R], zero on entry
    unsigned long long* counts; // [0] n_active, [1] mask of nodes holding a non-finite value
};

__device__ __forceinline__ void dmma_m8n8k4(double& d0, double& d1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
                 : "+d"(d0), "+d"(d1)
                 : "d"(a), "d"(b));
}

// Syndrome s = H z and squared norm of one codeword: P loads at stride L, issued in equal groups of up to ten
// (ten nodes, the MLP layers' code, then cost one trip to memory instead of two).
// CHECKED = false is the plain form: no per-value tests; a non-finite value, or one of magnitude
// >= kHuge (its square would leave the FP64 range and turn the zero test into inf > inf), shows up
// as a norm >= kHugeSquared and the caller repeats the codeword with CHECKED = true, which zeroes
// such values and erased nodes and records the nodes that held one.
template <typename T, int RT, bool CHECKED>
__device__ __forceinline__ void codeword_syndrome(const T* zp, int64_t L, int P, const double* sH,
                                                  unsigned long long erased, double (&s)[RT], double& nz,
                                                  unsigned long long& bad) {
    constexpr int U = RT <= 8 ? 10 : 4;                  // most loads issued together (fewer where the syndrome fills the registers)
#pragma unroll
    for (int r = 0; r < RT; ++r) s[r] = 0.0;
    nz = 0.0;
    auto absorb = [&](double zz, int pnode, const double* hcol) {
        if (CHECKED) {
            if (!(fabs(zz) < kHuge)) { bad |= 1ULL << pnode; zz = 0.0; }   // NaN, Inf, or a square outside the FP64 range
            if ((erased >> pnode) & 1ULL) zz = 0.0;
        }
        nz = fma(zz, zz, nz);
        const double2* h = reinterpret_cast<const double2*>(hcol);
#pragma unroll
        for (int r = 0; r < RT / 2; ++r) {
            const double2 hv = h[r];
            s[2 * r] = fma(hv.x, zz, s[2 * r]);
            s[2 * r + 1] = fma(hv.y, zz, s[2 * r + 1]);
        }
    };
    // groups of equal size (no short last group: every group costs one trip to memory)
    const int n_groups = (P + U - 1) / U, gs = (P + n_groups - 1) / n_groups;
    for (int p0 = 0; p0 < P; p0 += gs, zp += gs * L, sH += gs * RT) {
        double z[U];
#pragma unroll
        for (int u = 0; u < U; ++u) z[u] = (u < gs && p0 + u < P) ? (double)__ldcs(zp + u * L) : 0.0;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (u < gs && p0 + u < P) absorb(z[u], p0 + u, sH + u * RT);
    }
}

// Streaming pass for up to eight parity checks.  One thread per output position (codeword): the
// syndrome in RT registers, the zero test.  The
// Gram matrix of the failing codewords is formed warp by warp on the FP64 tensor cores: the 32 scaled syndromes of a warp are staged in shared
// memory and fed to mma.m8n8k4 as both operands (G += S S^T, four codewords per instruction), so
// the accumulator costs two registers per 8 x 8 tile and the streaming loop needs no CTA barrier.
template <typename T, int RT>
__global__ void __launch_bounds__(kThreads, RT <= 8 ? 4 : (RT <= 24 ? 2 : 1)) syndrome_gram_kernel(SyndromeParams prm) {
    constexpr int NT = RT / 8;                          // 8 x 8 tiles per side of the Gram matrix
    constexpr int LD = RT + 4;                          // row pitch of the staging buffer (bank spread)
    constexpr int kWarps = kThreads / 32;
    extern __shared__ __align__(16) double sm[];
    double* sH = sm;                                    // [P][RT] node-major, rows >= R are zero
    double* sS = sm + RT * prm.P;                       // [kWarps][32][LD]
    double* sG = sS + kWarps * 32 * LD;                 // [RT][RT] CTA total
    for (int i = threadIdx.x; i < RT * prm.P; i += kThreads) {
        const int pnode = i / RT, r = i % RT;
        sH[i] = r < prm.R ? prm.H[r * prm.P + pnode] : 0.0;
    }
    for (int i = threadIdx.x; i < RT * RT; i += kThreads) sG[i] = 0.0;
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double* myS = sS + warp * 32 * LD;
    double acc[NT][NT][2];
#pragma unroll
    for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int b = 0; b < NT; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
    unsigned long long bad_all = 0ULL;
    unsigned int my_active = 0;
    const T* Z = reinterpret_cast<const T*>(prm.Z);
    const int64_t n_batches = (prm.L + kThreads - 1) / kThreads;
    for (int64_t batch = blockIdx.x; batch < n_batches; batch += gridDim.x) {
        const int64_t l = batch * kThreads + threadIdx.x;
        {   // The syndrome registers leave room for few loads in flight per thread, so the codeword of this
            // thread's next trip is asked for now and waits in L2 when its loads are issued.
            const int64_t ln = l + (int64_t)gridDim.x * kThreads;
            if (RT > 8 && ln < prm.L) {          // up to eight parity checks: nine loads in flight already, no gain
                const T* zn = Z + ln;
                for (int pn = 0; pn < prm.P; ++pn, zn += prm.L) asm volatile("prefetch.global.L2 [%0];" ::"l"(zn));
            }
        }
        double s[RT];
        double nz = 0.0;
        if (l < prm.L) {
            if (prm.erased == 0ULL) codeword_syndrome<T, RT, false>(Z + l, prm.L, prm.P, sH, 0ULL, s, nz, bad_all);
            if (prm.erased != 0ULL || !(nz < kHugeSquared))
                codeword_syndrome<T, RT, true>(Z + l, prm.L, prm.P, sH, prm.erased, s, nz, bad_all);
        } else {
#pragma unroll
            for (int r = 0; r < RT; ++r) s[r] = 0.0;
        }
        double ns = 0.0;
#pragma unroll
        for (int r = 0; r < RT; ++r) ns = fma(s[r], s[r], ns);
        const bool active = (nz > 0.0) && (ns > prm.tau2 * nz);
        my_active += active ? 1u : 0u;
        if (__any_sync(0xffffffffu, active)) {           // G += sum over the warp's codewords of s s^T / ||z||^2
            const double w = active ? rsqrt(nz) : 0.0;
            double2* row = reinterpret_cast<double2*>(myS + lane * LD);
#pragma unroll
            for (int r = 0; r < RT / 2; ++r) row[r] = make_double2(s[2 * r] * w, s[2 * r + 1] * w);
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {                // codewords 4j .. 4j+3 of the warp
                const double* src = myS + (4 * j + (lane & 3)) * LD + (lane >> 2);
                double f[NT];
#pragma unroll
                for (int a = 0; a < NT; ++a) f[a] = src[8 * a];
#pragma unroll
                for (int a = 0; a < NT; ++a)
#pragma unroll
                    for (int b = a; b < NT; ++b) dmma_m8n8k4(acc[a][b][0], acc[a][b][1], f[a], f[b]);   // upper triangle
            }
            __syncwarp();
        }
    }
    // warp fragments -> CTA total (shared atomics) -> global (one atomic per upper-triangle entry)
#pragma unroll
    for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int b = a; b < NT; ++b) {
            const int r = 8 * a + (lane >> 2), c = 8 * b + 2 * (lane & 3);
            if (acc[a][b][0] != 0.0) atomicAdd(&sG[r * RT + c], acc[a][b][0]);
            if (acc[a][b][1] != 0.0) atomicAdd(&sG[r * RT + c + 1], acc[a][b][1]);
        }
    unsigned int act = my_active;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        act += __shfl_xor_sync(0xffffffffu, act, o);
        bad_all |= __shfl_xor_sync(0xffffffffu, bad_all, o);
    }
    if (lane == 0) {
        if (act) atomicAdd(&prm.counts[0], (unsigned long long)act);
        if (bad_all) atomicOr(&prm.counts[1], bad_all);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < prm.R * prm.R; i += kThreads) {
        const int r = i / prm.R, c = i % prm.R;
        if (r <= c && sG[r * RT + c] != 0.0) atomicAdd(&prm.gram[r * prm.R + c], sG[r * RT + c]);
    }
}

// Streaming pass for more than eight parity checks (the syndrome no longer fits beside enough loads in
// flight in one thread's registers).  A warp takes 32 consecutive output positions at a time and forms their syndromes
// on the FP64 tensor cores: S (RT x 32) = H (RT x P) Z (P x 32) as mma.m8n8k4 tiles, H's fragments from
// shared memory, Z's fragments loaded straight from global memory (a lane owns one node of a k-step
// of four and one of eight positions of a tile; the four tiles of a k-step cover 4 rows x 256 bytes),
// the accumulators in 2 * NT * 4 registers per lane.  Against one thread per codeword with the whole
// syndrome in its registers this needs an eighth of the arithmetic instructions, no shared-memory
// operand reads per node, and leaves registers for many loads in flight.  Squared norms of the
// codewords and of the syndromes are met by shuffles; the zero test follows per position.  The Gram
// matrix of the failing codewords is formed warp by warp on the tensor cores as well: the 32
// scaled syndromes of a warp are staged in shared memory and fed to mma.m8n8k4 as both operands
// (G += S S^T, four codewords per instruction).  A block of positions that holds a non-finite or
// huge value, and every block when nodes are erased, is redone codeword by codeword with the checked
// form above.
template <typename T, int RT>
__global__ void __launch_bounds__(kThreads, RT <= 24 ? 2 : 1) syndrome_gram_mma_kernel(SyndromeParams prm) {
    constexpr int NT = RT / 8;                          // 8 x 8 tiles per side of the Gram matrix
    constexpr int LD = RT + 4;                          // row pitch of the staging buffer (bank spread)
    constexpr int kWarps = kThreads / 32;
    constexpr int UK = 2;                               // k-steps (of four nodes) per chunk of loads; two chunks are in flight
    constexpr int NG = NT * (NT + 1) / 2;               // 8 x 8 tiles of the Gram matrix's upper triangle
    extern __shared__ __align__(16) double sm[];
    double* sH = sm;                                    // [P4][RT] node-major, rows >= R and nodes >= P are zero
    const int P4 = (prm.P + 3) & ~3;
    double* sS = sm + RT * P4;                          // [kWarps][32][LD]
    double* sA = sS + kWarps * 32 * LD;                 // [kWarps][NG][32][2] Gram fragments of every warp (kept out of the registers)
    double* sG = sA + kWarps * NG * 64;                 // [RT][RT] CTA total
    for (int i = threadIdx.x; i < RT * P4; i += kThreads) {
        const int pnode = i / RT, r = i % RT;
        sH[i] = (r < prm.R && pnode < prm.P) ? prm.H[r * prm.P + pnode] : 0.0;
    }
    for (int i = threadIdx.x; i < kWarps * NG * 64; i += kThreads) sA[i] = 0.0;
    for (int i = threadIdx.x; i < RT * RT; i += kThreads) sG[i] = 0.0;
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int kq = lane & 3, nq = lane >> 2;            // node within a k-step / position within a tile (fragment coordinates)
    double* myS = sS + warp * 32 * LD;
    double2* myA = reinterpret_cast<double2*>(sA + warp * NG * 64) + lane;   // fragment g of this lane: myA[32 g]
    unsigned long long bad_all = 0ULL;
    unsigned int my_active = 0;
    const T* Z = reinterpret_cast<const T*>(prm.Z);
    const int n_ksteps = P4 >> 2;
    const int n_chunks = (n_ksteps + UK - 1) / UK;
    const int64_t n_blocks = (prm.L + 31) / 32;
    const int64_t stride = (int64_t)gridDim.x * kWarps;
    double za[UK][4], zb[UK][4];                         // two chunks of loads: one being multiplied, one in flight
    bool have_first = false;                             // za already holds (or awaits) chunk 0 of the current block
    for (int64_t blk = (int64_t)blockIdx.x * kWarps + warp; blk < n_blocks; blk += stride) {
        const int64_t base = blk * 32;
        bool any_active = false;
        bool redo = prm.erased != 0ULL;
        if (!redo) {
            {   // this warp's next block: asked for now, waiting in L2 when its loads are issued
                const int64_t nb = (blk + stride) * 32 + 8 * kq;       // lane (kq, nq): 64-byte piece kq of node nq, nq + 8, ...
                if (nb < prm.L)
                    for (int pn = nq; pn < prm.P; pn += 8) asm volatile("prefetch.global.L2 [%0];" ::"l"(Z + (int64_t)pn * prm.L + nb));
            }
            double d[NT][4][2];                          // syndromes: rows 8 mt + nq, positions 8 t + 2 kq + {0, 1}
            double pz[4] = {0.0, 0.0, 0.0, 0.0};         // this lane's share of ||z||^2 of position 8 t + nq
#pragma unroll
            for (int mt = 0; mt < NT; ++mt)
#pragma unroll
                for (int t = 0; t < 4; ++t) d[mt][t][0] = d[mt][t][1] = 0.0;
            auto load_chunk = [&](int64_t b0, int c, double (&z)[UK][4]) {
#pragma unroll
                for (int u = 0; u < UK; ++u) {
                    const int ks = c * UK + u, node = 4 * ks + kq;
                    const T* zp = Z + (int64_t)node * prm.L + b0 + nq;
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        z[u][t] = (ks < n_ksteps && node < prm.P && b0 + 8 * t + nq < prm.L) ? (double)__ldcs(zp + 8 * t) : 0.0;
                }
            };
            auto use_chunk = [&](int c, const double (&z)[UK][4]) {
#pragma unroll
                for (int u = 0; u < UK; ++u) {
                    const int ks = c * UK + u;
                    if (ks < n_ksteps) {                 // warp-uniform
                        const double* hp = sH + (4 * ks + kq) * RT + nq;
#pragma unroll
                        for (int t = 0; t < 4; ++t) pz[t] = fma(z[u][t], z[u][t], pz[t]);
#pragma unroll
                        for (int mt = 0; mt < NT; ++mt) {
                            const double h = hp[8 * mt];
#pragma unroll
                            for (int t = 0; t < 4; ++t) dmma_m8n8k4(d[mt][t][0], d[mt][t][1], h, z[u][t]);
                        }
                    }
                }
            };
            if (!have_first) load_chunk(base, 0, za);
            have_first = false;
            for (int c = 0; c < n_chunks; c += 2) {
                if (c + 1 < n_chunks) load_chunk(base, c + 1, zb);
                use_chunk(c, za);
                if (c + 2 < n_chunks) {
                    load_chunk(base, c + 2, za);
                } else if (blk + stride < n_blocks) {
                    // za is free: the first chunk of this warp's next block travels while the rest of
                    // this block is multiplied, tested and added to the Gram matrix
                    load_chunk((blk + stride) * 32, 0, za);
                    have_first = true;
                }
                if (c + 1 < n_chunks) use_chunk(c + 1, zb);
            }
            // ||z||^2 of position 8 t + nq: sum over the four lanes of the position
            bool huge = false;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                pz[t] += __shfl_xor_sync(0xffffffffu, pz[t], 1);
                pz[t] += __shfl_xor_sync(0xffffffffu, pz[t], 2);
                huge |= !(pz[t] < kHugeSquared);
            }
            redo = __any_sync(0xffffffffu, huge);
            if (!redo) {
                bool act_any = false;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        double ns = 0.0;                 // ||s||^2 of position 8 t + 2 kq + e: over the tiles, then over the eight row lanes
#pragma unroll
                        for (int mt = 0; mt < NT; ++mt) ns = fma(d[mt][t][e], d[mt][t][e], ns);
                        ns += __shfl_xor_sync(0xffffffffu, ns, 4);
                        ns += __shfl_xor_sync(0xffffffffu, ns, 8);
                        ns += __shfl_xor_sync(0xffffffffu, ns, 16);
                        const double nz = __shfl_sync(0xffffffffu, pz[t], (2 * kq + e) * 4);
                        const bool active = (nz > 0.0) && (ns > prm.tau2 * nz);
                        act_any |= active;
                        if (nq == 0) my_active += active ? 1u : 0u;     // one of the eight row lanes counts
                        const double w = active ? rsqrt(nz) : 0.0;
#pragma unroll
                        for (int mt = 0; mt < NT; ++mt) d[mt][t][e] *= w;
                    }
                }
                any_active = __any_sync(0xffffffffu, act_any);
                if (any_active) {
#pragma unroll
                    for (int t = 0; t < 4; ++t)
#pragma unroll
                        for (int e = 0; e < 2; ++e)
#pragma unroll
                            for (int mt = 0; mt < NT; ++mt) myS[(8 * t + 2 * kq + e) * LD + 8 * mt + nq] = d[mt][t][e];
                }
            }
        }
        if (redo) {                                      // lane = position, checked values
            const int64_t l = base + lane;
            double s[RT];
            double nz = 0.0;
            if (l < prm.L) {
                codeword_syndrome<T, RT, true>(Z + l, prm.L, prm.P, sH, prm.erased, s, nz, bad_all);
            } else {
#pragma unroll
                for (int r = 0; r < RT; ++r) s[r] = 0.0;
            }
            double ns = 0.0;
#pragma unroll
            for (int r = 0; r < RT; ++r) ns = fma(s[r], s[r], ns);
            const bool active = (nz > 0.0) && (ns > prm.tau2 * nz);
            my_active += active ? 1u : 0u;
            any_active = __any_sync(0xffffffffu, active);
            if (any_active) {
                const double w = active ? rsqrt(nz) : 0.0;
                double2* row = reinterpret_cast<double2*>(myS + lane * LD);
#pragma unroll
                for (int r = 0; r < RT / 2; ++r) row[r] = make_double2(s[2 * r] * w, s[2 * r + 1] * w);
            }
        }
        if (any_active) {                                // G += sum over the block's codewords of s s^T / ||z||^2
            __syncwarp();
            double acc[NG][2];
#pragma unroll
            for (int g = 0; g < NG; ++g) { const double2 v = myA[32 * g]; acc[g][0] = v.x; acc[g][1] = v.y; }
#pragma unroll
            for (int j = 0; j < 8; ++j) {                // codewords 4j .. 4j+3 of the block
                const double* src = myS + (4 * j + (lane & 3)) * LD + (lane >> 2);
                double f[NT];
#pragma unroll
                for (int a = 0; a < NT; ++a) f[a] = src[8 * a];
                int g = 0;
#pragma unroll
                for (int a = 0; a < NT; ++a)
#pragma unroll
                    for (int b = a; b < NT; ++b, ++g) dmma_m8n8k4(acc[g][0], acc[g][1], f[a], f[b]);   // upper triangle
            }
#pragma unroll
            for (int g = 0; g < NG; ++g) myA[32 * g] = make_double2(acc[g][0], acc[g][1]);
            __syncwarp();
        }
    }
    // warp fragments -> CTA total (shared atomics) -> global (one atomic per upper-triangle entry)
    {
        int g = 0;
#pragma unroll
        for (int a = 0; a < NT; ++a)
#pragma unroll
            for (int b = a; b < NT; ++b, ++g) {
                const double2 v = myA[32 * g];
                const int r = 8 * a + (lane >> 2), c = 8 * b + 2 * (lane & 3);
                if (v.x != 0.0) atomicAdd(&sG[r * RT + c], v.x);
                if (v.y != 0.0) atomicAdd(&sG[r * RT + c + 1], v.y);
            }
    }
    unsigned int act = my_active;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        act += __shfl_xor_sync(0xffffffffu, act, o);
        bad_all |= __shfl_xor_sync(0xffffffffu, bad_all, o);
    }
    if (lane == 0) {
        if (act) atomicAdd(&prm.counts[0], (unsigned long long)act);
        if (bad_all) atomicOr(&prm.counts[1], bad_all);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < prm.R * prm.R; i += kThreads) {
        const int r = i / prm.R, c = i % prm.R;
        if (r <= c && sG[r * RT + c] != 0.0) atomicAdd(&prm.gram[r * prm.R + c], sG[r * RT + c]);
    }
}

struct FinishParams {
    const double* H;            // [R][P]
    const double* gram;         // upper triangle filled
    const unsigned long long* counts;
    gpd_locate_result* result;
    int P, R;
    double tau2, tau_in;
    unsigned long long erased;
};

// Shared memory of the finish kernel for R parity checks and P nodes (doubles first, then ints, bytes).
__host__ __device__ inline size_t finish_smem_bytes(int R, int P) {
    const int ld = R | 1;
    return sizeof(double) * ((size_t)4 * R * ld + 2 * (size_t)R * P + (size_t)R + (size_t)P) +
           sizeof(int) * ((size_t)P + (size_t)R) + (size_t)P;
}

// One warp.  The Gram matrix G of the failing codewords has rank = number of erroneous nodes (a
// few) plus a noise floor far below the threshold.  A diagonally pivoted Cholesky factorisation
// G = L L^T + (remainder below 2^-30 of the eigenvalue threshold) gives its numerical rank (pivots
// above the threshold) and its range (the leading columns of L); the verification uses
// ||(I - Pi) L||_F^2 = tr((I - Pi) L L^T (I - Pi)).
__global__ void __launch_bounds__(32) locate_finish_kernel(FinishParams prm) {
    extern __shared__ __align__(16) double fs[];
    const int lane = threadIdx.x;
    const int R = prm.R, P = prm.P, ld = R | 1;
    double* A = fs;                          // [R][ld] G -> Schur complement; fallback search: L with span(H_base) projected out
    double* Lm = A + R * ld;                 // [R][ld] Cholesky columns
    double* M = Lm + R * ld;                 // [R][ld] orthonormal basis of span(H_A) (verification, fallback search)
    double* U = M + R * ld;                  // [R][ld] orthonormal basis of the retained subspace in columns
    double* Hs = U + R * ld;                 // [R][P]
    double* Hp = Hs + R * P;                 // [R][P] fallback search: H with span(H_base) projected out
    double* lam = Hp + R * P;                // [R] pivots of the factorisation
    double* dist = lam + R;                  // [P]
    int* free_nodes = reinterpret_cast<int*>(dist + P);   // [P] fallback search: nodes outside the base set, increasing
    int* comb = free_nodes + P;              // [R] fallback search: current combination (indices into free_nodes)
    unsigned char* inside = reinterpret_cast<unsigned char*>(comb + R);   // [P]
    gpd_locate_result* res = prm.result;
    const unsigned long long n_active = prm.counts[0];
    const unsigned long long forced = prm.counts[1] | prm.erased;
    const int n_forced = __popcll(forced);

    // header fields common to every exit
    for (int p = lane; p < kMaxNodes; p += 32) {
        res->forced[p] = (p < P && ((forced >> p) & 1ULL)) ? 1 : 0;
        res->flagged[p] = res->forced[p];
    }
    if (lane == 0) {
        res->n_active = (int64_t)n_active;
        res->device_status = 0;
        res->rank = 0;
        res->residual = 0.0;
        res->max_inside = 0.0;
        res->min_outside = 0.0;
        res->n_flagged = n_forced;
    }
    if (n_active == 0ULL && forced == 0ULL) {
        if (lane == 0) res->outcome = GPD_NO_ERROR;
        return;
    }
    const int budget = R - 1;
    if (n_forced > budget) {
        if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
        return;
    }
    for (int i = lane; i < R * P; i += 32) Hs[i] = prm.H[i];
    for (int i = lane; i < R * R; i += 32) {
        const int r = i / R, c = i % R;
        A[r * ld + c] = prm.gram[r <= c ? r * R + c : c * R + r];
    }
    __syncwarp();
    const int lane_i = lane / R, lane_j = lane % R, step_i = 32 / R, step_j = 32 % R;   // entry lane + 32 k of an R x R matrix

    int rank = 0, nl = 0;
    unsigned long long flagged = forced;
    double max_in = 0.0, min_out = 1e300, remainder = 0.0;
    if (n_active > 0ULL) {
        const double theta = prm.tau2 * (double)n_active / (double)R;     // eigenvalue threshold
        // ---- diagonally pivoted Cholesky: G = L L^T + remainder -------------------------------
        const double stop = theta * 9.313225746154785e-10;                // 2^-30
        unsigned int used = 0u;
        for (int k = 0; k < R; ++k) {
            const bool mine = lane < R && !((used >> lane) & 1u);
            double v = mine ? A[lane * ld + lane] : -1.0;
            int idx = lane;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double ov = __shfl_xor_sync(0xffffffffu, v, o);
                const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
                if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
            }
            if (!(v > stop)) break;
            if (lane == 0) lam[nl] = v;                                     // pivot of this step
            const double li = mine ? A[lane * ld + idx] * rsqrt(v) : 0.0;   // rows of earlier pivots are zero
            if (lane < R) Lm[lane * ld + nl] = li;
            __syncwarp();
            for (int e = lane, i = lane_i, c = lane_j; e < R * R; e += 32, i += step_i, c += step_j) {
                if (c >= R) { c -= R; ++i; }
                A[i * ld + c] -= Lm[i * ld + nl] * Lm[c * ld + nl];
            }
            used |= 1u << idx;
            ++nl;
            __syncwarp();
        }
        {   // what the factorisation left: trace of the Schur complement (every eigenvalue of it is below `stop` R)
            double d = (lane < R && !((used >> lane) & 1u)) ? fmax(A[lane * ld + lane], 0.0) : 0.0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            remainder = d;
        }
        // ---- numerical rank: pivots above the eigenvalue threshold ---------------------------------
        // The pivots of the diagonally pivoted factorisation are non-increasing and bracket the
        // eigenvalues from below up to the dimension: lambda_k / (R - k + 1) <= d_k, and the pivots past
        // the true rank are at the level of what is left (the noise floor).  Erroneous nodes put
        // eigenvalues orders of magnitude above the threshold and the floor lies orders below it, so
        // counting pivots gives the count of eigenvalues above the threshold without an eigen-solver.
        for (int k = 0; k < nl; ++k) rank += lam[k] > theta ? 1 : 0;
        if (lane == 0) res->rank = rank;
        if (rank > budget) {
            if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
            return;
        }
        // ---- retained subspace: the first `rank` columns of L, orthonormalised --------------------
        // (columns of the Gram matrix with earlier pivots projected out: they span its range up to
        // the floor, as the leading eigenvectors do)
        for (int e = 0; e < rank; ++e) {
            double u = lane < R ? Lm[lane * ld + e] : 0.0;
            for (int pass = 0; pass < 2; ++pass) {
                for (int f = 0; f < e; ++f) {
                    double part = lane < R ? U[lane * ld + f] * u : 0.0;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                    if (lane < R) u -= part * U[lane * ld + f];
                }
            }
            double nn = u * u;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
            if (lane < R) U[lane * ld + e] = u * rsqrt(nn);
            __syncwarp();
        }
        // ---- distance of every H_p to the retained subspace --------------------------------
        for (int p = lane; p < P; p += 32) {
            double hn = 0.0;
            for (int r = 0; r < R; ++r) hn += Hs[r * P + p] * Hs[r * P + p];
            double resid[kMaxR];
            for (int r = 0; r < R; ++r) resid[r] = Hs[r * P + p];
            for (int pass = 0; pass < 2; ++pass) {           // project twice (re-orthogonalisation)
                for (int e = 0; e < rank; ++e) {
                    double dot = 0.0;
                    for (int r = 0; r < R; ++r) dot += U[r * ld + e] * resid[r];
                    for (int r = 0; r < R; ++r) resid[r] -= dot * U[r * ld + e];
                }
            }
            double rn = 0.0;
            for (int r = 0; r < R; ++r) rn += resid[r] * resid[r];
            dist[p] = sqrt(rn / hn);
            inside[p] = dist[p] <= prm.tau_in ? 1 : 0;
        }
        __syncwarp();
        int n_inside = 0;
        for (int base = 0; base < P; base += 32) {       // lanes over nodes: support mask and the two extremes
            const int p = base + lane;
            const bool in = p < P && inside[p];
            const unsigned int m = __ballot_sync(0xffffffffu, in);
            n_inside += __popc(m);
            flagged |= (unsigned long long)m << base;
            double mi = in ? dist[p] : 0.0, mo = (p < P && !in) ? dist[p] : 1e300;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                mi = fmax(mi, __shfl_xor_sync(0xffffffffu, mi, o));
                mo = fmin(mo, __shfl_xor_sync(0xffffffffu, mo, o));
            }
            max_in = fmax(max_in, mi);
            min_out = fmin(min_out, mo);
        }
        if (lane == 0) { res->max_inside = max_in; res->min_outside = min_out; }
        if (n_inside != rank) {
            // Rank-deficient error matrix (errors of several nodes confined to fewer codewords than
            // nodes): fewer columns of H lie in the syndromes' range than its rank.  Those that do
            // are erroneous all the same, so Algorithm 1's search is run over the supports that
            // contain them: by increasing size, lexicographic within a size, the first support
            // that leaves no syndrome energy outside its span is taken.  A size is only searched
            // while the running number of supports stays within kMaxFallbackSupports.
            const int nb = __popcll(flagged);
            bool found = false;
            if (nb <= budget) {
                const double limit_fb = prm.tau2 * (double)n_active;
                // orthonormal basis of span(H_base) in the columns of M (twice-applied Gram-Schmidt)
                int na0 = 0;
                for (int p = 0; p < P; ++p) {
                    if (!((flagged >> p) & 1ULL)) continue;
                    double v = lane < R ? Hs[lane * P + p] : 0.0;
                    for (int pass = 0; pass < 2; ++pass)
                        for (int e = 0; e < na0; ++e) {
                            const double qe = lane < R ? M[lane * ld + e] : 0.0;
                            double part = qe * v;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                            v -= part * qe;
                        }
                    double nn = v * v;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
                    if (lane < R) M[lane * ld + na0] = v * rsqrt(nn);
                    __syncwarp();
                    ++na0;
                }
                // A <- (I - Pi_base) L (column k of the Cholesky factor, lane = row); Hp <- (I - Pi_base) H
                double base_res = 0.0;
                for (int k = 0; k < nl; ++k) {
                    double v = lane < R ? Lm[lane * ld + k] : 0.0;
                    for (int pass = 0; pass < 2; ++pass)
                        for (int e = 0; e < na0; ++e) {
                            const double qe = lane < R ? M[lane * ld + e] : 0.0;
                            double part = qe * v;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                            v -= part * qe;
                        }
                    if (lane < R) A[lane * ld + k] = v;
                    base_res = fma(v, v, base_res);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) base_res += __shfl_xor_sync(0xffffffffu, base_res, o);
                int n_free = 0;
                for (int p = 0; p < P; ++p) {
                    if ((flagged >> p) & 1ULL) continue;
                    double v = lane < R ? Hs[lane * P + p] : 0.0;
                    for (int pass = 0; pass < 2; ++pass)
                        for (int e = 0; e < na0; ++e) {
                            const double qe = lane < R ? M[lane * ld + e] : 0.0;
                            double part = qe * v;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                            v -= part * qe;
                        }
                    if (lane < R) Hp[lane * P + p] = v;
                    if (lane == 0) free_nodes[n_free] = p;
                    ++n_free;
                }
                __syncwarp();
                long long tried = 1;                                     // the base set itself
                if (base_res + remainder <= limit_fb) found = true;
                for (int ex = 1; !found && nb + ex <= budget && ex <= n_free; ++ex) {
                    // number of supports of this size: C(n_free, ex), computed exactly while it stays small
                    long long cnt = 1;
                    for (int i = 1; i <= ex; ++i) {
                        cnt = cnt * (n_free - ex + i) / i;
                        if (cnt > 4LL * kMaxFallbackSupports * 64) break;   // far beyond the bound: stop before it can overflow
                    }
                    tried += cnt;
                    if (tried > kMaxFallbackSupports) break;
                    if (lane < ex) comb[lane] = lane;
                    __syncwarp();
                    int redo = 0;                                        // columns U[.][redo ..] must be rebuilt
                    while (true) {
                        // orthonormalise the projected columns of this combination (columns of U)
                        for (int j = redo; j < ex; ++j) {
                            double v = lane < R ? Hp[lane * P + free_nodes[comb[j]]] : 0.0;
                            for (int pass = 0; pass < 2; ++pass)
                                for (int e = 0; e < j; ++e) {
                                    const double qe = lane < R ? U[lane * ld + e] : 0.0;
                                    double part = qe * v;
#pragma unroll
                                    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                                    v -= part * qe;
                                }
                            double nn = v * v;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
                            if (lane < R) U[lane * ld + j] = nn > 0.0 ? v * rsqrt(nn) : 0.0;
                            __syncwarp();
                        }
                        // syndrome energy outside span(H_base, H_combination)
                        double rr = 0.0;
                        for (int k = 0; k < nl; ++k) {
                            double v = lane < R ? A[lane * ld + k] : 0.0;
                            for (int e = 0; e < ex; ++e) {
                                const double qe = lane < R ? U[lane * ld + e] : 0.0;
                                double part = qe * v;
#pragma unroll
                                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                                v -= part * qe;
                            }
                            rr = fma(v, v, rr);
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) rr += __shfl_xor_sync(0xffffffffu, rr, o);
                        if (rr + remainder <= limit_fb) {
                            for (int j = 0; j < ex; ++j) flagged |= 1ULL << free_nodes[comb[j]];
                            found = true;
                            break;
                        }
                        // next combination in lexicographic order (every lane takes the same steps)
                        int j = ex - 1;
                        while (j >= 0 && comb[j] == n_free - ex + j) --j;
                        if (j < 0) break;
                        __syncwarp();
                        if (lane == 0) {
                            ++comb[j];
                            for (int i = j + 1; i < ex; ++i) comb[i] = comb[i - 1] + 1;
                        }
                        redo = j;
                        __syncwarp();
                    }
                }
            }
            if (!found) {
                if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
                return;
            }
        }
    }
    const int n_flagged = __popcll(flagged);
    if (n_flagged > budget) {
        if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
        return;
    }
    // ---- verification: syndrome energy outside span(H_A), A = flagged nodes ------------------
    // Orthonormal basis of span(H_A) by twice-applied modified Gram-Schmidt (columns of Qa).
    double* Qa = M;
    int na = 0;
    for (int p = 0; p < P; ++p) {
        if (!((flagged >> p) & 1ULL)) continue;
        if (lane < R) Qa[lane * ld + na] = Hs[lane * P + p];
        __syncwarp();
        for (int pass = 0; pass < 2; ++pass) {
            for (int e = 0; e < na; ++e) {
                double part = lane < R ? Qa[lane * ld + e] * Qa[lane * ld + na] : 0.0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane < R) Qa[lane * ld + na] -= part * Qa[lane * ld + e];
                __syncwarp();
            }
        }
        double nn = lane < R ? Qa[lane * ld + na] * Qa[lane * ld + na] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
        if (lane < R) Qa[lane * ld + na] *= rsqrt(nn);
        __syncwarp();
        ++na;
    }
    double residual = 0.0;
    if (n_active > 0ULL) {
        // tr((I-Pi) G (I-Pi)) = ||(I-Pi) L||_F^2 + (what is left of the remainder: at most its trace).
        // Lane k projects column k of L, in place.
        if (lane < nl) {
            for (int pass = 0; pass < 2; ++pass) {
                for (int e = 0; e < na; ++e) {
                    double dot = 0.0;
                    for (int r = 0; r < R; ++r) dot += Qa[r * ld + e] * Lm[r * ld + lane];
                    for (int r = 0; r < R; ++r) Lm[r * ld + lane] -= dot * Qa[r * ld + e];
                }
            }
            for (int r = 0; r < R; ++r) residual += Lm[r * ld + lane] * Lm[r * ld + lane];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) residual += __shfl_xor_sync(0xffffffffu, residual, o);
        residual += remainder;
    }
    const double limit = prm.tau2 * (double)(n_active > 0ULL ? n_active : 1ULL);
    if (lane == 0) {
        res->residual = residual / (double)(n_active > 0ULL ? n_active : 1ULL);
        res->n_flagged = residual > limit ? n_forced : n_flagged;
        res->outcome = residual > limit ? GPD_DECODE_FAILURE : GPD_CORRECTED;
    }
    if (residual <= limit)
        for (int p = lane; p < P; p += 32) res->flagged[p] = (flagged >> p) & 1ULL ? 1 : 0;
}

inline gpd_status launch_finish(const FinishParams& fp, cudaStream_t st) {
    const size_t smem = finish_smem_bytes(fp.R, fp.P);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(locate_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return GPD_ERR_CUDA;
    locate_finish_kernel<<<1, 32, smem, st>>>(fp);
    return launch_ok();
}

template <typename T, int RT>
gpd_status launch_syndrome(const SyndromeParams& prm, cudaStream_t st) {
    if constexpr (RT <= 8) {
        const size_t smem = sizeof(double) * ((size_t)RT * prm.P + (size_t)kThreads * (RT + 4) + (size_t)RT * RT);
        const int64_t batches = (prm.L + kThreads - 1) / kThreads;
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(batches, sm_count() * 4));
        syndrome_gram_kernel<T, RT><<<grid, kThreads, smem, st>>>(prm);
    } else {
        constexpr int NG = (RT / 8) * (RT / 8 + 1) / 2;
        const size_t smem = sizeof(double) * ((size_t)RT * ((prm.P + 3) & ~3) + (size_t)kThreads * (RT + 4) +
                                              (size_t)(kThreads / 32) * NG * 64 + (size_t)RT * RT);
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(syndrome_gram_mma_kernel<T, RT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return GPD_ERR_CUDA;
        const int64_t batches = (prm.L + kThreads - 1) / kThreads;
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(batches, sm_count() * (RT <= 24 ? 2 : 1)));
        syndrome_gram_mma_kernel<T, RT><<<grid, kThreads, smem, st>>>(prm);
    }
    return launch_ok();
}

template <typename T>
gpd_status dispatch_syndrome(const SyndromeParams& prm, cudaStream_t st) {
    if (prm.R <= 8) return launch_syndrome<T, 8>(prm, st);
    if (prm.R <= 16) return launch_syndrome<T, 16>(prm, st);
    if (prm.R <= 24) return launch_syndrome<T, 24>(prm, st);
    return launch_syndrome<T, 32>(prm, st);
}

}  // namespace

gpd_status locate_launch(gpd_plan_s* plan, gpd_product which, const void* outputs, uint64_t erased_mask,
                         gpd_locate_result* result, void* workspace, cudaStream_t st) {
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
    double* gram = reinterpret_cast<double*>(ws + wl.off_gram);
    unsigned long long* counts = reinterpret_cast<unsigned long long*>(ws + wl.off_counts);
    // Gram matrix and counters start at zero (they sit next to each other in the workspace)
    if (cudaMemsetAsync(ws + wl.off_gram, 0, (size_t)(wl.off_decode - wl.off_gram), st) != cudaSuccess)
        return GPD_ERR_CUDA;
    const double* H = plan->dev.base + pi.off_H;
    if (pi.R > 0) {
        SyndromeParams sp{};
        sp.Z = outputs; sp.H = H; sp.L = pi.br * pi.bc; sp.P = plan->P; sp.R = pi.R;
        sp.tau2 = plan->tau_col * plan->tau_col; sp.erased = erased_mask;
        sp.gram = gram; sp.counts = counts;
        rc = plan->elem_size == 4 ? dispatch_syndrome<float>(sp, st) : dispatch_syndrome<double>(sp, st);
        if (rc != GPD_OK) return rc;
    }
    FinishParams fp{};
    fp.H = H; fp.gram = gram; fp.counts = counts; fp.result = result;
    fp.P = plan->P; fp.R = pi.R; fp.tau2 = plan->tau_col * plan->tau_col; fp.tau_in = plan->tau_in;
    fp.erased = erased_mask;
    return launch_finish(fp, st);
}

// ---------------------------------------------------------------------------------------------
// Variant with built-in scratch: no device allocation anywhere on its path.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxR = GPD_STATIC_MAX_PARITY;
constexpr size_t kStaticGramBytes = sizeof(double) * kStaticMaxR * kStaticMaxR;        // Gram matrix
constexpr size_t kStaticCountBytes = 256;                                               // counters
constexpr size_t kStaticHBytes = sizeof(double) * kStaticMaxR * kMaxNodes;              // parity checks
constexpr size_t kStaticBytes = kStaticGramBytes + kStaticCountBytes + kStaticHBytes;

// One copy per GPU that loads the library, held until the process exits.  Shared by every call of
// gpd_locate_errors_static on that GPU.
static __device__ __align__(256) unsigned char g_locate_scratch[kStaticBytes];

std::mutex g_static_mu;
unsigned char* g_static_ptr[64] = {nullptr};      // device address of g_locate_scratch, per device

// In host code `g_locate_scratch` is only a handle; the device address has to be asked for, with
// the device current, once per device.
gpd_status static_scratch(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GPD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_locate_scratch) != cudaSuccess || !p) return GPD_ERR_CUDA;
        g_static_ptr[dev] = reinterpret_cast<unsigned char*>(p);
    }
    *out = g_static_ptr[dev];
    return GPD_OK;
}

}  // namespace

gpd_status locate_static_launch(gpd_plan_s* plan, gpd_product which, const void* outputs,
                                uint64_t erased_mask, gpd_locate_result* result, cudaStream_t st) {
    if (which != GPD_FWD && which != GPD_BWD && which != GPD_AUDIT) return GPD_ERR_ARG;
    // digit-plane shares: forward product only, except in the training mode (its backward outputs and the
    // FP64 shares that lead W's buffer are plain doubles)
    if (plan->sliced && !plan->train && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;
    const ProductInfo& pi = plan->prod[which];
    if (pi.Q == 0) return GPD_ERR_P_TOO_SMALL;
    if (pi.R > kStaticMaxR) return GPD_ERR_STATIC_LIMIT;
    unsigned char* base = nullptr;
    gpd_status rc = static_scratch(&base);
    if (rc != GPD_OK) return rc;
    double* gram = reinterpret_cast<double*>(base);
    unsigned long long* counts = reinterpret_cast<unsigned long long*>(base + kStaticGramBytes);
    double* H = reinterpret_cast<double*>(base + kStaticGramBytes + kStaticCountBytes);
    // the array keeps the previous call's contents: Gram matrix and counters must start at zero
    if (cudaMemsetAsync(base, 0, kStaticGramBytes + kStaticCountBytes, st) != cudaSuccess) return GPD_ERR_CUDA;
    if (pi.R > 0 &&
        cudaMemcpyAsync(H, pi.H.data(), sizeof(double) * pi.R * plan->P, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GPD_ERR_CUDA;
    if (pi.R > 0) {
        SyndromeParams sp{};
        sp.Z = outputs; sp.H = H; sp.L = pi.br * pi.bc; sp.P = plan->P; sp.R = pi.R;
        sp.tau2 = plan->tau_col * plan->tau_col; sp.erased = erased_mask;
        sp.gram = gram; sp.counts = counts;
        if (plan->elem_size == 4)
            rc = pi.R <= 8 ? launch_syndrome<float, 8>(sp, st) : launch_syndrome<float, 16>(sp, st);
        else
            rc = pi.R <= 8 ? launch_syndrome<double, 8>(sp, st) : launch_syndrome<double, 16>(sp, st);
        if (rc != GPD_OK) return rc;
    }
    FinishParams fp{};
    fp.H = H; fp.gram = gram; fp.counts = counts; fp.result = result;
    fp.P = plan->P; fp.R = pi.R; fp.tau2 = plan->tau_col * plan->tau_col; fp.tau_in = plan->tau_in;
    fp.erased = erased_mask;
    return launch_finish(fp, st);
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_locate_errors(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                                        const uint8_t* erased_host, gpd_locate_result* result_dev,
                                        void* workspace_dev, void* stream) {
    if (!plan || !outputs_dev || !result_dev) return GPD_ERR_ARG;
    if (!workspace_dev) return GPD_ERR_WORKSPACE;
    uint64_t mask = 0;
    if (erased_host)
        for (int p = 0; p < plan->P; ++p)
            if (erased_host[p]) mask |= 1ULL << p;
    return locate_launch(plan, which, outputs_dev, mask, result_dev, workspace_dev, as_stream(stream));
}

extern "C" gpd_status gpd_locate_errors_static(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                                               const uint8_t* erased_host, gpd_locate_result* result_dev,
                                               void* stream) {
    if (!plan || !outputs_dev || !result_dev) return GPD_ERR_ARG;
    uint64_t mask = 0;
    if (erased_host)
        for (int p = 0; p < plan->P; ++p)
            if (erased_host[p]) mask |= 1ULL << p;
    return locate_static_launch(plan, which, outputs_dev, mask, result_dev, as_stream(stream));
}
