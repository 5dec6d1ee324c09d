// Per-codeword error correction under the adversarial model (lemma on real-number error correction:
// a (P, Q) MDS code corrects t = floor((P - Q) / 2) errors of arbitrary value in one codeword;
// section on decoding methods: find the solution of H e = H z with the fewest non-zeros).
// Every output position is one codeword of P node values and is repaired on its own, so different
// positions may blame different nodes.
//
//   1. position_scan_kernel: one thread per position; syndrome r = H z (orthonormal H in shared
//      memory), zero test ||r||^2 <= tau^2 ||z||^2; positions that fail it are appended to a list.
//      The syndromes of the first listed positions are kept beside the list, so that their
//      repair does not read the codeword a second time.
//   2. position_fix_kernel: one thread per listed position.  The code is a polynomial code, so the
//      sparsest solution is found the Reed-Solomon way in real arithmetic: power-sum syndromes
//      S_j = sum_p w_p b_p^j z_p (w the barycentric weights), and for nu = 1 .. t the locator
//      x^nu + sum_i l_i x^i from the Hankel system sum_i l_i S_{j+i} = -S_{j+nu}; its nu smallest
//      values over the points name the support A; the error values are the least-squares solution
//      of H_A e = r; the support is accepted when what is left of r passes the zero test.  The
//      accepted errors are subtracted in place.
//   3. Outcome and counters go into the result struct: written by the last block of the repair
//      kernel to finish (position_finish_kernel when the code has no parity check to scan with).
#include "gpd_internal.h"

namespace gpd {

namespace {

struct PosParams {
    void* Z;                              // [P][L]
    const double* H;                      // [R][P] orthonormal parity check
    const double* Hg;                     // [R][P] power-sum parity check
    const double* points;                 // [P]
    unsigned long long* counters;         // [0] listed, [1] active, [2] corrected, [3] failed, [4] entries,
                                          // [5] largest support, [6] touched-node mask, [7] finished blocks
    unsigned int* list;                   // positions that failed the zero test
    double* rec;                          // [rec_cap][R + 1]: syndrome r and ||z||^2 of the first listed positions
    unsigned long long rec_cap;
    gpd_position_result* result;
    int64_t L;
    int P, R;
    double tau2;
};

template <typename T, int RT>                 // RT: parity checks rounded up to 8, 16 or 32
__global__ void __launch_bounds__(256, RT <= 8 ? 4 : 1) position_scan_kernel(PosParams prm) {
    extern __shared__ __align__(16) double sH[];   // [P][RT] node-major, zero past row R
    for (int i = threadIdx.x; i < RT * prm.P; i += 256) {
        const int pnode = i / RT, j = i - pnode * RT;
        sH[i] = j < prm.R ? prm.H[j * prm.P + pnode] : 0.0;
    }
    __syncthreads();
    const T* Z = reinterpret_cast<const T*>(prm.Z);
    const int lane = threadIdx.x & 31;
    constexpr int U = RT <= 8 ? 10 : 4;           // loads issued together, in groups of equal size
    const int n_groups = (prm.P + U - 1) / U, gs = (prm.P + n_groups - 1) / n_groups;
    // all lanes of a warp run the same rounds (the counters are updated once per warp and round)
    for (int64_t base = (int64_t)blockIdx.x * 256; base < prm.L; base += (int64_t)gridDim.x * 256) {
        const int64_t pos = base + threadIdx.x;
        const bool valid = pos < prm.L;
        double r[RT];
#pragma unroll
        for (int j = 0; j < RT; ++j) r[j] = 0.0;
        double z2 = 0.0;
        bool finite = true;
        if (valid) {
            const T* zp = Z + pos;
            const double* h = sH;
            for (int p0 = 0; p0 < prm.P; p0 += gs, zp += gs * prm.L, h += gs * RT) {
                double z[U];
#pragma unroll
                for (int u = 0; u < U; ++u) z[u] = (u < gs && p0 + u < prm.P) ? (double)__ldcs(zp + u * prm.L) : 0.0;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (u < gs && p0 + u < prm.P) {
                        z2 = fma(z[u], z[u], z2);
                        const double2* hv = reinterpret_cast<const double2*>(h + u * RT);
#pragma unroll
                        for (int j = 0; j < RT / 2; ++j) {
                            const double2 hh = hv[j];
                            r[2 * j] = fma(hh.x, z[u], r[2 * j]);
                            r[2 * j + 1] = fma(hh.y, z[u], r[2 * j + 1]);
                        }
                    }
                }
            }
            if (!(z2 < kHugeSquared)) {           // rare: a non-finite value, or a finite one whose square leaves the FP64 range
                zp = Z + pos;
                for (int p = 0; p < prm.P; ++p, zp += prm.L) finite &= fabs((double)__ldcs(zp)) < kHuge;
            }
        }
        double r2 = 0.0;
#pragma unroll
        for (int j = 0; j < RT; ++j) r2 = fma(r[j], r[j], r2);
        const bool bad = valid && !finite;                    // reported as failed, left untouched
        const bool listed = valid && finite && r2 > prm.tau2 * z2;
        const unsigned int m_bad = __ballot_sync(0xffffffffu, bad), m_list = __ballot_sync(0xffffffffu, listed);
        if (m_bad | m_list) {
            unsigned long long slot = 0ULL;
            if (lane == 0) {
                atomicAdd(&prm.counters[1], (unsigned long long)(__popc(m_bad) + __popc(m_list)));
                if (m_bad) atomicAdd(&prm.counters[3], (unsigned long long)__popc(m_bad));
                if (m_list) slot = atomicAdd(&prm.counters[0], (unsigned long long)__popc(m_list));
            }
            slot = __shfl_sync(0xffffffffu, slot, 0);
            if (listed) {
                const unsigned long long mine = slot + __popc(m_list & ((1u << lane) - 1u));
                prm.list[mine] = (unsigned int)pos;
                if (mine < prm.rec_cap) {             // hand the syndrome over: the repair then needs no second read of z
                    double* rec = prm.rec + mine * (unsigned long long)(prm.R + 1);
#pragma unroll
                    for (int j = 0; j < RT; ++j)
                        if (j < prm.R) rec[j] = r[j];
                    rec[prm.R] = z2;
                }
            }
        }
    }
}

// Gaussian elimination with partial pivoting on the n x (n + 1) system held in a; false when a
// pivot vanishes against the size of the matrix.  Every loop has the compile-time bound TT and
// every index is static after unrolling, so that for small TT the system stays in registers.
template <int TT>
__device__ __forceinline__ bool solve_small(double (&a)[TT][TT + 1], int n, double (&x)[TT]) {
    constexpr int UF = TT <= 4 ? 32 : 1;     // small systems: fully unrolled, register-resident
    double amax = 0.0;
#pragma unroll UF
    for (int i = 0; i < TT; ++i)
#pragma unroll UF
        for (int j = 0; j < TT; ++j)
            if (i < n && j < n) amax = fmax(amax, fabs(a[i][j]));
    if (!(amax > 0.0)) return false;
    bool ok = true;
    double pinv[TT];                         // reciprocal pivots, used again by the back substitution
#pragma unroll UF
    for (int k = 0; k < TT; ++k) {
        if (k < n) {
#pragma unroll UF
            for (int i = k + 1; i < TT; ++i) {                   // bring the largest entry of column k up
                if (i < n && fabs(a[i][k]) > fabs(a[k][k])) {
#pragma unroll UF
                    for (int j = 0; j <= TT; ++j) { const double t = a[k][j]; a[k][j] = a[i][j]; a[i][j] = t; }
                }
            }
            if (fabs(a[k][k]) <= 1e-13 * amax) ok = false;
            const double inv = 1.0 / a[k][k];
            pinv[k] = inv;
#pragma unroll UF
            for (int i = k + 1; i < TT; ++i) {
                if (i < n) {
                    const double f = a[i][k] * inv;
#pragma unroll UF
                    for (int j = 0; j <= TT; ++j)
                        if (j >= k) a[i][j] -= f * a[k][j];
                }
            }
        }
    }
    if (!ok) return false;
#pragma unroll UF
    for (int i = TT - 1; i >= 0; --i) {
        if (i < n) {
            double s = a[i][TT];
#pragma unroll UF
            for (int j = 0; j < TT; ++j)
                if (j > i && j < n) s -= a[i][j] * x[j];
            x[i] = s * pinv[i];
        }
    }
    return true;
}

// Outcome and counters into the result struct, by the threads tid = 0 .. nthr-1 of one block.  The
// counters are read past L1: other blocks' atomics filled them.
__device__ __forceinline__ void write_position_result(const PosParams& prm, int tid, int nthr) {
    gpd_position_result* res = prm.result;
    const unsigned long long active = __ldcg(&prm.counters[1]), failed = __ldcg(&prm.counters[3]);
    if (tid == 0) {
        res->outcome = active == 0ULL ? GPD_NO_ERROR : (failed ? GPD_DECODE_FAILURE : GPD_CORRECTED);
        res->max_errors = (int32_t)__ldcg(&prm.counters[5]);
        res->device_status = 0;
        res->reserved = 0;
        res->n_active = (int64_t)active;
        res->n_corrected = (int64_t)__ldcg(&prm.counters[2]);
        res->n_failed = (int64_t)failed;
        res->n_entries = (int64_t)__ldcg(&prm.counters[4]);
    }
    const unsigned long long touched = __ldcg(&prm.counters[6]);
    for (int p = tid; p < kMaxNodes; p += nthr) res->touched[p] = (p < prm.P && ((touched >> p) & 1ULL)) ? 1 : 0;
}

// A block that has finished takes a ticket; the last one of the grid writes the result.
__device__ __forceinline__ void finish_by_last_block(const PosParams& prm) {
    __shared__ bool s_last;
    __threadfence();                                  // this thread's counter updates and repairs are visible ...
    __syncthreads();                                  // ... and so are those of the whole block
    if (threadIdx.x == 0) {
        s_last = atomicAdd(&prm.counters[7], 1ULL) + 1ULL == (unsigned long long)gridDim.x;
        __threadfence();
    }
    __syncthreads();
    if (s_last) write_position_result(prm, threadIdx.x, blockDim.x);
}

// One round of the repair for a support of exactly NU nodes, everything sized by NU at compile time
// (small codes): locator from the Hankel system, its NU smallest values over the points, least
// squares H_A e = r through the normal equations with one step of refinement, zero test of what is
// left of r.  Same arithmetic, in the same order, as the general form inside position_fix_kernel.
template <int NU, int RT, int TT>
__device__ __forceinline__ bool try_support(const double (&S)[RT], const double (&r)[RT], const double* sH,
                                            const double* sPts, const double* sG, int P, int R, double limit,
                                            int (&nodes)[TT], double (&err)[TT]) {
    static_assert(2 * NU <= RT && NU <= TT, "support size against the parity checks");
    double a[NU][NU + 1], lam[NU];
#pragma unroll
    for (int j = 0; j < NU; ++j) {
#pragma unroll
        for (int i = 0; i < NU; ++i) a[j][i] = S[j + i];
        a[j][NU] = -S[j + NU];
    }
    if (!solve_small<NU>(a, NU, lam)) return false;
    double small_v[NU];
    int nd[NU];
#pragma unroll
    for (int k = 0; k < NU; ++k) { small_v[k] = __longlong_as_double(0x7ff0000000000000LL); nd[k] = 0; }
#pragma unroll 5
    for (int p = 0; p < P; ++p) {
        const double x = sPts[p];
        double v = 1.0;
#pragma unroll
        for (int i = NU - 1; i >= 0; --i) v = fma(v, x, lam[i]);
        v = fabs(v);
        double cv = v < kHuge ? v : kHuge;
        int cn = p;
#pragma unroll
        for (int k = 0; k < NU; ++k) {
            if (cv < small_v[k]) {
                const double tv = small_v[k]; small_v[k] = cv; cv = tv;
                const int tn = nd[k]; nd[k] = cn; cn = tn;
            }
        }
    }
    double gram[NU][NU];
#pragma unroll
    for (int i = 0; i < NU; ++i)
#pragma unroll
        for (int j = 0; j < NU; ++j) gram[i][j] = sG[nd[i] * P + nd[j]];
    double e[NU];
#pragma unroll
    for (int i = 0; i < NU; ++i) e[i] = 0.0;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        double v[RT];
#pragma unroll
        for (int q = 0; q < RT; ++q) {
            double w = r[q];
            if (q < R) {
#pragma unroll
                for (int i = 0; i < NU; ++i) w = fma(-sH[q * P + nd[i]], e[i], w);
            }
            v[q] = w;
        }
#pragma unroll
        for (int i = 0; i < NU; ++i) {
#pragma unroll
            for (int j = 0; j < NU; ++j) a[i][j] = gram[i][j];
            double s2 = 0.0;
#pragma unroll
            for (int q = 0; q < RT; ++q)
                if (q < R) s2 = fma(sH[q * P + nd[i]], v[q], s2);
            a[i][NU] = s2;
        }
        double delta[NU];
        if (!solve_small<NU>(a, NU, delta)) return false;
#pragma unroll
        for (int i = 0; i < NU; ++i) e[i] += delta[i];
    }
    double left = 0.0;
#pragma unroll
    for (int q = 0; q < RT; ++q) {
        if (q < R) {
            double w = r[q];
#pragma unroll
            for (int i = 0; i < NU; ++i) w = fma(-sH[q * P + nd[i]], e[i], w);
            left = fma(w, w, left);
        }
    }
#pragma unroll
    for (int i = 0; i < NU; ++i) { nodes[i] = nd[i]; err[i] = e[i]; }
    return left <= limit;
}

// RT: parity checks rounded up (8 or 32); TT: errors per codeword rounded up (4 or 16).  The
// right-hand side of a system sits in column TT of its rows.
// Small codes (TT <= 4): a block takes 32 positions at a time and has one warp per support size; warp
// nu - 1 tries supports of nu nodes for all 32 (the sizes are tried side by side instead of one after
// the other: a position's repair is a serial chain, and the chain for the largest size is a little over
// half of the sum), and warp 0 then takes, for every position, the smallest size that passed - the
// decision of the sequential search.  Larger codes: 64 positions per block, sizes in turn.
template <typename T, int RT, int TT>
__global__ void __launch_bounds__(128) position_fix_kernel(PosParams prm) {
    constexpr bool kSizesSideBySide = TT <= 4 && RT == 8;
    constexpr int kPerBlock = kSizesSideBySide ? 32 : 64;     // positions a block takes per trip
    __shared__ int s_nodes[kSizesSideBySide ? 4 : 1][32][4];
    __shared__ double s_err[kSizesSideBySide ? 4 : 1][32][4];
    __shared__ unsigned char s_ok[kSizesSideBySide ? 4 : 1][32];
    const int nthr = blockDim.x;
    extern __shared__ double sm[];        // H [R][P], Hg [R][P], points [P], small codes: H^T H [P][P]
    double* sH = sm;
    double* sHg = sm + prm.R * prm.P;
    double* sPts = sHg + prm.R * prm.P;
    double* sT = sPts + prm.P;            // [R][R] = Hg H^T: S = T r, since the rows of Hg lie in the row space of H
    double* sG = sT + prm.R * prm.R;
    if ((unsigned long long)blockIdx.x * kPerBlock >= prm.counters[0]) {   // nothing listed for this block
        finish_by_last_block(prm);
        return;
    }
    for (int i = threadIdx.x; i < prm.R * prm.P; i += nthr) { sH[i] = prm.H[i]; sHg[i] = prm.Hg[i]; }
    for (int i = threadIdx.x; i < prm.P; i += nthr) sPts[i] = prm.points[i];
    __syncthreads();
    constexpr int UF = TT <= 4 ? 32 : 1;     // small codes: loops fully unrolled, everything in registers
    constexpr bool kGramTable = TT <= 4;     // normal equations read their entries from H^T H
    for (int i = threadIdx.x; i < prm.R * prm.R; i += nthr) {
        const int a = i / prm.R, b = i - a * prm.R;
        double s2 = 0.0;
        for (int p = 0; p < prm.P; ++p) s2 = fma(sHg[a * prm.P + p], sH[b * prm.P + p], s2);
        sT[i] = s2;
    }
    if (kGramTable) {
        for (int i = threadIdx.x; i < prm.P * prm.P; i += nthr) {
            const int a = i / prm.P, b = i - a * prm.P;
            double s2 = 0.0;
            for (int q = 0; q < prm.R; ++q) s2 = fma(sH[q * prm.P + a], sH[q * prm.P + b], s2);
            sG[i] = s2;
        }
        __syncthreads();
    }
    T* Z = reinterpret_cast<T*>(prm.Z);
    const int P = prm.P, R = prm.R, t = R / 2;
    const unsigned long long listed = prm.counters[0];
    // all lanes of a warp run the same rounds (the counters are updated once per warp and round)
    for (unsigned long long base = (unsigned long long)blockIdx.x * kPerBlock; base < listed;
         base += (unsigned long long)gridDim.x * kPerBlock) {
        const unsigned long long it = base + (kSizesSideBySide ? (threadIdx.x & 31) : threadIdx.x);
        const bool valid = it < listed;
        const int64_t pos = valid ? prm.list[it] : 0;
        double r[RT], S[RT];
#pragma unroll UF
        for (int j = 0; j < RT; ++j) { r[j] = 0.0; S[j] = 0.0; }
        double z2 = 0.0;
        if (it < prm.rec_cap) {
            // the scan left r and ||z||^2 of this position behind
            const double* rec = prm.rec + it * (unsigned long long)(R + 1);
            if (valid) {
#pragma unroll UF
                for (int j = 0; j < RT; ++j)
                    if (j < R) r[j] = rec[j];
                z2 = rec[R];
            }
#pragma unroll UF
            for (int j = 0; j < RT; ++j) {
                if (j < R) {
                    double s2 = 0.0;
#pragma unroll UF
                    for (int k = 0; k < RT; ++k)
                        if (k < R) s2 = fma(sT[j * R + k], r[k], s2);
                    S[j] = s2;
                }
            }
        }
        // beyond the records: read the codeword again.  Its P values lie L elements apart: several loads
        // are issued before the first is used
        constexpr int U = 9;
        for (int p0 = 0; p0 < P && it >= prm.rec_cap; p0 += U) {
            double zv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) zv[u] = p0 + u < P ? (double)Z[(int64_t)(p0 + u) * prm.L + pos] : 0.0;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (p0 + u < P) {
                    const double z = zv[u];
                    const int p = p0 + u;
                    z2 = fma(z, z, z2);
#pragma unroll UF
                    for (int j = 0; j < RT; ++j) {
                        if (j < R) {
                            r[j] = fma(sH[j * P + p], z, r[j]);
                            S[j] = fma(sHg[j * P + p], z, S[j]);
                        }
                    }
                }
            }
        }
        const double limit = prm.tau2 * z2;
        int accepted = 0;
        int nodes[TT];
        double err[TT];
#pragma unroll UF
        for (int i = 0; i < TT; ++i) { nodes[i] = 0; err[i] = 0.0; }
        if constexpr (kSizesSideBySide) {
            const int wv = threadIdx.x >> 5, ln = threadIdx.x & 31, nu = wv + 1;     // this warp's support size
            bool ok = false;
            if (valid && nu <= t) {
                switch (nu) {                          // one instantiation per support size
                    case 1: ok = try_support<1, RT, TT>(S, r, sH, sPts, sG, P, R, limit, nodes, err); break;
                    case 2: ok = try_support<2, RT, TT>(S, r, sH, sPts, sG, P, R, limit, nodes, err); break;
                    case 3: ok = try_support<3, RT, TT>(S, r, sH, sPts, sG, P, R, limit, nodes, err); break;
                    default: ok = try_support<4, RT, TT>(S, r, sH, sPts, sG, P, R, limit, nodes, err); break;
                }
            }
            s_ok[wv][ln] = ok ? 1 : 0;
#pragma unroll
            for (int i = 0; i < TT; ++i) { s_nodes[wv][ln][i] = nodes[i]; s_err[wv][ln][i] = err[i]; }
            __syncthreads();
            if (wv == 0) {                             // the smallest size that passed, as the search in turn would find
                for (int w2 = 0; w2 < t && accepted == 0; ++w2) {
                    if (s_ok[w2][ln]) {
                        accepted = w2 + 1;
#pragma unroll
                        for (int i = 0; i < TT; ++i) { nodes[i] = s_nodes[w2][ln][i]; err[i] = s_err[w2][ln][i]; }
                    }
                }
            }
        }
#pragma unroll 1
        for (int nu = 1; !kSizesSideBySide && valid && nu <= t && accepted == 0; ++nu) {
            if constexpr (kSizesSideBySide) {
            } else {
                double a[TT][TT + 1], lam[TT];
#pragma unroll UF
                for (int j = 0; j < TT; ++j) {
                    lam[j] = 0.0;
#pragma unroll UF
                    for (int i = 0; i <= TT; ++i) a[j][i] = 0.0;
                }
                // Hankel system of the locator: sum_i l_i S_{j+i} = -S_{j+nu}, j = 0 .. nu-1
                for (int j = 0; j < nu; ++j) {
                    for (int i = 0; i < nu; ++i) a[j][i] = S[j + i];
                    a[j][TT] = -S[j + nu];
                }
                if (!solve_small<TT>(a, nu, lam)) continue;
                // the nu points where the locator is smallest, smallest first (of equal values the lower
                // point): one pass over the points with an insertion into the sorted list kept so far
                {
                    double small_v[TT];
#pragma unroll UF
                    for (int k = 0; k < TT; ++k) { small_v[k] = __longlong_as_double(0x7ff0000000000000LL); nodes[k] = 0; }
#pragma unroll 5
                    for (int p = 0; p < P; ++p) {
                        const double x = sPts[p];
                        double v = 1.0;
#pragma unroll UF
                        for (int i = TT - 1; i >= 0; --i)
                            if (i < nu) v = fma(v, x, lam[i]);
                        v = fabs(v);
                        double cv = v < kHuge ? v : kHuge;       // every point is finite in the list, so each enters once
                        int cn = p;
#pragma unroll UF
                        for (int k = 0; k < TT; ++k) {
                            if (k < nu && cv < small_v[k]) {
                                const double tv = small_v[k]; small_v[k] = cv; cv = tv;
                                const int tn = nodes[k]; nodes[k] = cn; cn = tn;
                            }
                        }
                    }
                }
                // normal equations of H_A e = r: H_A^T H_A does not change between the two passes below
                double gram[TT][TT];
#pragma unroll UF
                for (int i = 0; i < TT; ++i)
#pragma unroll UF
                    for (int j = 0; j < TT; ++j) {
                        double s2 = 0.0;
                        if (i < nu && j < nu) {
                            if (kGramTable) {
                                s2 = sG[nodes[i] * P + nodes[j]];
                            } else {
                                for (int q = 0; q < R; ++q) s2 = fma(sH[q * P + nodes[i]], sH[q * P + nodes[j]], s2);
                            }
                        }
                        gram[i][j] = s2;
                    }
                // least squares H_A e = r through the normal equations, then one step of refinement on the
                // residual (neighbouring nodes make H_A ill-conditioned; the refinement brings the error
                // values back to the accuracy of an orthogonal factorisation)
                bool solved = true;
#pragma unroll UF
                for (int i = 0; i < TT; ++i) err[i] = 0.0;
#pragma unroll 1
                for (int pass = 0; pass < 2 && solved; ++pass) {
                    double v[RT];
#pragma unroll UF
                    for (int q = 0; q < RT; ++q) {
                        double w = r[q];
                        if (q < R) {
#pragma unroll UF
                            for (int i = 0; i < TT; ++i)
                                if (i < nu) w = fma(-sH[q * P + nodes[i]], err[i], w);
                        }
                        v[q] = w;
                    }
#pragma unroll UF
                    for (int i = 0; i < TT; ++i) {
#pragma unroll UF
                        for (int j = 0; j <= TT; ++j) a[i][j] = 0.0;
                        if (i < nu) {
#pragma unroll UF
                            for (int j = 0; j < TT; ++j)
                                if (j < nu) a[i][j] = gram[i][j];
                            double s2 = 0.0;
#pragma unroll UF
                            for (int q = 0; q < RT; ++q)
                                if (q < R) s2 = fma(sH[q * P + nodes[i]], v[q], s2);
                            a[i][TT] = s2;
                        }
                    }
                    double delta[TT];
#pragma unroll UF
                    for (int i = 0; i < TT; ++i) delta[i] = 0.0;
                    solved = solve_small<TT>(a, nu, delta);
                    if (solved) {
#pragma unroll UF
                        for (int i = 0; i < TT; ++i)
                            if (i < nu) err[i] += delta[i];
                    }
                }
                if (!solved) continue;
                double left = 0.0;
#pragma unroll UF
                for (int q = 0; q < RT; ++q) {
                    if (q < R) {
                        double w = r[q];
#pragma unroll UF
                        for (int i = 0; i < TT; ++i)
                            if (i < nu) w = fma(-sH[q * P + nodes[i]], err[i], w);
                        left = fma(w, w, left);
                    }
                }
                if (left <= limit) accepted = nu;
            }
        }
        unsigned long long mask = 0ULL;
#pragma unroll UF
        for (int i = 0; i < TT; ++i) {
            if (i < accepted) {
                T* cell = Z + (int64_t)nodes[i] * prm.L + pos;
                *cell = (T)((double)*cell - err[i]);
                mask |= 1ULL << nodes[i];
            }
        }
        if (kSizesSideBySide && threadIdx.x >= 32) {   // the other sizes' warps: nothing to write back or count
            __syncthreads();                           // (pairs with the barrier at the end of warp 0's trip)
            continue;
        }
        const unsigned int n_fixed = __popc(__ballot_sync(0xffffffffu, valid && accepted > 0));
        const unsigned int n_lost = __popc(__ballot_sync(0xffffffffu, valid && accepted == 0));
        const unsigned int n_ent = __reduce_add_sync(0xffffffffu, (unsigned int)accepted);
        const unsigned int n_max = __reduce_max_sync(0xffffffffu, (unsigned int)accepted);
        const unsigned int m_lo = __reduce_or_sync(0xffffffffu, (unsigned int)mask);
        const unsigned int m_hi = __reduce_or_sync(0xffffffffu, (unsigned int)(mask >> 32));
        if ((threadIdx.x & 31) == 0) {
            if (n_fixed) atomicAdd(&prm.counters[2], (unsigned long long)n_fixed);
            if (n_lost) atomicAdd(&prm.counters[3], (unsigned long long)n_lost);
            if (n_ent) {
                atomicAdd(&prm.counters[4], (unsigned long long)n_ent);
                atomicMax(&prm.counters[5], (unsigned long long)n_max);
                atomicOr(&prm.counters[6], ((unsigned long long)m_hi << 32) | m_lo);
            }
        }
        if (kSizesSideBySide) __syncthreads();         // the result slots are written again in the next trip
    }
    finish_by_last_block(prm);
}

__global__ void position_finish_kernel(PosParams prm) { write_position_result(prm, threadIdx.x, blockDim.x); }

constexpr int64_t kPosHeaderBytes = 256;  // counters

}  // namespace

// Listed positions whose syndrome the scan keeps for the repair: one in 32 (at least 4096); a run
// with more failures than that reads the remaining codewords a second time.
int64_t position_records(int64_t L) { return std::min<int64_t>(L, std::max<int64_t>(4096, L / 32)); }

int64_t position_workspace_bytes(const gpd_plan_s* plan) {
    int64_t L = 0, rec = 0;
    for (int w : {GPD_FWD, GPD_BWD, GPD_AUDIT}) {
        if (plan->prod[w].Q == 0) continue;
        const int64_t Lw = plan->prod[w].br * plan->prod[w].bc;
        L = std::max<int64_t>(L, Lw);
        rec = std::max<int64_t>(rec, position_records(Lw) * (plan->prod[w].R + 1) * (int64_t)sizeof(double));
    }
    return kPosHeaderBytes + (L * 4 + 255) / 256 * 256 + rec;
}

gpd_status correct_positions_launch(gpd_plan_s* plan, gpd_product which, void* outputs, gpd_position_result* result,
                                    void* workspace, cudaStream_t st) {
    if (which != GPD_FWD && which != GPD_BWD && which != GPD_AUDIT) return GPD_ERR_ARG;
    // digit-plane shares: forward product only, except in the training mode (its backward outputs and the
    // FP64 shares that lead W's buffer are plain doubles)
    if (plan->sliced && !plan->train && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;
    const ProductInfo& pi = plan->prod[which];
    if (pi.Q == 0) return GPD_ERR_P_TOO_SMALL;
    const int64_t L = pi.br * pi.bc;
    if (L >= (int64_t)1 << 32) return GPD_ERR_UNSUPPORTED;               // positions are listed as 32-bit indices
    gpd_status rc = ensure_device(plan);
    if (rc != GPD_OK) return rc;
    PosParams prm{};
    prm.Z = outputs;
    prm.H = plan->dev.base + pi.off_H;
    prm.Hg = plan->dev.base + pi.off_Hg;
    prm.points = plan->dev.base + plan->dev.off_points;
    prm.counters = reinterpret_cast<unsigned long long*>(workspace);
    prm.list = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(workspace) + kPosHeaderBytes);
    prm.rec = reinterpret_cast<double*>(reinterpret_cast<char*>(workspace) + kPosHeaderBytes + (L * 4 + 255) / 256 * 256);
    prm.rec_cap = (unsigned long long)position_records(L);
    prm.result = result;
    prm.L = L; prm.P = plan->P; prm.R = pi.R;
    prm.tau2 = plan->tau_col * plan->tau_col;
    if (cudaMemsetAsync(workspace, 0, kPosHeaderBytes, st) != cudaSuccess) return GPD_ERR_CUDA;
    if (pi.R > 0) {
        const int RT = pi.R <= 8 ? 8 : pi.R <= 16 ? 16 : 32;
        const size_t smem1 = sizeof(double) * RT * plan->P;
        const int grid1 = (int)std::max<int64_t>(1, std::min<int64_t>((L + 255) / 256, sm_count() * 8));
        const bool f32 = plan->elem_size == 4;
        if (RT == 8) f32 ? position_scan_kernel<float, 8><<<grid1, 256, smem1, st>>>(prm)
                         : position_scan_kernel<double, 8><<<grid1, 256, smem1, st>>>(prm);
        else if (RT == 16) f32 ? position_scan_kernel<float, 16><<<grid1, 256, smem1, st>>>(prm)
                               : position_scan_kernel<double, 16><<<grid1, 256, smem1, st>>>(prm);
        else f32 ? position_scan_kernel<float, 32><<<grid1, 256, smem1, st>>>(prm)
                 : position_scan_kernel<double, 32><<<grid1, 256, smem1, st>>>(prm);
        if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
        const size_t smem2 = sizeof(double) * (2 * pi.R * plan->P + plan->P + pi.R * pi.R + (pi.R <= 8 ? plan->P * plan->P : 0));
        const int per_block = pi.R <= 8 ? 32 : 64;                       // positions a block takes per trip
        const int grid2 = (int)std::max<int64_t>(1, std::min<int64_t>((L + per_block - 1) / per_block, sm_count() * 8));
        const int threads_small = 32 * std::max(1, pi.R / 2);            // one warp per support size
        if (pi.R <= 8 && smem2 > 40 * 1024) {                            // beside 6 KB of static shared memory: past the default limit
            const cudaError_t e = f32 ? cudaFuncSetAttribute(position_fix_kernel<float, 8, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2)
                                      : cudaFuncSetAttribute(position_fix_kernel<double, 8, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
            if (e != cudaSuccess) return GPD_ERR_CUDA;
        }
        if (pi.R <= 8) f32 ? position_fix_kernel<float, 8, 4><<<grid2, threads_small, smem2, st>>>(prm)
                           : position_fix_kernel<double, 8, 4><<<grid2, threads_small, smem2, st>>>(prm);
        else f32 ? position_fix_kernel<float, 32, 16><<<grid2, 64, smem2, st>>>(prm)
                 : position_fix_kernel<double, 32, 16><<<grid2, 64, smem2, st>>>(prm);
        return launch_ok();                          // the last block of the repair kernel writes the result
    }
    position_finish_kernel<<<1, 64, 0, st>>>(prm);   // no parity checks: nothing was scanned
    return launch_ok();
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_correct_positions(gpd_plan_t plan, gpd_product which, void* outputs_dev,
                                            gpd_position_result* result_dev, void* workspace_dev, void* stream) {
    if (!plan || !outputs_dev || !result_dev) return GPD_ERR_ARG;
    if (!workspace_dev) return GPD_ERR_WORKSPACE;
    return correct_positions_launch(plan, which, outputs_dev, result_dev, workspace_dev, as_stream(stream));
}
