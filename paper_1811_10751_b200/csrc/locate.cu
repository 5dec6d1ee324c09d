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
// Pass 2 (one warp): eigen-decomposition of G by cyclic Jacobi; numerical rank rho; the error
// support is the set of nodes whose parity-check column H_p lies in the span of the top-rho
// eigenvectors (any P-Q columns of H are independent, so for at most P-Q-1 erroneous nodes no
// other column does); the support is verified by the syndrome energy left outside span(H_A).
// More than P-Q-1 nodes, a rank-deficient error matrix or an ambiguous geometry end in a
// declared decoding failure (Theorem 3, third claim).
#include "gpd_internal.h"

namespace gpd {

namespace {

constexpr int kThreads = 256;

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

// Syndrome s = H z and squared norm of one codeword: P loads at stride L, issued eight at a time.
// CHECKED = false is the plain form: no per-value tests, a non-finite value shows up as a non-finite
// norm and the caller repeats the codeword with CHECKED = true, which zeroes non-finite values
// and erased nodes and records the nodes that held a non-finite value.
template <typename T, int RT, bool CHECKED>
__device__ __forceinline__ void codeword_syndrome(const T* zp, int64_t L, int P, const double* sH,
                                                  unsigned long long erased, double (&s)[RT], double& nz,
                                                  unsigned long long& bad) {
    constexpr int U = RT <= 8 ? 8 : 4;                   // loads issued together (fewer where the syndrome fills the registers)
#pragma unroll
    for (int r = 0; r < RT; ++r) s[r] = 0.0;
    nz = 0.0;
    auto absorb = [&](double zz, int pnode, const double* hcol) {
        if (CHECKED) {
            if (!isfinite(zz)) { bad |= 1ULL << pnode; zz = 0.0; }
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
    int p0 = 0;
    for (; p0 + U <= P; p0 += U, zp += U * L, sH += U * RT) {
        double z[U];
#pragma unroll
        for (int u = 0; u < U; ++u) z[u] = (double)__ldcs(zp + u * L);
#pragma unroll
        for (int u = 0; u < U; ++u) absorb(z[u], p0 + u, sH + u * RT);
    }
    if (p0 < P) {                                        // the last P mod U nodes
        double z[U];
#pragma unroll
        for (int u = 0; u < U; ++u) z[u] = (p0 + u < P) ? (double)__ldcs(zp + u * L) : 0.0;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (p0 + u < P) absorb(z[u], p0 + u, sH + u * RT);
    }
}

// One thread per output position (codeword): the syndrome in RT registers, the zero test.  The
// Gram matrix of the failing codewords is formed
// warp by warp on the FP64 tensor cores: the 32 scaled syndromes of a warp are staged in shared
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
        double s[RT];
        double nz = 0.0;
        if (l < prm.L) {
            if (prm.erased == 0ULL) codeword_syndrome<T, RT, false>(Z + l, prm.L, prm.P, sH, 0ULL, s, nz, bad_all);
            if (prm.erased != 0ULL || !isfinite(nz))
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

struct FinishParams {
    const double* H;            // [R][P]
    const double* gram;         // upper triangle filled
    const unsigned long long* counts;
    gpd_locate_result* result;
    int P, R;
    double tau2, tau_in;
    unsigned long long erased;
};

// One warp.  Shared: G[R][R], V[R][R] (eigenvectors in columns), Hs[R][P], Qa[R][R], lam[R].
__global__ void __launch_bounds__(32) locate_finish_kernel(FinishParams prm) {
    __shared__ double G[kMaxR][kMaxR + 1];
    __shared__ double V[kMaxR][kMaxR + 1];
    __shared__ double Qa[kMaxR][kMaxR + 1];
    __shared__ double Hs[kMaxR][kMaxNodes];
    __shared__ double lam[kMaxR];
    __shared__ double rot_c[kMaxR + 1], rot_s[kMaxR + 1];        // per index: row_i <- c row_i + s row_partner
    __shared__ int partner[kMaxR + 1], pair_p[kMaxR / 2 + 1], pair_q[kMaxR / 2 + 1];
    __shared__ int order[kMaxR];
    __shared__ unsigned char inside[kMaxNodes];
    __shared__ double dist[kMaxNodes];
    const int lane = threadIdx.x;
    const int R = prm.R, P = prm.P;
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
    for (int i = lane; i < R * P; i += 32) Hs[i / P][i % P] = prm.H[i];
    for (int i = lane; i < R * R; i += 32) {
        const int r = i / R, c = i % R;
        G[r][c] = prm.gram[r <= c ? r * R + c : c * R + r];
        V[r][c] = r == c ? 1.0 : 0.0;
    }
    __syncwarp();

    double (*Ga)[kMaxR + 1] = G, (*Gb)[kMaxR + 1] = Qa;          // current / next Gram matrix of the Jacobi rounds
    int rank = 0;
    unsigned long long flagged = forced;
    double max_in = 0.0, min_out = 1e300;
    if (n_active > 0ULL) {
        // ---- Jacobi: G <- J^T G J, V <- V J ----------------------------------------------
        double tr = 0.0;
        for (int i = 0; i < R; ++i) tr += G[i][i];
        // Rotations of one round act on disjoint index pairs (round-robin pairing of n = R or R + 1
        // indices: n - 1 rounds of n / 2 pairs), so their angles are found side by side (lane = pair)
        // and applied together: every index i gets its partner and the pair (c_i, s_i) with
        // new row_i = c_i row_i + s_i row_partner, and G' = J^T G J is written entry by entry into
        // the other of two buffers (Qa is free until the verification), V column pair by column pair.
        const int n = (R + 1) & ~1, half = n >> 1;
        const int lane_i = lane / R, lane_j = lane % R, step_i = 32 / R, step_j = 32 % R;   // entry e = lane + 32 k is (i, j)
        for (int sweep = 0; sweep < 40; ++sweep) {
            double off = 0.0;
            for (int i = lane; i < R * R; i += 32) {
                const int r = i / R, c = i % R;
                if (r != c) off += Ga[r][c] * Ga[r][c];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
            if (off <= 1e-27 * tr * tr) break;          // off-diagonal mass at the FP64 rounding floor
            for (int rd = 0; rd < n - 1; ++rd) {
                if (lane < half) {
                    const int a = lane == 0 ? n - 1 : (rd + lane) % (n - 1);
                    const int b = lane == 0 ? rd : (rd + n - 1 - lane) % (n - 1);
                    const int p = min(a, b), q = max(a, b);
                    double c = 1.0, sn = 0.0;
                    if (q < R) {
                        const double gpq = Ga[p][q], gpp = Ga[p][p], gqq = Ga[q][q];
                        if (!(fabs(gpq) <= 1e-300 || fabs(gpq) <= 1e-20 * sqrt(fabs(gpp * gqq)))) {
                            // tan of the rotation angle (the root of smaller magnitude) is o2 / den with
                            // den = d + sign(d) hypot(d, o2); cosine and sine follow from (den, o2)
                            // normalised, which takes two reciprocal square roots and no division
                            const double d = gqq - gpp, o2 = 2.0 * gpq, h2 = d * d + o2 * o2;
                            const double den = d + copysign(h2 * rsqrt(h2), d);
                            const double rn = rsqrt(den * den + o2 * o2);
                            c = fabs(den) * rn;
                            sn = copysign(o2, o2 * den) * rn;
                        }
                        rot_c[q] = c; rot_s[q] = sn; partner[q] = p;
                    }
                    rot_c[p] = c; rot_s[p] = -sn; partner[p] = q < R ? q : p;
                    pair_p[lane] = p; pair_q[lane] = q;
                }
                __syncwarp();
                for (int e = lane, i = lane_i, jj = lane_j; e < R * R; e += 32, i += step_i, jj += step_j) {   // G' = J^T G J
                    if (jj >= R) { jj -= R; ++i; }
                    const int ip = partner[i], jp = partner[jj];
                    const double ci = rot_c[i], si = rot_s[i], cj = rot_c[jj], sj = rot_s[jj];
                    const double t0 = ci * Ga[i][jj] + si * Ga[ip][jj];
                    const double t1 = ci * Ga[i][jp] + si * Ga[ip][jp];
                    Gb[i][jj] = (jj == ip && si != 0.0) ? 0.0 : cj * t0 + sj * t1;   // the rotated pair's entry is zero by construction
                }
                for (int it = lane; it < half * R; it += 32) {      // V <- V J (columns p, q)
                    const int t = it / R, i = it - t * R, p = pair_p[t], q = pair_q[t];
                    if (q >= R || rot_s[q] == 0.0) continue;
                    const double c = rot_c[q], sn = rot_s[q];
                    const double va = V[i][p], vb = V[i][q];
                    V[i][p] = c * va - sn * vb;
                    V[i][q] = sn * va + c * vb;
                }
                __syncwarp();
                double (*tmp)[kMaxR + 1] = Ga; Ga = Gb; Gb = tmp;
            }
        }
        // ---- eigenvalues in descending order ---------------------------------------------
        if (lane == 0) {
            for (int i = 0; i < R; ++i) { lam[i] = Ga[i][i]; order[i] = i; }
            for (int i = 1; i < R; ++i) {                    // insertion sort, R <= 32
                const int oi = order[i];
                int j = i - 1;
                while (j >= 0 && lam[order[j]] < lam[oi]) { order[j + 1] = order[j]; --j; }
                order[j + 1] = oi;
            }
        }
        __syncwarp();
        const double theta = prm.tau2 * (double)n_active / (double)R;
        for (int i = 0; i < R; ++i) rank += lam[order[i]] > theta ? 1 : 0;
        if (lane == 0) res->rank = rank;
        if (rank > budget) {
            if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
            return;
        }
        // ---- distance of every H_p to span of the top-rank eigenvectors --------------------
        for (int p = lane; p < P; p += 32) {
            double hn = 0.0;
            for (int r = 0; r < R; ++r) hn += Hs[r][p] * Hs[r][p];
            double resid[kMaxR];
            for (int r = 0; r < R; ++r) resid[r] = Hs[r][p];
            for (int pass = 0; pass < 2; ++pass) {           // project twice (re-orthogonalisation)
                for (int e = 0; e < rank; ++e) {
                    const int col = order[e];
                    double dot = 0.0;
                    for (int r = 0; r < R; ++r) dot += V[r][col] * resid[r];
                    for (int r = 0; r < R; ++r) resid[r] -= dot * V[r][col];
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
            if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
            return;
        }
    }
    const int n_flagged = __popcll(flagged);
    if (n_flagged > budget) {
        if (lane == 0) res->outcome = GPD_DECODE_FAILURE;
        return;
    }
    // ---- verification: syndrome energy outside span(H_A), A = flagged nodes ------------------
    // Orthonormal basis of span(H_A) by twice-applied modified Gram-Schmidt (columns of Qa).
    int na = 0;
    for (int p = 0; p < P; ++p) {
        if (!((flagged >> p) & 1ULL)) continue;
        if (lane < R) Qa[lane][na] = Hs[lane][p];
        __syncwarp();
        for (int pass = 0; pass < 2; ++pass) {
            for (int e = 0; e < na; ++e) {
                double part = lane < R ? Qa[lane][e] * Qa[lane][na] : 0.0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane < R) Qa[lane][na] -= part * Qa[lane][e];
                __syncwarp();
            }
        }
        double nn = lane < R ? Qa[lane][na] * Qa[lane][na] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
        if (lane < R) Qa[lane][na] *= rsqrt(nn);
        __syncwarp();
        ++na;
    }
    double residual = 0.0;
    if (n_active > 0ULL) {
        // tr((I-Pi) G (I-Pi)) = sum_i lambda_i ||(I-Pi) u_i||^2, every term non-negative.
        // Lane i projects eigenvector i (column i of V, in place: V is not needed afterwards).
        if (lane < R) {
            for (int pass = 0; pass < 2; ++pass) {
                for (int e = 0; e < na; ++e) {
                    double dot = 0.0;
                    for (int r = 0; r < R; ++r) dot += Qa[r][e] * V[r][lane];
                    for (int r = 0; r < R; ++r) V[r][lane] -= dot * Qa[r][e];
                }
            }
            double un = 0.0;
            for (int r = 0; r < R; ++r) un += V[r][lane] * V[r][lane];
            residual = fmax(lam[lane], 0.0) * un;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) residual += __shfl_xor_sync(0xffffffffu, residual, o);
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

template <typename T, int RT>
gpd_status launch_syndrome(const SyndromeParams& prm, cudaStream_t st) {
    const size_t smem = sizeof(double) * ((size_t)RT * prm.P + (size_t)kThreads * (RT + 4) + (size_t)RT * RT);
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(syndrome_gram_kernel<T, RT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess)
            return GPD_ERR_CUDA;
    }
    const int64_t batches = (prm.L + kThreads - 1) / kThreads;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(batches, 148 * 4));
    syndrome_gram_kernel<T, RT><<<grid, kThreads, smem, st>>>(prm);
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
    if (plan->sliced && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;   // digit-plane shares: forward product only
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
    locate_finish_kernel<<<1, 32, 0, st>>>(fp);
    return launch_ok();
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
    if (plan->sliced && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;   // digit-plane shares: forward product only
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
    locate_finish_kernel<<<1, 32, 0, st>>>(fp);
    return launch_ok();
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
