// Code construction on the host in FP64: evaluation points, exponent maps, coefficient tables,
// recovery thresholds and parity-check matrices (Section IV, Theorems 1-2; Section V-A).
#include <cmath>
#include <cstring>
#include <new>

#include "gpd_internal.h"
#include "gemm_common.h"
#include "slice_common.h"

namespace gpd {

namespace {

// V[p][e] = b_p^e by repeated multiplication.
std::vector<double> power_table(const std::vector<double>& b, int count) {
    const int P = (int)b.size();
    std::vector<double> V((size_t)P * count);
    for (int p = 0; p < P; ++p) {
        double acc = 1.0;
        for (int e = 0; e < count; ++e) {
            V[(size_t)p * count + e] = acc;
            acc *= b[p];
        }
    }
    return V;
}

// Orthonormal basis (rows of H, R x P) of the left null space of the P x Q Vandermonde matrix:
// Householder-triangularise V, then push the unit vectors e_Q .. e_{P-1} back through the
// reflectors; the images are the last P-Q columns of the full orthogonal factor.
std::vector<double> left_null_space(const std::vector<double>& b, int Q) {
    const int P = (int)b.size();
    const int R = P - Q;
    std::vector<double> H((size_t)std::max(R, 0) * P, 0.0);
    if (R <= 0) return H;
    std::vector<double> A = power_table(b, Q);            // P x Q, row-major
    std::vector<double> vs((size_t)Q * P, 0.0);           // reflector k in vs[k*P + k .. k*P + P-1]
    for (int k = 0; k < Q; ++k) {
        double nrm = 0.0;
        for (int r = k; r < P; ++r) nrm += A[(size_t)r * Q + k] * A[(size_t)r * Q + k];
        nrm = std::sqrt(nrm);
        double* v = &vs[(size_t)k * P];
        const double akk = A[(size_t)k * Q + k];
        const double alpha = akk >= 0.0 ? -nrm : nrm;
        for (int r = k; r < P; ++r) v[r] = A[(size_t)r * Q + k];
        v[k] -= alpha;
        double vn = 0.0;
        for (int r = k; r < P; ++r) vn += v[r] * v[r];
        vn = std::sqrt(vn);
        if (vn > 0.0)
            for (int r = k; r < P; ++r) v[r] /= vn;
        for (int c = k; c < Q; ++c) {                     // A <- (I - 2 v v^T) A
            double dot = 0.0;
            for (int r = k; r < P; ++r) dot += v[r] * A[(size_t)r * Q + c];
            for (int r = k; r < P; ++r) A[(size_t)r * Q + c] -= 2.0 * dot * v[r];
        }
    }
    std::vector<double> x(P);
    for (int j = 0; j < R; ++j) {
        std::fill(x.begin(), x.end(), 0.0);
        x[Q + j] = 1.0;
        for (int k = Q - 1; k >= 0; --k) {                // x <- H_0 H_1 ... H_{Q-1} e_{Q+j}
            const double* v = &vs[(size_t)k * P];
            double dot = 0.0;
            for (int r = k; r < P; ++r) dot += v[r] * x[r];
            for (int r = k; r < P; ++r) x[r] -= 2.0 * dot * v[r];
        }
        for (int p = 0; p < P; ++p) H[(size_t)j * P + p] = x[p];
    }
    return H;
}

int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Row j of the power-sum parity check: w_p b_p^j, j = 0 .. R-1, with w_p = 1 / prod_{q != p} (b_p - b_q)
// scaled to largest magnitude 1.  sum_p w_p b_p^k f(b_p) is the divided difference of x^k f over all
// P points and vanishes when deg(x^k f) <= P - 2, i.e. for every codeword and k <= R - 1.
std::vector<double> power_sum_parity(const std::vector<double>& pts, int R) {
    const int P = (int)pts.size();
    std::vector<double> w(P, 1.0);
    double wmax = 0.0;
    for (int p = 0; p < P; ++p) {
        for (int q = 0; q < P; ++q)
            if (q != p) w[p] /= (pts[p] - pts[q]);
        wmax = std::max(wmax, std::fabs(w[p]));
    }
    std::vector<double> Hg((size_t)R * P);
    for (int p = 0; p < P; ++p) {
        double acc = w[p] / wmax;
        for (int j = 0; j < R; ++j) { Hg[(size_t)j * P + p] = acc; acc *= pts[p]; }
    }
    return Hg;
}

}  // namespace

WorkspaceLayout workspace_layout() {
    WorkspaceLayout w{};
    int64_t off = 0;
    w.off_gram = off;   off = align_up(off + (int64_t)sizeof(double) * kMaxR * kMaxR, 256);
    w.off_counts = off; off = align_up(off + (int64_t)sizeof(unsigned long long) * 8, 256);
    w.off_decode = off; off = align_up(off + (int64_t)sizeof(double) * kMaxWanted * kMaxNodes, 256);
    w.off_flags = off;  off = align_up(off + (int64_t)sizeof(int) * 8, 256);
    w.off_regen = off;  off = align_up(off + (int64_t)sizeof(double) * kMaxNodes * kMaxNodes, 256);
    w.total = off;
    return w;
}

gpd_status ensure_device(gpd_plan_s* plan) {
    std::lock_guard<std::mutex> lock(plan->mu);
    if (plan->uploaded) return GPD_OK;
    std::vector<double> host;
    auto push = [&](const std::vector<double>& v) {
        int64_t off = (int64_t)host.size();
        host.insert(host.end(), v.begin(), v.end());
        while (host.size() % 32) host.push_back(0.0);      // keep every table 256-byte aligned
        return off;
    };
    DeviceTables& d = plan->dev;
    d.off_points = push(plan->points);
    d.off_coefW = push(plan->coefW);
    d.off_coefX = push(plan->coefX);
    d.off_coefDT = push(plan->coefDT);
    d.off_coefDup = push(plan->coefDup);
    d.off_coefXup = push(plan->coefXup);
    for (int w : {GPD_FWD, GPD_BWD, GPD_AUDIT}) plan->prod[w].off_H = push(plan->prod[w].H);
    for (int w : {GPD_FWD, GPD_BWD, GPD_AUDIT}) plan->prod[w].off_Hg = push(plan->prod[w].Hg);
    for (int w : {GPD_FWD, GPD_BWD, GPD_AUDIT}) {
        if (plan->prod[w].Q == 0) continue;
        d.off_dcache[w] = push(std::vector<double>((size_t)plan->prod[w].grid_rows * plan->prod[w].grid_cols * plan->P, 0.0));
    }
    d.off_dcache_gate = push(std::vector<double>(1, 0.0));
    d.n_doubles = (int64_t)host.size();
    if (cudaGetDevice(&plan->device) != cudaSuccess) return GPD_ERR_CUDA;
    const int64_t table_bytes = (int64_t)sizeof(double) * (int64_t)host.size();      // a multiple of 256
    const int64_t scratch_bytes = (plan->elem_size == 4 && !plan->sliced) ? sgemm_3xtf32_scratch_bytes(sm_count()) : 0;
    if (cudaMalloc(&d.base, (size_t)(table_bytes + scratch_bytes)) != cudaSuccess) return GPD_ERR_CUDA;
    d.splitk = scratch_bytes ? reinterpret_cast<char*>(d.base) + table_bytes : nullptr;
    d.splitk_bytes = scratch_bytes;
    if (cudaMemcpy(d.base, host.data(), sizeof(double) * host.size(), cudaMemcpyHostToDevice) !=
        cudaSuccess) {
        cudaFree(d.base);
        d.base = nullptr;
        return GPD_ERR_CUDA;
    }
    if (decode_cache_fill(plan) != GPD_OK || cudaDeviceSynchronize() != cudaSuccess) {
        cudaFree(d.base);
        d.base = nullptr;
        return GPD_ERR_CUDA;
    }
    plan->uploaded = true;
    return GPD_OK;
}

}  // namespace gpd

using namespace gpd;

extern "C" const char* gpd_status_string(gpd_status s) {
    switch (s) {
        case GPD_OK: return "ok";
        case GPD_ERR_ARG: return "invalid argument";
        case GPD_ERR_SHAPE: return "splits do not divide the matrix dimensions";
        case GPD_ERR_POINTS: return "evaluation points repeated or non-finite";
        case GPD_ERR_P_TOO_SMALL: return "fewer nodes than the recovery threshold";
        case GPD_ERR_Q_TOO_LARGE: return "threshold, node count or parity count above the supported maximum";
        case GPD_ERR_WORKSPACE: return "workspace missing";
        case GPD_ERR_CUDA: return "CUDA runtime error";
        case GPD_ERR_TIMEOUT: return "bounded device-side wait expired";
        case GPD_ERR_UNSUPPORTED: return "unsupported combination";
        case GPD_ERR_STATIC_LIMIT:
            return "parity count above GPD_STATIC_MAX_PARITY: the built-in scratch of the no-allocation "
                   "entry point is too small for this product; use gpd_locate_errors with a workspace";
    }
    return "unknown status";
}

extern "C" gpd_status gpd_plan(const gpd_shape* shape, const gpd_split* split, int32_t P,
                               const double* points_host, gpd_precision precision, gpd_plan_t* out) {
    return gpd_plan_subst(shape, split, GPD_SUBST_U_EQ_VN, P, points_host, precision, out);
}

extern "C" gpd_status gpd_plan_subst(const gpd_shape* shape, const gpd_split* split, gpd_substitution subst,
                                     int32_t P, const double* points_host, gpd_precision precision,
                                     gpd_plan_t* out) {
    if (!shape || !split || !out) return GPD_ERR_ARG;
    *out = nullptr;
    if (subst != GPD_SUBST_U_EQ_VN && subst != GPD_SUBST_V_EQ_UM) return GPD_ERR_ARG;
    const bool alt = subst == GPD_SUBST_V_EQ_UM;
    if (precision != GPD_PREC_AUTO && precision != GPD_PREC_FP32 && precision != GPD_PREC_FP64 &&
        precision != GPD_PREC_FP64_SLICED && precision != GPD_PREC_FP64_SLICED40 &&
        precision != GPD_PREC_FP64_SLICED_TRAIN)
        return GPD_ERR_ARG;
    const int m = split->m, n = split->n, d1 = split->d1, d2 = split->d2;
    if (shape->N1 <= 0 || shape->N0 <= 0 || shape->B <= 0 || m <= 0 || n <= 0 || d1 <= 0 || d2 <= 0)
        return GPD_ERR_SHAPE;
    if (shape->N1 % m || shape->N0 % n || shape->B % d1 || shape->B % d2) return GPD_ERR_SHAPE;
    if (P <= 0) return GPD_ERR_P_TOO_SMALL;
    // u = v^n, w = v^(mn): Theorem 2 and the proof of Theorem 6, first case;
    // v = u^m, w = u^(mn): second case (forward and backward tolerances swap roles)
    const int64_t Qf = alt ? (int64_t)m * n * d1 + (int64_t)m * n - m : (int64_t)m * n * d1 + n - 1;
    const int64_t Qb = alt ? (int64_t)m * n * d2 + m - 1 : (int64_t)m * n * (d2 + 1) - n;
    const int64_t Qw = (int64_t)m * n;                     // coefficients of the share polynomial
    if (P > kMaxNodes || Qf > kMaxQ) return GPD_ERR_Q_TOO_LARGE;
    if (m * n > kMaxBlocks || n * d1 > kMaxBlocks || d2 * m > kMaxBlocks || m * d1 > kMaxWanted ||
        d2 * n > kMaxWanted)
        return GPD_ERR_Q_TOO_LARGE;
    if (P < Qf) return GPD_ERR_P_TOO_SMALL;
    if (P - Qf > kMaxR) return GPD_ERR_Q_TOO_LARGE;

    gpd_plan_s* plan = new (std::nothrow) gpd_plan_s();
    if (!plan) return GPD_ERR_ARG;
    plan->shape = *shape;
    plan->split = *split;
    plan->P = P;
    plan->Qf = (int)Qf; plan->Qb = (int)Qb; plan->Qw = (int)Qw;
    plan->points.resize(P);
    if (points_host) {
        for (int p = 0; p < P; ++p) plan->points[p] = points_host[p];
    } else {
        // Chebyshev points of the first kind, mirrored so that b_{P-1-p} = -b_p holds exactly
        const double pi = 3.14159265358979323846;
        for (int p = 0; p < (P + 1) / 2; ++p) {
            const double c = (2 * p + 1 == P) ? 0.0 : std::cos((2.0 * p + 1.0) * pi / (2.0 * P));
            plan->points[p] = c;
            plan->points[P - 1 - p] = -c;
        }
    }
    for (int p = 0; p < P; ++p) {
        if (!std::isfinite(plan->points[p])) { delete plan; return GPD_ERR_POINTS; }
        for (int q = 0; q < p; ++q)
            if (plan->points[p] == plan->points[q]) { delete plan; return GPD_ERR_POINTS; }
    }
    plan->alt_subst = alt;
    plan->points_symmetric = true;
    for (int p = 0; p < P; ++p) plan->points_symmetric &= plan->points[P - 1 - p] == -plan->points[p];
    const bool bwd_ok = (P >= Qb) && (Qb <= kMaxQ) && (P - Qb <= kMaxR);
    const bool audit_ok = (P - Qw <= kMaxR);
    const int64_t q_for_prec = bwd_ok ? std::max(Qf, Qb) : Qf;
    plan->prec = precision == GPD_PREC_AUTO ? (q_for_prec <= 9 ? GPD_PREC_FP32 : GPD_PREC_FP64) : precision;
    plan->elem_size = plan->prec == GPD_PREC_FP32 ? 4 : 8;
    plan->tau_col = plan->prec == GPD_PREC_FP32 ? kTauColFp32 : kTauColFp64;
    plan->tau_in = plan->prec == GPD_PREC_FP32 ? kTauInFp32 : kTauInFp64;
    plan->train = plan->prec == GPD_PREC_FP64_SLICED_TRAIN;
    plan->sliced = plan->prec == GPD_PREC_FP64_SLICED || plan->prec == GPD_PREC_FP64_SLICED40 || plan->train;
    plan->slices = plan->prec == GPD_PREC_FP64_SLICED40 ? 5 : plan->sliced ? 6 : 0;

    // powers up to the largest exponent used by any encoding
    const int max_exp = (int)std::max<int64_t>(std::max(Qf, Qb), Qw) + 1;
    const std::vector<double> pw = power_table(plan->points, max_exp);
    auto at = [&](int p, int e) { return pw[(size_t)p * max_exp + e]; };
    plan->coefW.resize((size_t)P * m * n);
    plan->coefX.resize((size_t)P * n * d1);
    plan->coefDT.resize((size_t)P * d2 * m);
    plan->coefDup.resize((size_t)P * m);
    plan->coefXup.resize((size_t)P * n);
    for (int p = 0; p < P; ++p) {
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < n; ++j)
                plan->coefW[((size_t)p * m + i) * n + j] = at(p, alt ? i + m * j : n * i + j);
        for (int j = 0; j < n; ++j)
            for (int k = 0; k < d1; ++k)
                plan->coefX[((size_t)p * n + j) * d1 + k] =
                    at(p, alt ? m * (n - 1 - j) + m * n * k : (n - 1 - j) + m * n * k);
        for (int k = 0; k < d2; ++k)
            for (int i = 0; i < m; ++i)
                plan->coefDT[((size_t)p * d2 + k) * m + i] =
                    at(p, alt ? m * n * k + (m - 1 - i) : m * n * k + n * (m - 1 - i));
        for (int i = 0; i < m; ++i) plan->coefDup[(size_t)p * m + i] = at(p, alt ? i : n * i);
        for (int j = 0; j < n; ++j) plan->coefXup[(size_t)p * n + j] = at(p, alt ? m * j : j);
    }
    // products
    ProductInfo& f = plan->prod[GPD_FWD];
    f.Q = (int)Qf; f.R = P - f.Q; f.grid_rows = m; f.grid_cols = d1;
    f.br = shape->N1 / m; f.bc = shape->B / d1;
    for (int i = 0; i < m; ++i)
        for (int k = 0; k < d1; ++k)
            f.wanted[i * d1 + k] = alt ? i + m * (n - 1) + m * n * k : n * i + m * n * k + n - 1;
    f.H = left_null_space(plan->points, f.Q);
    f.Hg = power_sum_parity(plan->points, f.R);
    ProductInfo& b = plan->prod[GPD_BWD];
    if (bwd_ok) {
        b.Q = (int)Qb; b.R = P - b.Q; b.grid_rows = d2; b.grid_cols = n;
        b.br = shape->B / d2; b.bc = shape->N0 / n;
        for (int k = 0; k < d2; ++k)
            for (int j = 0; j < n; ++j)
                b.wanted[k * n + j] = alt ? m * n * k + (m - 1) + m * j : m * n * k + n * (m - 1) + j;
        b.H = left_null_space(plan->points, b.Q);
        b.Hg = power_sum_parity(plan->points, b.R);
    }
    ProductInfo& a = plan->prod[GPD_AUDIT];
    if (audit_ok) {
        a.Q = (int)Qw; a.R = P - a.Q; a.grid_rows = m; a.grid_cols = n;
        a.br = shape->N1 / m; a.bc = shape->N0 / n;
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < n; ++j) a.wanted[i * n + j] = alt ? i + m * j : n * i + j;
        a.H = left_null_space(plan->points, a.Q);
        a.Hg = power_sum_parity(plan->points, a.R);
    }
    if (plan->sliced && !sliced_supported(plan)) { delete plan; return GPD_ERR_UNSUPPORTED; }
    *out = plan;
    return GPD_OK;
}

extern "C" gpd_status gpd_plan_upload(gpd_plan_t plan) {
    if (!plan) return GPD_ERR_ARG;
    return ensure_device(plan);
}

extern "C" gpd_status gpd_plan_destroy(gpd_plan_t plan) {
    if (!plan) return GPD_ERR_ARG;
    if (plan->uploaded && plan->dev.base) cudaFree(plan->dev.base);
    delete plan;
    return GPD_OK;
}

extern "C" gpd_status gpd_plan_query(gpd_plan_t plan, gpd_query what, int64_t* value) {
    if (!plan || !value) return GPD_ERR_ARG;
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int64_t P = plan->P;
    switch (what) {
        case GPD_Q_THRESHOLD_FWD: *value = plan->prod[GPD_FWD].Q; break;
        case GPD_Q_THRESHOLD_BWD: *value = plan->Qb; break;
        case GPD_Q_THRESHOLD_AUDIT: *value = plan->Qw; break;
        case GPD_Q_ELEMENT_SIZE: *value = plan->elem_size; break;
        case GPD_Q_W_SHARE_ELEMS:
            *value = plan->train ? (train_layout(plan).total_bytes + 7) / 8 : P * (s.N1 / c.m) * (s.N0 / c.n);
            break;
        case GPD_Q_X_SHARE_ELEMS: *value = P * (s.N0 / c.n) * (s.B / c.d1); break;
        case GPD_Q_DT_SHARE_ELEMS: *value = P * (s.B / c.d2) * (s.N1 / c.m); break;
        case GPD_Q_DHAT_ELEMS: *value = P * (s.N1 / c.m) * s.B; break;
        case GPD_Q_XHAT_ELEMS: *value = P * (s.N0 / c.n) * s.B; break;
        case GPD_Q_OUT_ELEMS_FWD: *value = P * (s.N1 / c.m) * (s.B / c.d1); break;
        case GPD_Q_OUT_ELEMS_BWD: *value = P * (s.B / c.d2) * (s.N0 / c.n); break;
        case GPD_Q_WORKSPACE_BYTES: *value = workspace_layout().total; break;
        case GPD_Q_STEP_WORKSPACE_BYTES: {
            // locate/decode scratch + the larger of {X~ + S~} and {Delta~^T + C~^T} and {Delta^ + X^}
            const int64_t e = plan->elem_size;
            const int64_t fwd = P * (s.N0 / c.n) * (s.B / c.d1) + P * (s.N1 / c.m) * (s.B / c.d1);
            const int64_t bwd = P * (s.B / c.d2) * (s.N1 / c.m) + P * (s.B / c.d2) * (s.N0 / c.n);
            const int64_t upd = P * (s.N1 / c.m) * s.B + P * (s.N0 / c.n) * s.B;
            const int64_t big = std::max(fwd, std::max(bwd, upd));
            *value = workspace_layout().total + ((big * e + 255) / 256 + 2) * 256;
            break;
        }
        case GPD_Q_POSITION_WORKSPACE_BYTES: *value = position_workspace_bytes(plan); break;
        case GPD_Q_PRECISION: *value = plan->prec; break;
        case GPD_Q_NODES: *value = P; break;
        case GPD_Q_TABLES_ON_DEVICE: {
            std::lock_guard<std::mutex> lock(plan->mu);
            *value = plan->uploaded ? 1 : 0;
            break;
        }
        default: return GPD_ERR_ARG;
    }
    return GPD_OK;
}

extern "C" gpd_status gpd_plan_table(gpd_plan_t plan, gpd_table which, double* host_out,
                                     int64_t capacity, int64_t* count) {
    if (!plan || !count) return GPD_ERR_ARG;
    const std::vector<double>* src = nullptr;
    switch (which) {
        case GPD_TABLE_POINTS: src = &plan->points; break;
        case GPD_TABLE_PARITY_FWD: src = &plan->prod[GPD_FWD].H; break;
        case GPD_TABLE_PARITY_BWD: src = &plan->prod[GPD_BWD].H; break;
        case GPD_TABLE_PARITY_AUDIT: src = &plan->prod[GPD_AUDIT].H; break;
        case GPD_TABLE_COEF_W: src = &plan->coefW; break;
        case GPD_TABLE_COEF_X: src = &plan->coefX; break;
        case GPD_TABLE_COEF_DT: src = &plan->coefDT; break;
        default: return GPD_ERR_ARG;
    }
    *count = (int64_t)src->size();
    if (host_out) {
        if (capacity < *count) return GPD_ERR_ARG;
        std::memcpy(host_out, src->data(), sizeof(double) * src->size());
    }
    return GPD_OK;
}
