// coded_layer_step: one layer of the coded training iteration (Sections VI and VIII) composed
// from the stage launches on one stream.  Nothing here synchronises with the host; a decoding
// failure is carried on the device (the decode and update kernels test the result struct).
#include "gpd_internal.h"

namespace gpd {

namespace {
int64_t align256(int64_t x) { return (x + 255) / 256 * 256; }
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status coded_layer_step(gpd_plan_t plan, int32_t phases, void* W_shares_dev,
                                       const float* X_dev, const float* Delta_dev, const float* DeltaT_dev,
                                       gpd_activation_kind activation, float eta, float lambda,
                                       uint64_t inject_seed, double inject_prob, double inject_scale,
                                       float* S_out_dev, float* Xnext_out_dev, float* CT_out_dev,
                                       gpd_locate_result* results_dev, void* workspace_dev, void* stream) {
    if (!plan || !W_shares_dev || !results_dev) return GPD_ERR_ARG;
    if (!workspace_dev) return GPD_ERR_WORKSPACE;
    if ((phases & ~(GPD_PHASE_FWD | GPD_PHASE_BWD | GPD_PHASE_UPD | GPD_PHASE_REGEN | GPD_PHASE_INJECT_SHARES)) ||
        !(phases & (GPD_PHASE_FWD | GPD_PHASE_BWD | GPD_PHASE_UPD)))
        return GPD_ERR_ARG;
    if (plan->sliced && !plan->train && phases != GPD_PHASE_FWD) return GPD_ERR_UNSUPPORTED;   // forward-only digit-plane modes
    // every requested phase is checked before anything is enqueued
    if ((phases & GPD_PHASE_FWD) && (!X_dev || !S_out_dev)) return GPD_ERR_ARG;
    if ((phases & GPD_PHASE_BWD) && (!DeltaT_dev || !CT_out_dev)) return GPD_ERR_ARG;
    if ((phases & GPD_PHASE_UPD) && (!Delta_dev || !X_dev)) return GPD_ERR_ARG;
    if ((phases & GPD_PHASE_BWD) && plan->prod[GPD_BWD].Q == 0) return GPD_ERR_P_TOO_SMALL;   // forward-only plan
    if ((phases & GPD_PHASE_REGEN) && plan->prod[GPD_AUDIT].Q == 0) return GPD_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    const gpd_shape& s = plan->shape;
    const gpd_split& c = plan->split;
    const int64_t P = plan->P, e = plan->elem_size;
    char* ws = reinterpret_cast<char*>(workspace_dev);
    void* small = ws;                                          // locate / decode scratch
    char* big = ws + align256(workspace_layout().total);       // operand shares + worker outputs
    gpd_status rc;

    if (phases & GPD_PHASE_FWD) {
        if (!X_dev || !S_out_dev) return GPD_ERR_ARG;
        void* Xsh = big;
        void* Z = big + align256(P * (s.N0 / c.n) * (s.B / c.d1) * e);
        if ((rc = encode_launch(plan, GPD_OPERAND_X_FWD, X_dev, Xsh, st)) != GPD_OK) return rc;
        if ((rc = worker_gemm_launch(plan, GPD_FWD, W_shares_dev, Xsh, Z, st)) != GPD_OK) return rc;
        if (inject_prob > 0.0 &&
            (rc = inject_launch(plan, GPD_FWD, Z, inject_seed + 0, GPD_INJECT_GAUSS, inject_prob, 0, 0,
                                inject_scale, nullptr, st)) != GPD_OK)
            return rc;
        if ((rc = locate_launch(plan, GPD_FWD, Z, 0, &results_dev[0], small, st)) != GPD_OK) return rc;
        if ((rc = decode_launch(plan, GPD_FWD, Z, false, 0, &results_dev[0], S_out_dev, Xnext_out_dev,
                                (int)activation, small, st)) != GPD_OK)
            return rc;
        if ((phases & GPD_PHASE_REGEN) &&
            (rc = regenerate_launch(plan, W_shares_dev, &results_dev[0], small, st)) != GPD_OK)
            return rc;
    }
    if (phases & GPD_PHASE_BWD) {
        if (!DeltaT_dev || !CT_out_dev) return GPD_ERR_ARG;
        void* Dsh = big;
        void* Z = big + align256(P * (s.B / c.d2) * (s.N1 / c.m) * e);
        if ((rc = encode_launch(plan, GPD_OPERAND_DELTAT_BWD, DeltaT_dev, Dsh, st)) != GPD_OK) return rc;
        if ((rc = worker_gemm_launch(plan, GPD_BWD, W_shares_dev, Dsh, Z, st)) != GPD_OK) return rc;
        if (inject_prob > 0.0 &&
            (rc = inject_launch(plan, GPD_BWD, Z, inject_seed + 1, GPD_INJECT_GAUSS, inject_prob, 0, 0,
                                inject_scale, nullptr, st)) != GPD_OK)
            return rc;
        if ((rc = locate_launch(plan, GPD_BWD, Z, 0, &results_dev[1], small, st)) != GPD_OK) return rc;
        if ((rc = decode_launch(plan, GPD_BWD, Z, false, 0, &results_dev[1], CT_out_dev, nullptr,
                                GPD_ACT_IDENTITY, small, st)) != GPD_OK)
            return rc;
    }
    if (phases & GPD_PHASE_UPD) {
        if (!Delta_dev || !X_dev) return GPD_ERR_ARG;
        void* Dhat = big;
        void* Xhat = big + align256(P * (s.N1 / c.m) * s.B * e);
        if ((rc = encode_launch(plan, GPD_OPERAND_DELTA_UPD, Delta_dev, Dhat, st)) != GPD_OK) return rc;
        if ((rc = encode_launch(plan, GPD_OPERAND_X_UPD, X_dev, Xhat, st)) != GPD_OK) return rc;
        const gpd_locate_result* gate = (phases & GPD_PHASE_BWD) ? &results_dev[1] : nullptr;
        if ((rc = update_launch(plan, W_shares_dev, Dhat, Xhat, eta, lambda, gate, st)) != GPD_OK) return rc;
        if ((phases & GPD_PHASE_INJECT_SHARES) && inject_prob > 0.0 &&
            (rc = inject_launch(plan, GPD_AUDIT, W_shares_dev, inject_seed + 2, GPD_INJECT_GAUSS, inject_prob, 0, 0,
                                inject_scale, nullptr, st)) != GPD_OK)
            return rc;
    }
    return GPD_OK;
}
