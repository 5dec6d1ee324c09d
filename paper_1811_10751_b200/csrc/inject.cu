// Seeded soft-error injection into the worker-output buffer (Error Model 2 of Section V-B:
// the whole output of an erroneous node receives additive continuous noise; plus the single
// bit-flip and sparse-additive variants the workloads ask for).  Faults are values in buffers.
//
// Random draws: SplitMix64 (Steele, Lea, Flood 2014) used as a counter-based generator,
//   mix64(z) = output function applied to z + GAMMA;  draw(key, ctr) = mix64(key + ctr*GAMMA);
//   key(seed, tag, p) = mix64(mix64(seed ^ tag*TAGMUL) + p),
// so every entry's error is a pure function of (seed, node, entry).
#include <cmath>

#include "gpd_internal.h"
#include "slice_common.h"

namespace gpd {

namespace {

constexpr unsigned long long kGamma = 0x9E3779B97F4A7C15ULL;
constexpr unsigned long long kTagMul = 0xD6E8FEB86659FD93ULL;
enum { TAG_NODE = 1, TAG_PHI = 2, TAG_ENTRY = 3, TAG_MAG = 4, TAG_FIRST = 5, TAG_BITFLIP = 6, TAG_GAUSS = 7 };

__host__ __device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z += kGamma;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ unsigned long long draw(unsigned long long key, unsigned long long ctr) {
    return mix64(key + ctr * kGamma);
}
__host__ __device__ __forceinline__ unsigned long long make_key(unsigned long long seed, int tag,
                                                                unsigned long long p) {
    return mix64(mix64(seed ^ ((unsigned long long)tag * kTagMul)) + p);
}
__host__ __device__ __forceinline__ double unit(unsigned long long r) {
    return (double)(r >> 11) * (1.0 / 9007199254740992.0);   // 2^-53
}

struct InjectParams {
    int n_sel;             // additive / gauss: number of selected nodes, listed in sel[]
    unsigned char sel[kMaxNodes];
    void* out;             // [P][L]
    int64_t L;
    int P;
    int elem_size;
    unsigned long long seed;
    double prob;           // < 0: use node_mask
    unsigned long long node_mask;
    int count;
    double scale;
    unsigned long long* hit_mask;
};

__host__ __device__ __forceinline__ bool node_selected(const InjectParams& prm, int p) {
    if (prm.prob < 0.0) return (prm.node_mask >> p) & 1ULL;
    return unit(draw(make_key(prm.seed, TAG_NODE, 0), (unsigned long long)p)) < prm.prob;
}

__global__ void write_mask_kernel(unsigned long long* dst, unsigned long long value) { *dst = value; }

// Per-node constants of the additive mode, evaluated on the host with the same generator.
struct AdditiveNode {
    unsigned long long phi_cut;   // entry l is hit when (draw(k_entry, l) >> 11) < phi_cut, i.e. unit(draw) < phi
    unsigned long long first;     // the one entry that is always hit
    unsigned long long k_entry, k_mag;
};
struct AdditiveParams {
    AdditiveNode node[kMaxNodes];
    unsigned char sel[kMaxNodes];
    void* out;
    int64_t L;
    double scale;
};

inline AdditiveNode additive_node(unsigned long long seed, int p, int64_t L) {
    AdditiveNode a;
    const double phi = 1.0 - unit(draw(make_key(seed, TAG_PHI, 0), (unsigned long long)p));
    // unit(r) < phi  <=>  (r >> 11) < ceil(phi 2^53): integers below 2^53 on both sides
    a.phi_cut = (unsigned long long)std::ceil(phi * 9007199254740992.0);
    a.first = draw(make_key(seed, TAG_FIRST, 0), (unsigned long long)p) % (unsigned long long)L;
    a.k_entry = make_key(seed, TAG_ENTRY, (unsigned long long)p);
    a.k_mag = make_key(seed, TAG_MAG, (unsigned long long)p);
    return a;
}

template <typename T>
__global__ void __launch_bounds__(256) inject_additive_kernel(const __grid_constant__ AdditiveParams prm) {
    const AdditiveNode& nd = prm.node[blockIdx.y];
    T* out = reinterpret_cast<T*>(prm.out) + (int64_t)prm.sel[blockIdx.y] * prm.L;
    for (int64_t l = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; l < prm.L;
         l += (int64_t)gridDim.x * blockDim.x) {
        const bool hit = ((unsigned long long)l == nd.first) || ((draw(nd.k_entry, (unsigned long long)l) >> 11) < nd.phi_cut);
        if (!hit) continue;
        const unsigned long long r = draw(nd.k_mag, (unsigned long long)l);
        const int k = -4 + (int)((r >> 53) % 12ULL);
        // (1 + f) 2^k with f = the low 52 bits of r as a fraction: those bits are the mantissa, k the
        // exponent, bit 52 the sign
        const unsigned long long bits = (((r >> 52) & 1ULL) << 63) | ((unsigned long long)(1023 + k) << 52) |
                                        (r & ((1ULL << 52) - 1ULL));
        const double mag = __longlong_as_double((long long)bits) * prm.scale;
        out[l] = (T)((double)out[l] + mag);
    }
}

template <typename T>
__global__ void __launch_bounds__(256) inject_gauss_kernel(InjectParams prm) {
    const int p = prm.sel[blockIdx.y];
    const unsigned long long key = make_key(prm.seed, TAG_GAUSS, (unsigned long long)p);
    T* out = reinterpret_cast<T*>(prm.out) + (int64_t)p * prm.L;
    for (int64_t l = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; l < prm.L;
         l += (int64_t)gridDim.x * blockDim.x) {
        const double u1 = ((double)(draw(key, 2ULL * l) >> 11) + 1.0) * (1.0 / 9007199254740992.0);
        const double u2 = unit(draw(key, 2ULL * l + 1ULL));
        const double g = sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);   // Box-Muller
        out[l] = (T)((double)out[l] + prm.scale * g);
    }
}

// `count` distinct nodes, one entry each, one bit each; sequential by nature, one thread.
template <typename T, typename U>
__global__ void inject_bitflip_kernel(InjectParams prm) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const unsigned long long key = make_key(prm.seed, TAG_BITFLIP, 0);
    const int nbits = (int)sizeof(T) * 8;
    unsigned long long ctr = 0, hit = 0;
    int done = 0;
    const int want = prm.count < prm.P ? prm.count : prm.P;
    T* out = reinterpret_cast<T*>(prm.out);
    while (done < want) {
        const int p = (int)(draw(key, ctr++) % (unsigned long long)prm.P);
        if ((hit >> p) & 1ULL) continue;
        const int64_t l = (int64_t)(draw(key, ctr++) % (unsigned long long)prm.L);
        T* cell = out + (int64_t)p * prm.L + l;
        const T old = *cell;
        U word;
        memcpy(&word, &old, sizeof(T));
        T neu = old;
        for (int tries = 0; tries < 4096; ++tries) {
            const int b = (int)(draw(key, ctr++) % (unsigned long long)nbits);
            const U flipped = word ^ ((U)1 << b);
            memcpy(&neu, &flipped, sizeof(T));
            const double delta = fabs((double)neu - (double)old);
            if (!isfinite((double)neu) || delta >= 0.015625 * prm.scale) break;    // 2^-6 * scale
        }
        *cell = neu;
        hit |= 1ULL << p;
        ++done;
    }
    if (prm.hit_mask) *prm.hit_mask = hit;
}

}  // namespace

gpd_status inject_launch(gpd_plan_s* plan, gpd_product which, void* outputs, uint64_t seed, int mode,
                         double prob, uint64_t node_mask, int count, double scale, uint64_t* hit_mask,
                         cudaStream_t st) {
    if (which != GPD_FWD && which != GPD_BWD && which != GPD_AUDIT) return GPD_ERR_ARG;
    // digit-plane shares: forward product only, except in the training mode (its backward outputs and the
    // FP64 shares that lead W's buffer are plain doubles)
    if (plan->sliced && !plan->train && which != GPD_FWD) return GPD_ERR_UNSUPPORTED;
    const ProductInfo& pi = plan->prod[which];
    if (pi.Q == 0) return GPD_ERR_P_TOO_SMALL;
    InjectParams prm{};
    prm.out = outputs;
    prm.L = pi.br * pi.bc;
    prm.P = plan->P;
    prm.elem_size = plan->elem_size;
    prm.seed = seed;
    prm.prob = prob;
    prm.node_mask = node_mask;
    prm.count = count;
    prm.scale = scale;
    prm.hit_mask = reinterpret_cast<unsigned long long*>(hit_mask);
    const bool f32 = plan->elem_size == 4;
    // training mode, errors written into the stored shares: they land in the FP64 shares, from which the
    // sliced copies that the products read are then cut again
    const bool recut = plan->train && which == GPD_AUDIT;
    if (mode == GPD_INJECT_BITFLIP) {
        if (count < 0) return GPD_ERR_ARG;
        if (f32) inject_bitflip_kernel<float, unsigned int><<<1, 32, 0, st>>>(prm);
        else inject_bitflip_kernel<double, unsigned long long><<<1, 32, 0, st>>>(prm);
        if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
        return recut ? reslice_launch(plan, outputs, st) : GPD_OK;
    }
    if (mode != GPD_INJECT_ADDITIVE && mode != GPD_INJECT_GAUSS) return GPD_ERR_ARG;
    // Which nodes are hit is a pure function of (seed, node): evaluated here with the same
    // generator, so that only the selected nodes get thread blocks.
    unsigned long long mask = 0;
    for (int p = 0; p < prm.P; ++p)
        if (node_selected(prm, p)) { prm.sel[prm.n_sel++] = (unsigned char)p; mask |= 1ULL << p; }
    if (prm.hit_mask) {
        write_mask_kernel<<<1, 1, 0, st>>>(prm.hit_mask, mask);
        if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
    }
    if (prm.n_sel == 0) return GPD_OK;
    // one entry per thread up to 8192 CTAs per node: a single round trip to memory for most threads
    dim3 grid((unsigned)std::min<int64_t>((prm.L + 255) / 256, 8192), (unsigned)prm.n_sel);
    if (mode == GPD_INJECT_ADDITIVE) {
        AdditiveParams ap{};
        for (int i = 0; i < prm.n_sel; ++i) {
            ap.sel[i] = prm.sel[i];
            ap.node[i] = additive_node(prm.seed, prm.sel[i], prm.L);
        }
        ap.out = prm.out; ap.L = prm.L; ap.scale = prm.scale;
        if (f32) inject_additive_kernel<float><<<grid, 256, 0, st>>>(ap);
        else inject_additive_kernel<double><<<grid, 256, 0, st>>>(ap);
    } else if (mode == GPD_INJECT_GAUSS) {
        if (f32) inject_gauss_kernel<float><<<grid, 256, 0, st>>>(prm);
        else inject_gauss_kernel<double><<<grid, 256, 0, st>>>(prm);
    } else {
        return GPD_ERR_ARG;
    }
    if (launch_ok() != GPD_OK) return GPD_ERR_CUDA;
    return recut ? reslice_launch(plan, outputs, st) : GPD_OK;
}

}  // namespace gpd

using namespace gpd;

extern "C" gpd_status gpd_inject(gpd_plan_t plan, gpd_product which, void* outputs_dev, uint64_t seed,
                                 gpd_inject_mode mode, double prob, uint64_t node_mask, int32_t count,
                                 double scale, uint64_t* hit_mask_dev, void* stream) {
    if (!plan || !outputs_dev) return GPD_ERR_ARG;
    return inject_launch(plan, which, outputs_dev, seed, (int)mode, prob, node_mask, count, scale,
                         hit_mask_dev, as_stream(stream));
}
