// Angular deviation per expert and the capacity rule (abstract; Lemma 3; Theorem 1; Sec. 3.2.3).
//
// Per-expert minimum of the token cosines (integer min on an order-preserving
// encoding, so the result does not depend on scheduling), then a finish that
// decodes the minima and evaluates the closed forms in fp64 on one thread.
// Batches up to 262144 tokens run as ONE kernel on one thread-block cluster (hardware
// cluster barrier between the two steps); large ones as memset + grid-wide
// minimum + single-CTA finish.  Nothing is read back by the host.
#include <math.h>
#include <stdlib.h>

#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace locmoe {

namespace {

constexpr int kSmemExperts = 8192;

// Monotone map float -> uint32 (larger float, larger code).
__device__ __forceinline__ uint32_t order_code(float f) {
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_decode(uint32_t c) {
    return __uint_as_float((c & 0x80000000u) ? (c & 0x7fffffffu) : ~c);
}

__global__ void __launch_bounds__(256) mincos_kernel(const int32_t* __restrict__ idx, const float* __restrict__ cs,
                                                     int T, int E, uint32_t* __restrict__ gmin, int use_smem) {
    extern __shared__ uint32_t smin[];
    if (use_smem) {
        for (int e = threadIdx.x; e < E; e += blockDim.x) smin[e] = 0xffffffffu;
        __syncthreads();
    }
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < T; t += gridDim.x * blockDim.x) {
        int e = idx[t];
        if (e < 0 || e >= E) continue;
        uint32_t c = order_code(cs[t]);
        if (use_smem) atomicMin(&smin[e], c);
        else atomicMin(&gmin[e], c);
    }
    if (use_smem) {
        __syncthreads();
        for (int e = threadIdx.x; e < E; e += blockDim.x)
            if (smin[e] != 0xffffffffu) atomicMin(&gmin[e], smin[e]);
    }
}

// Continued fraction of the regularised incomplete beta function (Lentz's
// method on the classical even/odd coefficient pair); valid for
// x < (a + 1) / (a + b + 2).  Returns I_x(a, b) given ln x and ln(1 - x).
__device__ double beta_cf(double a, double b, double x, double lnx, double ln1mx) {
    const double tiny = 1e-300, eps = 1e-15;
    double c = 1.0, d = 1.0 - (a + b) * x / (a + 1.0);
    if (fabs(d) < tiny) d = tiny;
    d = 1.0 / d;
    double h = d;
    for (int m = 1; m <= 20000; ++m) {
        double m2 = 2.0 * m;
        double num = m * (b - m) * x / ((a + m2 - 1.0) * (a + m2));
        d = 1.0 + num * d; if (fabs(d) < tiny) d = tiny;
        c = 1.0 + num / c; if (fabs(c) < tiny) c = tiny;
        d = 1.0 / d;
        h *= d * c;
        num = -(a + m) * (a + b + m) * x / ((a + m2) * (a + m2 + 1.0));
        d = 1.0 + num * d; if (fabs(d) < tiny) d = tiny;
        c = 1.0 + num / c; if (fabs(c) < tiny) c = tiny;
        d = 1.0 / d;
        double del = d * c;
        h *= del;
        if (fabs(del - 1.0) < eps) break;
    }
    double lnfront = a * lnx + b * ln1mx - (lgamma(a) + lgamma(b) - lgamma(a + b));
    return exp(lnfront) * h / a;
}

// Lemma 3: p_delta = 1 - I_{delta^2}(1/2, (d-1)/2) = I_{1-delta^2}((d-1)/2, 1/2),
// evaluated on whichever side the continued fraction converges, never as a
// difference of nearly equal numbers when p_delta is small.
__device__ double p_delta_device(double delta, int d) {
    if (delta <= 0.0) return 1.0;
    if (delta >= 1.0) return 0.0;
    const double b = 0.5 * (double)(d - 1);
    const double x = delta * delta, y = 1.0 - x;
    const double lnx = 2.0 * log(delta), lny = log1p(-x);
    if (y < (b + 1.0) / (b + 2.5)) return beta_cf(b, 0.5, y, lny, lnx);
    return 1.0 - beta_cf(0.5, b, x, lnx, lny);
}

// Decodes the per-expert minima (nsets partial arrays of E codes each, combined by min), writes delta_e /
// theta_e, and lets thread 0 evaluate the closed forms and the integer rule.  One CTA, any block size <= 1024.
__device__ void capacity_finish(const uint32_t* __restrict__ gmin, int nsets, int T, int E, int H, int D,
                                const locmoe_capacity_rule_t& rule, float* __restrict__ delta_e,
                                float* __restrict__ theta_e, locmoe_capacity_t* __restrict__ cap) {
    __shared__ float s_min[32];
    __shared__ int s_empty[32];
    float lmin = INFINITY;
    int lempty = 0;
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        uint32_t c = 0xffffffffu;
        for (int k = 0; k < nsets; ++k) c = min(c, __ldcg(gmin + (size_t)k * E + e));
        float de;
        if (c == 0xffffffffu) { de = 1.0f; ++lempty; }
        else { de = order_decode(c); lmin = fminf(lmin, de); }
        delta_e[e] = de;
        theta_e[e] = acosf(fminf(fmaxf(de, -1.0f), 1.0f));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lmin = fminf(lmin, __shfl_xor_sync(0xffffffffu, lmin, o));
        lempty += __shfl_xor_sync(0xffffffffu, lempty, o);
    }
    if ((threadIdx.x & 31) == 0) { s_min[threadIdx.x >> 5] = lmin; s_empty[threadIdx.x >> 5] = lempty; }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const int nwarps = (blockDim.x + 31) >> 5;
    for (int w = 1; w < nwarps; ++w) { lmin = fminf(lmin, s_min[w]); lempty += s_empty[w]; }

    int flags = 0;
    double delta = (double)lmin;
    delta = delta < 0.0 ? 0.0 : (delta > 1.0 ? 1.0 : delta);
    if (rule.delta_override >= 0.0) {
        delta = rule.delta_override > 1.0 ? 1.0 : rule.delta_override;
        flags |= LOCMOE_FLAG_DELTA_OVERRIDE;
    }
    const double n = (double)E, dT = (double)T, dD = (double)D;
    const double p = p_delta_device(delta, H);
    const double arg = delta * delta * (double)H / (2.0 - delta * delta);
    double ec;
    if (rule.bound_form == LOCMOE_BOUND_ERFC) ec = 1.0 / (n * erfc(sqrt(arg)));
    else if (rule.bound_form == LOCMOE_BOUND_EXP) ec = exp(arg) / n;
    else ec = 1.0 / (n * p);

    // integer rule: each product / quotient rounded once (no fused multiply-add)
    double m = __dmul_rn(rule.min_mult, ec);
    if (!(m < dT)) { m = dT; flags |= LOCMOE_FLAG_MIN_SATURATED; }
    if (m < 0.0) m = 0.0;
    const double Cmin = ceil(m);
    const double cfT = __dmul_rn(rule.capacity_factor, dT);
    const double conv_e = ceil(__ddiv_rn(cfT, n));
    const double conv_l = ceil(__ddiv_rn(cfT, __dmul_rn(dD, n)));
    const double min_l = ceil(__ddiv_rn(Cmin, dD));
    double ce = Cmin > conv_e ? Cmin : conv_e;
    double cl = min_l > conv_l ? min_l : conv_l;
    if (min_l > conv_l) flags |= LOCMOE_FLAG_MIN_BINDS;
    ce = ce < 1.0 ? 1.0 : (ce > dT ? dT : ce);
    cl = cl < 1.0 ? 1.0 : (cl > dT ? dT : cl);
    cap->delta = delta;
    cap->p_delta = p;
    cap->ec_min = ec;
    cap->C_expert = (int32_t)ce;
    cap->C_local = (int32_t)cl;
    cap->n_empty_experts = lempty;
    cap->flags = flags;
}

__global__ void __launch_bounds__(256) capacity_finish_kernel(const uint32_t* __restrict__ gmin, int T, int E, int H,
                                                              int D, locmoe_capacity_rule_t rule,
                                                              float* __restrict__ delta_e, float* __restrict__ theta_e,
                                                              locmoe_capacity_t* __restrict__ cap) {
    capacity_finish(gmin, 1, T, E, H, D, rule, delta_e, theta_e, cap);
}

// Whole stage in one kernel on one cluster: every CTA reduces its share of the tokens into per-expert minima in
// shared memory and stores them (plain stores, no initialisation needed) as its own row of the scratch; after the
// hardware cluster barrier CTA 0 combines the rows and finishes.
constexpr int kCapCS = 8;
constexpr int kCapThreads = 1024;

__global__ void __cluster_dims__(kCapCS, 1, 1) __launch_bounds__(kCapThreads, 1)
capacity_cluster_kernel(const int32_t* __restrict__ idx, const float* __restrict__ cs, uint32_t* __restrict__ part,
                        int T, int E, int H, int D, locmoe_capacity_rule_t rule, float* __restrict__ delta_e,
                        float* __restrict__ theta_e, locmoe_capacity_t* __restrict__ cap) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ uint32_t smin[];
    cg::cluster_group cluster = cg::this_cluster();
    const int cta = (int)cluster.block_rank();
    for (int e = threadIdx.x; e < E; e += blockDim.x) smin[e] = 0xffffffffu;
    __syncthreads();
    for (int t = cta * kCapThreads + threadIdx.x; t < T; t += kCapCS * kCapThreads) {
        const int e = idx[t];
        if (e >= 0 && e < E) atomicMin(&smin[e], order_code(cs[t]));
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) part[(size_t)cta * E + e] = smin[e];
    cluster.sync();
    if (cta == 0) capacity_finish(part, kCapCS, T, E, H, D, rule, delta_e, theta_e, cap);
}

}  // namespace

// One-cluster kernel when the per-expert minima fit in shared memory and the batch is moderate;
// LOCMOE_PATH=grid|cluster overrides the size rule (testing aid).
bool capacity_cluster_eligible(const locmoe_shape_t& s) {
    if (s.E > kSmemExperts) return false;
    const char* o = getenv("LOCMOE_PATH");
    if (o && o[0] == 'g') return false;
    if (o && o[0] == 'c') return true;
    return s.T <= (1 << 18);   // beyond that, eight CTAs take longer to read the tokens than two more launches cost
}

size_t capacity_ws_bytes(const locmoe_shape_t& s) { return ((size_t)kCapCS * s.E * sizeof(uint32_t) + 255) & ~(size_t)255; }

int launch_capacity(const locmoe_shape_t& s, const int32_t* idx, const float* cos_sim,
                    const locmoe_capacity_rule_t& rule, float* delta_e, float* theta_e,
                    locmoe_capacity_t* cap_dev, void* ws, cudaStream_t st) {
    uint32_t* gmin = static_cast<uint32_t*>(ws);
    if (capacity_cluster_eligible(s)) {
        return launch_pdl(capacity_cluster_kernel, kCapCS, kCapThreads, (size_t)s.E * sizeof(uint32_t), st, idx, cos_sim, gmin,
                          s.T, s.E, s.H, s.n_nodes * s.dev_per_node, rule, delta_e, theta_e, cap_dev);
    }
    if (cudaMemsetAsync(gmin, 0xff, (size_t)s.E * sizeof(uint32_t), st) != cudaSuccess) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    const int use_smem = s.E <= kSmemExperts;
    int blocks = (s.T + 256 * 8 - 1) / (256 * 8);
    if (blocks > 2 * sm_count()) blocks = 2 * sm_count();
    if (blocks < 1) blocks = 1;
    mincos_kernel<<<blocks, 256, use_smem ? (size_t)s.E * sizeof(uint32_t) : 0, st>>>(idx, cos_sim, s.T, s.E, gmin,
                                                                                  use_smem);
    int rc = check_launch();
    if (rc) return rc;
    capacity_finish_kernel<<<1, 256, 0, st>>>(gmin, s.T, s.E, s.H, s.n_nodes * s.dev_per_node, rule, delta_e, theta_e,
                                               cap_dev);
    return check_launch();
}

}  // namespace locmoe
