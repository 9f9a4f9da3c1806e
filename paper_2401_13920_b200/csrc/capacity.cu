// Angular deviation per expert and the capacity rule (abstract; Lemma 3; Theorem 1; Sec. 3.2.3).
//
// Two small kernels after a memset of the scratch: a grid-wide per-expert minimum
// of the token cosines (integer atomicMin on an order-preserving encoding, so
// the result does not depend on scheduling), and a single-CTA finish that
// decodes the minima and evaluates the closed forms in fp64 on one thread.
// Nothing is read back by the host.
#include <math.h>

#include "common.cuh"

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

__global__ void __launch_bounds__(256) capacity_finish_kernel(const uint32_t* __restrict__ gmin, int T, int E, int H,
                                                              int D, locmoe_capacity_rule_t rule,
                                                              float* __restrict__ delta_e, float* __restrict__ theta_e,
                                                              locmoe_capacity_t* __restrict__ cap) {
    __shared__ float s_min[256];
    __shared__ int s_empty[256];
    float lmin = INFINITY;
    int lempty = 0;
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        uint32_t c = gmin[e];
        float de;
        if (c == 0xffffffffu) { de = 1.0f; ++lempty; }
        else { de = order_decode(c); lmin = fminf(lmin, de); }
        delta_e[e] = de;
        theta_e[e] = acosf(fminf(fmaxf(de, -1.0f), 1.0f));
    }
    s_min[threadIdx.x] = lmin;
    s_empty[threadIdx.x] = lempty;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) {
            s_min[threadIdx.x] = fminf(s_min[threadIdx.x], s_min[threadIdx.x + o]);
            s_empty[threadIdx.x] += s_empty[threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x != 0) return;

    int flags = 0;
    double delta = (double)s_min[0];
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
    cap->n_empty_experts = s_empty[0];
    cap->flags = flags;
}

}  // namespace

size_t capacity_ws_bytes(const locmoe_shape_t& s) { return ((size_t)s.E * sizeof(uint32_t) + 255) & ~(size_t)255; }

int launch_capacity(const locmoe_shape_t& s, const int32_t* idx, const float* cos_sim,
                    const locmoe_capacity_rule_t& rule, float* delta_e, float* theta_e,
                    locmoe_capacity_t* cap_dev, void* ws, cudaStream_t st) {
    uint32_t* gmin = static_cast<uint32_t*>(ws);
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
