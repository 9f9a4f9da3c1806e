// Device code shared by the capacity kernels and by the route stage when it carries the capacity along:
// the order-preserving code of a cosine, and the finish that turns per-expert minima into the capacity record
// (Lemma 3, Theorem 1, the integer rule of Sec. 3.2.3).
#pragma once

#include <math.h>

#include "common.cuh"

namespace locmoe {

// Monotone map float -> uint32 (larger float, larger code).
__device__ __forceinline__ uint32_t order_code(float f) {
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_decode(uint32_t c) {
    return __uint_as_float((c & 0x80000000u) ? (c & 0x7fffffffu) : ~c);
}

// Continued fraction of the regularised incomplete beta function, valid for x < (a + 1) / (a + b + 2):
//   I_x(a, b) = x^a (1 - x)^b / (a B(a, b)) * h,   h = 1 / (1 + d_1 / (1 + d_2 / (1 + ...)))
// with the classical even/odd coefficients d_n.  Returns h, evaluated by the forward three-term recurrence of
// the convergents A_n / B_n, four coefficients per trip: their divisions do not depend on one another, and the
// only division on the dependent chain is the renormalisation (B_n = 1) once per trip, which also yields the
// convergent for the stopping test.
__device__ inline double beta_cf_h(double a, double b, double x) {
    const double eps = 1e-15;
    double Ap = 0.0, Bp = 1.0, A = 1.0, B = 1.0;   // convergents n = 0 and n = 1
    double h = 1.0;
    for (int m0 = 0; m0 < 40000; m0 += 2) {
        double c[4];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const double m = (double)(m0 + q), e = m + 1.0;
            c[2 * q] = -(a + m) * (a + b + m) * x / ((a + 2.0 * m) * (a + 2.0 * m + 1.0));     // d_{2m+1}
            c[2 * q + 1] = e * (b - e) * x / ((a + 2.0 * e - 1.0) * (a + 2.0 * e));            // d_{2m+2}
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const double An = A + c[k] * Ap, Bn = B + c[k] * Bp;
            Ap = A; Bp = B; A = An; B = Bn;
        }
        const double inv = 1.0 / B;
        A *= inv; Ap *= inv; Bp *= inv; B = 1.0;
        const bool done = fabs(A - h) <= eps * fabs(A);
        h = A;
        if (done) break;
    }
    return h;
}

// The same h by its power series, for one whole warp (all 32 lanes call it, all get the result):
//   h = 2F1(a + b, 1; a + 1; x) = sum_n t_n,  t_0 = 1,  t_(n+1) = t_n (a + b + n) x / (a + 1 + n),
// 64 terms: every lane forms two of the ratios (their divisions run side by side instead of one after the other
// as in the continued fraction), a shuffle scan multiplies them up, a shuffle sum adds the terms.  All terms are
// positive (no cancellation).  For x (a + b) < 5 the 64th term is below 1e-40 of the sum.
__device__ inline double beta_series_h_warp(double a, double b, double x) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const double n0 = (double)lane, n1 = (double)(lane + 32);
    double p0 = (a + b + n0) * x / (a + 1.0 + n0);     // ratio t_(lane+1) / t_lane
    double p1 = (a + b + n1) * x / (a + 1.0 + n1);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {                 // inclusive prefix products over the lanes
        const double u0 = __shfl_up_sync(full, p0, o), u1 = __shfl_up_sync(full, p1, o);
        if (lane >= o) { p0 *= u0; p1 *= u1; }
    }
    p1 *= __shfl_sync(full, p0, 31);                   // p0 = t_(lane+1), p1 = t_(lane+33)
    double s = p0 + p1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(full, s, o);
    return 1.0 + s;
}

// Scratch of the finish in shared memory.
struct FinishShared {
    float min[32];
    int empty[32];
    double part[4];    // h of the continued fraction, ln delta^2, ln(1 - delta^2), Theorem 1's erfc / exp form
};

// Decodes the per-expert minima (nsets partial arrays of E codes each, combined by min), writes delta_e /
// theta_e, and evaluates the closed forms and the integer rule.  Lemma 3:
//   p_delta = 1 - I_{delta^2}(1/2, (d-1)/2) = I_{1-delta^2}((d-1)/2, 1/2),
// on whichever side the continued fraction converges, never as a difference of nearly equal numbers when
// p_delta is small.  The independent pieces (continued fraction, the two logarithms, Theorem 1's other forms)
// run on four different warps at once; thread 0 puts them together.  lnbeta = ln B(1/2, (d-1)/2) does not depend on
// the data and comes from the host (ln_beta_half()).  One CTA of 128 to 1024 threads, a multiple of 32.
template <bool GLOBAL_SRC = true>
__device__ void capacity_finish(FinishShared& fs, const uint32_t* gmin, int nsets, int T, int E, int H,
                                int D, double lnbeta, const locmoe_capacity_rule_t& rule, float* __restrict__ delta_e,
                                float* __restrict__ theta_e, locmoe_capacity_t* __restrict__ cap) {
    float lmin = INFINITY;
    int lempty = 0;
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        uint32_t c = 0xffffffffu;
        for (int k = 0; k < nsets; ++k) c = min(c, GLOBAL_SRC ? __ldcg(gmin + (size_t)k * E + e) : gmin[(size_t)k * E + e]);
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
    if ((threadIdx.x & 31) == 0) { fs.min[threadIdx.x >> 5] = lmin; fs.empty[threadIdx.x >> 5] = lempty; }
    __syncthreads();
    const int role = (threadIdx.x & 31) == 0 ? (int)(threadIdx.x >> 5) : -1;   // lane 0 of warps 0..3 work on

    const int nwarps = (blockDim.x + 31) >> 5;
    lmin = fs.min[0]; lempty = fs.empty[0];
    for (int w = 1; w < nwarps; ++w) { lmin = fminf(lmin, fs.min[w]); lempty += fs.empty[w]; }
    int flags = 0;
    double delta = (double)lmin;
    delta = delta < 0.0 ? 0.0 : (delta > 1.0 ? 1.0 : delta);
    if (rule.delta_override >= 0.0) {
        delta = rule.delta_override > 1.0 ? 1.0 : rule.delta_override;
        flags |= LOCMOE_FLAG_DELTA_OVERRIDE;
    }
    const double bb = 0.5 * (double)(H - 1);
    const double x = delta * delta, y = 1.0 - x;
    const bool interior = delta > 0.0 && delta < 1.0;
    // small delta^2 d (every benchmark configuration, and the paper's delta = 0.03): the power series of I_x(1/2, bb)
    // on warp 0, about a microsecond; p_delta is then at least 1e-3, so forming it as 1 - I loses nothing.
    // Otherwise the continued fraction on one thread, on whichever side it converges.
    const bool series = interior && x * (bb + 0.5) < 5.0;
    const bool upper = !series && y < (bb + 1.0) / (bb + 2.5);   // the fraction converges for I_y(bb, 1/2)
    const double arg = x * (double)H / (2.0 - x);
    if (series) {
        if (threadIdx.x < 32) {
            const double h = beta_series_h_warp(0.5, bb, x);
            if (threadIdx.x == 0) fs.part[0] = h;
        }
    } else if (role == 0) {
        fs.part[0] = interior ? (upper ? beta_cf_h(bb, 0.5, y) : beta_cf_h(0.5, bb, x)) : 0.0;
    }
    if (role == 1) fs.part[1] = interior ? 2.0 * log(delta) : 0.0;
    if (role == 2) fs.part[2] = interior ? log1p(-x) : 0.0;
    if (role == 3) fs.part[3] = rule.bound_form == LOCMOE_BOUND_ERFC ? erfc(sqrt(arg))
                              : (rule.bound_form == LOCMOE_BOUND_EXP ? exp(arg) : 0.0);
    __syncthreads();
    if (role != 0) return;

    // the batch the rule counts: the caller's whole batch when this call sees one rank's share of it
    const double n = (double)E, dT = (double)(rule.T_global > 0 ? rule.T_global : T), dD = (double)D;
    double p;
    if (delta <= 0.0) p = 1.0;
    else if (delta >= 1.0) p = 0.0;
    else {
        const double lnx = fs.part[1], lny = fs.part[2], h = fs.part[0];
        p = upper ? exp(bb * lny + 0.5 * lnx - lnbeta) * h / bb
                  : 1.0 - exp(0.5 * lnx + bb * lny - lnbeta) * h / 0.5;
    }
    double ec;
    if (rule.bound_form == LOCMOE_BOUND_ERFC) ec = 1.0 / (n * fs.part[3]);
    else if (rule.bound_form == LOCMOE_BOUND_EXP) ec = fs.part[3] / n;
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

// ln B(1/2, (d-1)/2) = ln Gamma(1/2) + ln Gamma((d-1)/2) - ln Gamma(d/2), on the host.
double ln_beta_half(int d);

}  // namespace locmoe
