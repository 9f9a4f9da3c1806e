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

// Continued fraction of the regularised incomplete beta function, valid for x < (a + 1) / (a + b + 2):
//   I_x(a, b) = x^a (1 - x)^b / (a B(a, b)) * h,   h = 1 / (1 + d_1 / (1 + d_2 / (1 + ...)))
// with the classical even/odd coefficients d_n.  Returns h, evaluated by the forward three-term recurrence of
// the convergents A_n / B_n, four coefficients per trip: their divisions do not depend on one another, and the
// only division on the dependent chain is the renormalisation (B_n = 1) once per trip, which also yields the
// convergent for the stopping test.
__device__ double beta_cf_h(double a, double b, double x) {
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

// Scratch of the finish in shared memory.  lg[] does not depend on the data and is filled by finish_begin().
struct FinishShared {
    float min[32];
    int empty[32];
    double lg[2];      // ln Gamma((d-1)/2), ln Gamma(d/2)
    double part[4];    // h of the continued fraction, ln delta^2, ln(1 - delta^2), Theorem 1's erfc / exp form
};

// The last two warps of the CTA carry the data-independent log-gamma evaluations.
__device__ __forceinline__ void finish_begin(FinishShared& fs, int H) {
    const int first = (blockDim.x >> 5) - 2;
    const double bb = 0.5 * (double)(H - 1);
    if (threadIdx.x == first * 32) fs.lg[0] = lgamma(bb);
    if (threadIdx.x == (first + 1) * 32) fs.lg[1] = lgamma(bb + 0.5);
}

// Decodes the per-expert minima (nsets partial arrays of E codes each, combined by min), writes delta_e /
// theta_e, and evaluates the closed forms and the integer rule.  Lemma 3:
//   p_delta = 1 - I_{delta^2}(1/2, (d-1)/2) = I_{1-delta^2}((d-1)/2, 1/2),
// on whichever side the continued fraction converges, never as a difference of nearly equal numbers when
// p_delta is small.  The independent pieces (continued fraction, the two logarithms, Theorem 1's other forms)
// run on four different warps at once; thread 0 puts them together.  One CTA of 128 to 1024 threads, a multiple
// of 32, that has called finish_begin() before.
__device__ void capacity_finish(FinishShared& fs, const uint32_t* __restrict__ gmin, int nsets, int T, int E, int H,
                                int D, const locmoe_capacity_rule_t& rule, float* __restrict__ delta_e,
                                float* __restrict__ theta_e, locmoe_capacity_t* __restrict__ cap) {
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
    const bool upper = y < (bb + 1.0) / (bb + 2.5);   // the fraction converges for I_y(bb, 1/2)
    const double arg = x * (double)H / (2.0 - x);
    if (role == 0) fs.part[0] = interior ? (upper ? beta_cf_h(bb, 0.5, y) : beta_cf_h(0.5, bb, x)) : 0.0;
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
        const double lnbeta = 0.57236494292470008707 + fs.lg[0] - fs.lg[1];   // ln Gamma(1/2) = ln(pi) / 2
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

__global__ void __launch_bounds__(256) capacity_finish_kernel(const uint32_t* __restrict__ gmin, int T, int E, int H,
                                                              int D, locmoe_capacity_rule_t rule,
                                                              float* __restrict__ delta_e, float* __restrict__ theta_e,
                                                              locmoe_capacity_t* __restrict__ cap) {
    __shared__ FinishShared fs;
    finish_begin(fs, H);
    capacity_finish(fs, gmin, 1, T, E, H, D, rule, delta_e, theta_e, cap);
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
    __shared__ FinishShared fs;
    cg::cluster_group cluster = cg::this_cluster();
    const int cta = (int)cluster.block_rank();
    for (int e = threadIdx.x; e < E; e += blockDim.x) smin[e] = 0xffffffffu;
    __syncthreads();
    // CTA 0's last two warps evaluate the log-gammas instead of reading tokens; the other threads share the tokens
    constexpr int kMath = 64, kWorkers = kCapCS * kCapThreads - kMath;
    const bool math = cta == 0 && threadIdx.x >= kCapThreads - kMath;
    if (math) {
        finish_begin(fs, H);
    } else {
        const int wid = cta == 0 ? (int)threadIdx.x : cta * kCapThreads - kMath + (int)threadIdx.x;
        constexpr int kU = 8;   // tokens in flight per thread
        for (int t0 = wid; t0 < T; t0 += kU * kWorkers) {
            int e[kU];
            float c[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int t = t0 + u * kWorkers;
                e[u] = -1; c[u] = 0.0f;
                if (t < T) { e[u] = idx[t]; c[u] = cs[t]; }
            }
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (e[u] >= 0 && e[u] < E) atomicMin(&smin[e[u]], order_code(c[u]));
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) part[(size_t)cta * E + e] = smin[e];
    cluster.sync();
    if (cta == 0) capacity_finish(fs, part, kCapCS, T, E, H, D, rule, delta_e, theta_e, cap);
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
