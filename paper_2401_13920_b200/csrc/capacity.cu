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

#include "capacity_finish.cuh"
#include "common.cuh"

namespace cg = cooperative_groups;

namespace locmoe {

namespace {

constexpr int kSmemExperts = 8192;

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

__global__ void __launch_bounds__(256) capacity_finish_kernel(const uint32_t* __restrict__ gmin, int T, int E, int H,
                                                              int D, double lnbeta, locmoe_capacity_rule_t rule,
                                                              float* __restrict__ delta_e, float* __restrict__ theta_e,
                                                              locmoe_capacity_t* __restrict__ cap) {
    __shared__ FinishShared fs;
    capacity_finish(fs, gmin, 1, T, E, H, D, lnbeta, rule, delta_e, theta_e, cap);
}

// Whole stage in one kernel on one cluster: every CTA reduces its share of the tokens into per-expert minima in
// shared memory and stores them (plain stores, no initialisation needed) as its own row of the scratch; after the
// hardware cluster barrier CTA 0 combines the rows and finishes.
constexpr int kCapCS = 8;
constexpr int kCapThreads = 1024;

__global__ void __cluster_dims__(kCapCS, 1, 1) __launch_bounds__(kCapThreads, 1)
capacity_cluster_kernel(const int32_t* __restrict__ idx, const float* __restrict__ cs, uint32_t* __restrict__ part,
                        int T, int E, int H, int D, double lnbeta, locmoe_capacity_rule_t rule, float* __restrict__ delta_e,
                        float* __restrict__ theta_e, locmoe_capacity_t* __restrict__ cap) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ uint32_t smin[];
    __shared__ FinishShared fs;
    cg::cluster_group cluster = cg::this_cluster();
    const int cta = (int)cluster.block_rank();
    for (int e = threadIdx.x; e < E; e += blockDim.x) smin[e] = 0xffffffffu;
    __syncthreads();
    constexpr int kU = 8;   // tokens in flight per thread
    for (int t0 = cta * kCapThreads + threadIdx.x; t0 < T; t0 += kU * kCapCS * kCapThreads) {
        int e[kU];
        float c[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int t = t0 + u * kCapCS * kCapThreads;
            e[u] = -1; c[u] = 0.0f;
            if (t < T) { e[u] = idx[t]; c[u] = cs[t]; }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u)
            if (e[u] >= 0 && e[u] < E) atomicMin(&smin[e[u]], order_code(c[u]));
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) part[(size_t)cta * E + e] = smin[e];
    cluster.sync();
    if (cta == 0) capacity_finish(fs, part, kCapCS, T, E, H, D, lnbeta, rule, delta_e, theta_e, cap);
}

}  // namespace

double ln_beta_half(int d) {
    int sign = 0;
    const double b = 0.5 * (double)(d - 1);
    return 0.57236494292470008707 /* ln Gamma(1/2) = ln(pi) / 2 */ + lgamma_r(b, &sign) - lgamma_r(b + 0.5, &sign);
}

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
                          s.T, s.E, s.H, s.n_nodes * s.dev_per_node, ln_beta_half(s.H), rule, delta_e, theta_e, cap_dev);
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
    capacity_finish_kernel<<<1, 256, 0, st>>>(gmin, s.T, s.E, s.H, s.n_nodes * s.dev_per_node, ln_beta_half(s.H), rule, delta_e,
                                               theta_e, cap_dev);
    return check_launch();
}

}  // namespace locmoe
