// Locality loss, forward value (Sec. 3.2.2, second loss equation): L_loc = mu * KL(D_c || D_l).
// Reading (the paper writes no symbols for the two distributions): joint distributions over (source group,
// expert) pairs; D_c = the batch's demand counts, D_l = the same sources with every token on an expert the
// group hosts, mixed with a uniform floor `smooth` so that the divergence stays finite.  See locmoe.h.
// Integer sums are exact; floating-point sums run in a fixed order (strided per thread, then a tree), so the
// value is deterministic.
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kLocThreads = 256;

__device__ double block_sum(double v, double* sh) {
    sh[threadIdx.x] = v;
    __syncthreads();
    for (int o = kLocThreads / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}

// One CTA per group s: c_s(e), n_s and KL_s.
__global__ void __launch_bounds__(kLocThreads) loc_group_kernel(const int32_t* __restrict__ counts, int E, int per, int Eg,
                                                                double smooth, float* __restrict__ dc,
                                                                double* __restrict__ kl, long long* __restrict__ group_tokens) {
    __shared__ double sh[kLocThreads];
    __shared__ long long shn[kLocThreads];
    const int s = blockIdx.x;
    long long mine = 0;
    for (int e = threadIdx.x; e < E; e += kLocThreads)
        for (int m = 0; m < per; ++m) mine += counts[(size_t)(s * per + m) * E + e];
    shn[threadIdx.x] = mine;
    __syncthreads();
    for (int o = kLocThreads / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) shn[threadIdx.x] += shn[threadIdx.x + o];
        __syncthreads();
    }
    const long long ns = shn[0];
    double k = 0.0;
    for (int e = threadIdx.x; e < E; e += kLocThreads) {
        long long c = 0;
        for (int m = 0; m < per; ++m) c += counts[(size_t)(s * per + m) * E + e];
        const double cs = ns > 0 ? (double)c / (double)ns : 0.0;
        const double q = (e / Eg == s ? (1.0 - smooth) / (double)Eg : 0.0) + smooth / (double)E;
        dc[(size_t)s * E + e] = (float)cs;
        if (c > 0) k += cs * log(cs / q);
    }
    k = block_sum(k, sh);
    if (threadIdx.x == 0) { kl[s] = k; group_tokens[s] = ns; }
}

__global__ void __launch_bounds__(kLocThreads) loc_final_kernel(const double* __restrict__ kl,
                                                                const long long* __restrict__ group_tokens, int G, double mu,
                                                                double* __restrict__ loss) {
    __shared__ double sh[kLocThreads];
    double tot = 0.0;
    for (int s = threadIdx.x; s < G; s += kLocThreads) tot += (double)group_tokens[s];   // exact below 2^53
    tot = block_sum(tot, sh);
    double acc = 0.0;
    if (tot > 0.0)
        for (int s = threadIdx.x; s < G; s += kLocThreads) acc += (double)group_tokens[s] / tot * kl[s];
    acc = block_sum(acc, sh);
    if (threadIdx.x == 0) *loss = mu * acc;
}

}  // namespace

int launch_loc_loss(const locmoe_shape_t& s, const int32_t* counts, int level, double mu, double smooth, float* dc,
                    double* kl, long long* group_tokens, double* loss, cudaStream_t st) {
    const int D = s.n_nodes * s.dev_per_node;
    const int G = level ? s.n_nodes : D;
    loc_group_kernel<<<G, kLocThreads, 0, st>>>(counts, s.E, D / G, s.E / G, smooth, dc, kl, group_tokens);
    int rc = check_launch();
    if (rc) return rc;
    loc_final_kernel<<<1, kLocThreads, 0, st>>>(kl, group_tokens, G, mu, loss);
    return check_launch();
}

}  // namespace locmoe
