// Cosine-frequency diagnostic (Sec. 4.1, second cosine-histogram figure): over the tokens routed to one expert,
// the histogram of their cosine to that expert's gating weight and the histogram of their cosine to another
// expert's gating weight.  cos(x, w_i) = (sum of the i-th group of x) / (sqrt(d/n) |x|).
// One warp per routed token (the other tokens cost one index load); integer atomics, so the counts do not depend
// on scheduling.  A diagnostic: rows are read with plain coalesced loads, 1/n of the batch.
#include "common.cuh"

namespace locmoe {

namespace {

__device__ __forceinline__ float elem(const void* p, long long i, int dt) {
    if (dt == LOCMOE_F32) return reinterpret_cast<const float*>(p)[i];
    return __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(p)[i]) << 16);
}

__device__ __forceinline__ int bin_of(float c, float lo, float scale, int nbins) {
    float pos = floorf((c - lo) * scale);
    pos = fminf(fmaxf(pos, 0.0f), (float)(nbins - 1));
    return (int)pos;
}

__global__ void __launch_bounds__(256) cos_hist_kernel(const void* __restrict__ x, int dt, const int32_t* __restrict__ idx,
                                                       int T, int H, int g, int e, int j, int nbins, float lo, float scale,
                                                       int32_t* __restrict__ hist_e, int32_t* __restrict__ hist_j,
                                                       int32_t* __restrict__ n_routed) {
    const int lane = threadIdx.x & 31;
    const int nw = gridDim.x * (blockDim.x >> 5);
    for (int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); t < T; t += nw) {
        if (idx[t] != e) continue;
        const long long base = (long long)t * H;
        float sq = 0.0f, se = 0.0f, sj = 0.0f;
        for (int k = lane; k < H; k += 32) {
            const float v = elem(x, base + k, dt);
            sq = fmaf(v, v, sq);
            const int grp = k / g;
            if (grp == e) se += v;
            if (grp == j) sj += v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sq += __shfl_xor_sync(0xffffffffu, sq, o);
            se += __shfl_xor_sync(0xffffffffu, se, o);
            sj += __shfl_xor_sync(0xffffffffu, sj, o);
        }
        if (lane == 0) {
            const float den = sqrtf((float)g) * sqrtf(sq);
            const float ce = den > 0.0f ? se / den : 0.0f, cj = den > 0.0f ? sj / den : 0.0f;
            atomicAdd(&hist_e[bin_of(ce, lo, scale, nbins)], 1);
            atomicAdd(&hist_j[bin_of(cj, lo, scale, nbins)], 1);
            atomicAdd(n_routed, 1);
        }
    }
}

}  // namespace

int launch_cos_hist(const locmoe_shape_t& s, const void* x, const int32_t* idx, int e, int j, int nbins, float lo, float hi,
                    int32_t* hist_e, int32_t* hist_j, int32_t* n_routed, cudaStream_t st) {
    if (cudaMemsetAsync(hist_e, 0, sizeof(int32_t) * nbins, st) != cudaSuccess ||
        cudaMemsetAsync(hist_j, 0, sizeof(int32_t) * nbins, st) != cudaSuccess ||
        cudaMemsetAsync(n_routed, 0, sizeof(int32_t), st) != cudaSuccess) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    int blocks = (s.T + 7) / 8;
    if (blocks > 16 * sm_count()) blocks = 16 * sm_count();
    cos_hist_kernel<<<blocks, 256, 0, st>>>(x, s.x_dtype, idx, s.T, s.H, s.H / s.E, e, j, nbins, lo,
                                           (float)nbins / (hi - lo), hist_e, hist_j, n_routed);
    return check_launch();
}

}  // namespace locmoe
