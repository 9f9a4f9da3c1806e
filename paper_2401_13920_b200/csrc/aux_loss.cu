// Auxiliary load-balance loss, forward value (Sec. 3.2.2, first loss equation):
//   L_aux = alpha * n * sum_i f_i * P_i,
//   f_i = (1/T) #{tokens whose arg-max is expert i},   P_i = (1/T) sum over tokens of p_i(x).
// f comes from the per-expert demand counts of the route stage; P needs the column sums of the gate's
// probability matrix.  The sums are formed in a fixed order (fixed row blocks, then the blocks in index order),
// so the result is deterministic: no floating-point atomics.
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kRowsPerBlock = 256;

// partial[b][i] = sum of probs[t][i] over the rows t of block b (threads stride over columns, rows in order).
__global__ void __launch_bounds__(256) aux_partial_kernel(const float* __restrict__ probs, int T, int E,
                                                          float* __restrict__ partial) {
    const int r0 = blockIdx.x * kRowsPerBlock;
    const int r1 = min(r0 + kRowsPerBlock, T);
    for (int i = threadIdx.x; i < E; i += blockDim.x) {
        float s = 0.0f;
        for (int t = r0; t < r1; ++t) s += probs[(size_t)t * E + i];
        partial[(size_t)blockIdx.x * E + i] = s;
    }
}

__global__ void __launch_bounds__(256) aux_final_kernel(const float* __restrict__ partial, int nblk,
                                                        const int32_t* __restrict__ load, int T, int E, float alpha,
                                                        float* __restrict__ f, float* __restrict__ P,
                                                        float* __restrict__ loss) {
    __shared__ double acc[256];
    double local = 0.0;
    for (int i = threadIdx.x; i < E; i += blockDim.x) {
        double s = 0.0;
        for (int b = 0; b < nblk; ++b) s += (double)partial[(size_t)b * E + i];
        const double Pi = s / (double)T, fi = (double)load[i] / (double)T;
        P[i] = (float)Pi;
        f[i] = (float)fi;
        local += fi * Pi;
    }
    acc[threadIdx.x] = local;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) acc[threadIdx.x] += acc[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = (float)((double)alpha * (double)E * acc[0]);
}

}  // namespace

size_t aux_ws_bytes(const locmoe_shape_t& s) {
    const size_t nblk = ((size_t)s.T + kRowsPerBlock - 1) / kRowsPerBlock;
    return (nblk * s.E * sizeof(float) + 255) & ~(size_t)255;
}

int launch_aux_loss(const locmoe_shape_t& s, const float* probs, const int32_t* load, float alpha, float* f, float* P,
                    float* loss, void* ws, cudaStream_t st) {
    const int nblk = (s.T + kRowsPerBlock - 1) / kRowsPerBlock;
    float* partial = static_cast<float*>(ws);
    aux_partial_kernel<<<nblk, 256, 0, st>>>(probs, s.T, s.E, partial);
    int rc = check_launch();
    if (rc) return rc;
    aux_final_kernel<<<1, 256, 0, st>>>(partial, nblk, load, s.T, s.E, alpha, f, P, loss);
    return check_launch();
}

// The same loss from column sums the gate has already formed per CTA (locmoe_gate_ex): only the second level runs.
int launch_aux_from_partials(const locmoe_shape_t& s, const float* p_part, int n_rows, const int32_t* load, float alpha,
                             float* f, float* P, float* loss, cudaStream_t st) {
    aux_final_kernel<<<1, 256, 0, st>>>(p_part, n_rows, load, s.T, s.E, alpha, f, P, loss);
    return check_launch();
}

}  // namespace locmoe
