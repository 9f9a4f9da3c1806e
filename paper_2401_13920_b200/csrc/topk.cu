// Top-k variant of the router (the paper itself routes top-1; k > 1 is the family of routers it departs from).
//   select : the K experts with the largest gate probability per token, in descending order, a tie going to the
//            lower index; choice 0 is the gate's own arg-max and score.
//   fold   : the route stage is run on K * T "virtual tokens" v = c * T + t (all first choices before all second
//            choices, so a first choice never loses its slot to a second one); folding inv[row] to v mod T lets
//            the ordinary dispatch copy the right token row.
//   combine: out[t] = sum over the K choices of w_c * y[slot_c[t]] (first equation of Sec. 3.2.1 restricted to
//            the chosen experts), accumulated in fp32 in choice order and rounded once.
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxK = 8;

__global__ void __launch_bounds__(kThreads) topk_select_kernel(const float* __restrict__ probs, const int32_t* __restrict__ idx,
                                                               const float* __restrict__ gate_w, int T, int E, int K,
                                                               int32_t* __restrict__ idx_k, float* __restrict__ w_k) {
    const int lane = threadIdx.x & 31;
    const int nw = gridDim.x * (kThreads / 32);
    for (int t = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); t < T; t += nw) {
        const float* p = probs + (size_t)t * E;
        int chosen[kMaxK];
        chosen[0] = idx[t];
        if (lane == 0) { idx_k[t] = chosen[0]; w_k[t] = gate_w[t]; }
        for (int c = 1; c < K; ++c) {
            float best = -1.0f;
            int bi = 0x7fffffff;
            for (int i = lane; i < E; i += 32) {
                bool taken = false;
#pragma unroll
                for (int q = 0; q < kMaxK; ++q) taken |= q < c && chosen[q] == i;
                const float v = p[i];
                if (!taken && v > best) { best = v; bi = i; }   // ascending i: the lower index wins a tie
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
            chosen[c] = bi;
            if (lane == 0) { idx_k[(size_t)c * T + t] = bi; w_k[(size_t)c * T + t] = best; }
        }
    }
}

__global__ void __launch_bounds__(kThreads) topk_fold_kernel(int32_t* __restrict__ inv, long long rows, int T) {
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long r = (long long)blockIdx.x * kThreads + threadIdx.x; r < rows; r += stride) {
        const int v = inv[r];
        if (v >= T) inv[r] = v % T;
    }
}

// One octet (8 elements) of a row: raw 16-byte loads now, widening to fp32 at the point of use (fewer live registers).
struct RawOctet { uint4 a, b; };
__device__ __forceinline__ void load_raw(const void* base, size_t octet, int dt, RawOctet& r) {
    if (dt == LOCMOE_F32) {
        const uint4* p = reinterpret_cast<const uint4*>(base) + octet * 2;
        r.a = ld_stream(p); r.b = ld_stream(p + 1);
    } else {
        r.a = ld_stream(reinterpret_cast<const uint4*>(base) + octet);
    }
}
__device__ __forceinline__ void widen8(const RawOctet& r, int dt, float (&f)[8]) {
    if (dt == LOCMOE_F32) {
        f[0] = __uint_as_float(r.a.x); f[1] = __uint_as_float(r.a.y); f[2] = __uint_as_float(r.a.z); f[3] = __uint_as_float(r.a.w);
        f[4] = __uint_as_float(r.b.x); f[5] = __uint_as_float(r.b.y); f[6] = __uint_as_float(r.b.z); f[7] = __uint_as_float(r.b.w);
    } else {
        f[0] = bf16_lo(r.a.x); f[1] = bf16_hi(r.a.x); f[2] = bf16_lo(r.a.y); f[3] = bf16_hi(r.a.y);
        f[4] = bf16_lo(r.a.z); f[5] = bf16_hi(r.a.z); f[6] = bf16_lo(r.a.w); f[7] = bf16_hi(r.a.w);
    }
}

template <int K, int YDT>
__global__ void __launch_bounds__(kThreads) combine_topk_kernel(const void* __restrict__ y,
                                                                const int32_t* __restrict__ slot_k,
                                                                const float* __restrict__ w_k, void* __restrict__ out, int odt,
                                                                int T, int O, long long rows, int tpc) {
    const int lane = threadIdx.x & 31;
    const long long t_lo = (long long)blockIdx.x * tpc;
    const int t_hi = (int)min((long long)T, t_lo + tpc);
    for (int t = (int)t_lo + (threadIdx.x >> 5); t < t_hi; t += kThreads / 32) {
        int s[K];
        float w[K];
#pragma unroll
        for (int c = 0; c < K; ++c) {
            s[c] = slot_k[(size_t)c * T + t];
            w[c] = w_k[(size_t)c * T + t];
            if (s[c] < 0 || s[c] >= rows) s[c] = -1;
        }
        // octets in flight per lane: two for small K (as the top-1 combine), one otherwise (registers)
        constexpr int NO = K <= 2 ? 2 : 1;
        for (int o0 = lane; o0 < O; o0 += 32 * NO) {
            RawOctet raw[NO][K];
#pragma unroll
            for (int h = 0; h < NO; ++h) {
                const int o = o0 + 32 * h;
                if (o < O) {
#pragma unroll
                    for (int c = 0; c < K; ++c)
                        if (s[c] >= 0) load_raw(y, (size_t)s[c] * O + o, YDT, raw[h][c]);
                }
            }
#pragma unroll
            for (int h = 0; h < NO; ++h) {
                const int o = o0 + 32 * h;
                if (o >= O) continue;
                float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                bool first = true;
#pragma unroll
                for (int c = 0; c < K; ++c) {
                    if (s[c] < 0) continue;
                    float v[8];
                    widen8(raw[h][c], YDT, v);
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] = first ? __fmul_rn(w[c], v[k]) : __fmaf_rn(w[c], v[k], acc[k]);
                    first = false;
                }
                if (odt == LOCMOE_F32) {
                    uint4* p = reinterpret_cast<uint4*>(out) + ((size_t)t * O + o) * 2;
                    st_stream(p, make_uint4(__float_as_uint(acc[0]), __float_as_uint(acc[1]), __float_as_uint(acc[2]), __float_as_uint(acc[3])));
                    st_stream(p + 1, make_uint4(__float_as_uint(acc[4]), __float_as_uint(acc[5]), __float_as_uint(acc[6]), __float_as_uint(acc[7])));
                } else {
                    st_stream(reinterpret_cast<uint4*>(out) + (size_t)t * O + o,
                              make_uint4(cvt_bf16x2(make_float2(acc[0], acc[1])), cvt_bf16x2(make_float2(acc[2], acc[3])),
                                         cvt_bf16x2(make_float2(acc[4], acc[5])), cvt_bf16x2(make_float2(acc[6], acc[7]))));
                }
            }
        }
    }
}

}  // namespace

int launch_topk_select(const locmoe_shape_t& s, const float* probs, const int32_t* idx, const float* gate_w, int K,
                       int32_t* idx_k, float* w_k, cudaStream_t st) {
    int blocks = (s.T + 7) / 8;
    if (blocks > 32 * sm_count()) blocks = 32 * sm_count();
    topk_select_kernel<<<blocks, kThreads, 0, st>>>(probs, idx, gate_w, s.T, s.E, K, idx_k, w_k);
    return check_launch();
}

int launch_topk_fold(int T, long long rows, int32_t* inv, cudaStream_t st) {
    long long blocks = (rows + kThreads * 4 - 1) / (kThreads * 4);
    if (blocks > 8ll * sm_count()) blocks = 8ll * sm_count();
    if (blocks < 1) blocks = 1;
    topk_fold_kernel<<<(int)blocks, kThreads, 0, st>>>(inv, rows, T);
    return check_launch();
}

int launch_combine_topk(const locmoe_shape_t& s, int64_t rows, const void* y, int y_dtype, int K, const int32_t* slot_k,
                        const float* w_k, void* out, cudaStream_t st) {
    long long want = ((long long)s.T + 7) / 8, cap = 1024ll * sm_count();
    const int grid = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    const int tpc = (s.T + grid - 1) / grid;
    const int O = s.H / 8;
#define LOCMOE_TOPK_CASE(KK)                                                                                           \
    case KK:                                                                                                           \
        if (y_dtype == LOCMOE_F32)                                                                                     \
            combine_topk_kernel<KK, LOCMOE_F32><<<grid, kThreads, 0, st>>>(y, slot_k, w_k, out, s.x_dtype, s.T, O, rows, tpc);  \
        else                                                                                                           \
            combine_topk_kernel<KK, LOCMOE_BF16><<<grid, kThreads, 0, st>>>(y, slot_k, w_k, out, s.x_dtype, s.T, O, rows, tpc); \
        break;
    switch (K) {
        LOCMOE_TOPK_CASE(1) LOCMOE_TOPK_CASE(2) LOCMOE_TOPK_CASE(3) LOCMOE_TOPK_CASE(4)
        LOCMOE_TOPK_CASE(5) LOCMOE_TOPK_CASE(6) LOCMOE_TOPK_CASE(7) LOCMOE_TOPK_CASE(8)
        default: return LOCMOE_ERR_SHAPE;
    }
#undef LOCMOE_TOPK_CASE
    return check_launch();
}

}  // namespace locmoe
