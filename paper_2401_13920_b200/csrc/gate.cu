// GrAP gate kernel (Sec. 3.2.1): group means, ReLU, softmax, top-1, score, cosine.
//
// The token matrix is read exactly once, with 16-byte streaming loads, one warp
// per token row.  A lane sums the elements of each "unit" (the largest run of
// elements inside one 16-byte vector that cannot straddle a group boundary)
// in registers, drops the unit sums into a per-warp shared-memory strip, and
// after the row has been consumed the lanes add up the strip group by group.
// The strip is padded per group so that those reads are bank-conflict free.
// The next chunk of loads (possibly of the warp's next row) is always in
// flight while the current one is being reduced.
#include <math.h>

#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kCH = 4;  // 16-byte vectors per lane per chunk

struct GateArgs {
    const void* x;
    const float* eps;
    int32_t* idx;
    float* gate_w;
    float* cos_sim;
    float* probs;
    int T, H, E, g;
    int V;            // 16-byte vectors per row
    int nch;          // chunks per row
    int PU;           // units per group
    int PS;           // padded strip stride per group (floats)
    uint32_t magic;   // ceil(2^32 / PU) for p / PU by multiply-high
    int S, logS;      // lanes cooperating on one group in the strip reduction
    int warp_floats;  // shared floats per warp
    float inv_g, sqrt_g;
};

template <int DT>
struct Vec;
template <>
struct Vec<LOCMOE_F32> {
    static constexpr int VE = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <>
struct Vec<LOCMOE_BF16> {
    static constexpr int VE = 8;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
        f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
        f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
    }
};

// Sum of U consecutive floats as a balanced tree.
template <int U>
__device__ __forceinline__ float tree_sum(const float* f) {
    if constexpr (U == 1) return f[0];
    else return tree_sum<U / 2>(f) + tree_sum<U / 2>(f + U / 2);
}

// Softmax / arg-max / cosine of one row from the raw group sums in gsum[E].
__device__ __forceinline__ void gate_epilogue(const GateArgs& a, const float* gsum, float sq, int row, int lane) {
    const unsigned full = 0xffffffffu;
    float best = -1.0f;  // every logit is >= 0 after the ReLU
    int bi = 0x7fffffff;
    for (int i = lane; i < a.E; i += kWarp) {
        float G = fmaxf(gsum[i] * a.inv_g + (a.eps ? a.eps[i] : 0.0f), 0.0f);
        if (G > best) { best = G; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ob = __shfl_xor_sync(full, best, o);
        int oi = __shfl_xor_sync(full, bi, o);
        if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    float se = 0.0f;
    for (int i = lane; i < a.E; i += kWarp) {
        float G = fmaxf(gsum[i] * a.inv_g + (a.eps ? a.eps[i] : 0.0f), 0.0f);
        se += expf(G - best);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        se += __shfl_xor_sync(full, se, o);
        sq += __shfl_xor_sync(full, sq, o);
    }
    const float R = 1.0f / se;
    if (a.probs) {
        float* pr = a.probs + (size_t)row * a.E;
        for (int i = lane; i < a.E; i += kWarp) {
            float G = fmaxf(gsum[i] * a.inv_g + (a.eps ? a.eps[i] : 0.0f), 0.0f);
            pr[i] = expf(G - best) * R;
        }
    }
    if (lane == 0) {
        float nrm = sqrtf(sq);
        a.idx[row] = bi;
        a.gate_w[row] = R;
        a.cos_sim[row] = nrm > 0.0f ? gsum[bi] / (a.sqrt_g * nrm) : 0.0f;
    }
}

template <int DT, int U>
__global__ void __launch_bounds__(256) gate_vec_kernel(const GateArgs a) {
    constexpr int VE = Vec<DT>::VE;
    constexpr int UPV = VE / U;  // units per vector
    extern __shared__ float smem[];
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int wpb = blockDim.x >> 5;
    float* part = smem + (size_t)wib * a.warp_floats;
    float* gsum = part + (size_t)a.E * a.PS;
    const int nw = gridDim.x * wpb;
    const uint4* xv = reinterpret_cast<const uint4*>(a.x);
    const int pad = a.PS - a.PU;

    uint4 cur[kCH], nxt[kCH];
    int row = blockIdx.x * wpb + wib, ch = 0;
    float sq = 0.0f;

    auto load = [&](uint4 (&buf)[kCH], int r, int c) {
        const uint4* base = xv + (size_t)r * a.V;
#pragma unroll
        for (int k = 0; k < kCH; ++k) {
            int v = (c * kCH + k) * kWarp + lane;
            buf[k] = (v < a.V) ? ld_stream(base + v) : make_uint4(0, 0, 0, 0);
        }
    };

    if (row < a.T) load(cur, row, 0);
    while (row < a.T) {
        int ch2 = ch + 1, row2 = row;
        if (ch2 == a.nch) { ch2 = 0; row2 = row + nw; }
        if (row2 < a.T) load(nxt, row2, ch2);

#pragma unroll
        for (int k = 0; k < kCH; ++k) {
            int v = (ch * kCH + k) * kWarp + lane;
            if (v < a.V) {
                float f[VE];
                Vec<DT>::unpack(cur[k], f);
#pragma unroll
                for (int e = 0; e < VE; ++e) sq = fmaf(f[e], f[e], sq);
#pragma unroll
                for (int u = 0; u < UPV; ++u) {
                    int p = v * UPV + u;
                    int q = pad ? p + (int)__umulhi((uint32_t)p, a.magic) * pad : p;
                    part[q] = tree_sum<U>(f + u * U);
                }
            }
        }

        if (ch2 == 0) {  // row complete: reduce the strip group by group
            __syncwarp();
            if (a.S == 1) {
                for (int i = lane; i < a.E; i += kWarp) {
                    const float* pp = part + (size_t)i * a.PS;
                    float s = 0.0f;
                    for (int k = 0; k < a.PU; ++k) s += pp[k];
                    gsum[i] = s;
                }
            } else {
                int i = lane >> a.logS, sl = lane & (a.S - 1);
                float s = 0.0f;
                if (i < a.E) {
                    const float* pp = part + (size_t)i * a.PS;
                    for (int k = sl; k < a.PU; k += a.S) s += pp[k];
                }
                for (int o = a.S >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(full, s, o);
                if (i < a.E && sl == 0) gsum[i] = s;
            }
            __syncwarp();
            gate_epilogue(a, gsum, sq, row, lane);
            __syncwarp();
            sq = 0.0f;
        }
#pragma unroll
        for (int k = 0; k < kCH; ++k) cur[k] = nxt[k];
        row = row2;
        ch = ch2;
    }
}

// Fallback for rows that are not 16-byte friendly: plain element loads, one warp per row.
template <int DT>
__global__ void __launch_bounds__(256) gate_scalar_kernel(const GateArgs a) {
    extern __shared__ float smem[];
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int wpb = blockDim.x >> 5;
    float* gsum = smem + (size_t)wib * a.warp_floats;
    const int nw = gridDim.x * wpb;
    for (int row = blockIdx.x * wpb + wib; row < a.T; row += nw) {
        float sq = 0.0f;
        for (int i = 0; i < a.E; ++i) {
            float s = 0.0f;
            for (int j = lane; j < a.g; j += kWarp) {
                size_t o = (size_t)row * a.H + (size_t)i * a.g + j;
                float v;
                if (DT == LOCMOE_F32) v = reinterpret_cast<const float*>(a.x)[o];
                else v = __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(a.x)[o]) << 16);
                s += v;
                sq = fmaf(v, v, sq);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(full, s, o);
            if (lane == 0) gsum[i] = s;
        }
        __syncwarp();
        gate_epilogue(a, gsum, sq, row, lane);
        __syncwarp();
    }
}

int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

template <typename K>
int launch_persistent(K kernel, const GateArgs& a, int max_warps, cudaStream_t st) {
    // Largest CTA (in warps) whose strips fit in shared memory, then as many CTAs as are resident.
    int wpb = max_warps;
    size_t smem = 0;
    for (; wpb >= 1; wpb >>= 1) {
        smem = (size_t)wpb * a.warp_floats * sizeof(float);
        if (smem <= 200 * 1024) break;
    }
    if (wpb < 1) return LOCMOE_ERR_SHAPE;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, wpb * 32, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    long long want = ((long long)a.T + wpb - 1) / wpb;
    long long grid = (long long)per_sm * sm_count();
    if (grid > want) grid = want;
    kernel<<<(unsigned)grid, wpb * 32, smem, st>>>(a);
    return check_launch();
}

}  // namespace

int launch_gate(const locmoe_shape_t& s, const void* x, const float* eps, int32_t* idx, float* gate_w,
                float* cos_sim, float* probs, cudaStream_t st) {
    GateArgs a{};
    a.x = x; a.eps = eps; a.idx = idx; a.gate_w = gate_w; a.cos_sim = cos_sim; a.probs = probs;
    a.T = s.T; a.H = s.H; a.E = s.E; a.g = s.H / s.E;
    a.inv_g = 1.0f / (float)a.g;
    a.sqrt_g = sqrtf((float)a.g);
    const int esz = s.x_dtype == LOCMOE_F32 ? 4 : 2;
    const int VE = 16 / esz;
    const bool vec_ok = ((size_t)s.H * esz) % 16 == 0 && ((uintptr_t)x % 16) == 0 && s.H <= 65535;
    if (!vec_ok) {
        a.warp_floats = (s.E + 3) & ~3;
        if (s.x_dtype == LOCMOE_F32) return launch_persistent(gate_scalar_kernel<LOCMOE_F32>, a, 8, st);
        return launch_persistent(gate_scalar_kernel<LOCMOE_BF16>, a, 8, st);
    }
    const int U = gcd_int(a.g, VE);
    a.V = s.H / VE;
    a.nch = (a.V + kCH * kWarp - 1) / (kCH * kWarp);
    a.PU = a.g / U;
    a.S = 1; a.logS = 0;
    while (a.S * 2 * s.E <= kWarp && a.S * 2 <= a.PU) { a.S *= 2; a.logS++; }
    // stride congruent to S modulo 2S keeps the strip reads of a warp in distinct banks
    a.PS = a.PU;
    if (a.PU > 1) while (a.PS % (2 * a.S) != a.S) a.PS++;
    a.magic = a.PU > 1 ? (uint32_t)((0x100000000ull + a.PU - 1) / a.PU) : 0u;
    a.warp_floats = (s.E * a.PS + s.E + 3) & ~3;
#define LOCMOE_GATE_CASE(DT, UU) \
    if (s.x_dtype == DT && U == UU) return launch_persistent(gate_vec_kernel<DT, UU>, a, 8, st);
    LOCMOE_GATE_CASE(LOCMOE_F32, 4)
    LOCMOE_GATE_CASE(LOCMOE_F32, 2)
    LOCMOE_GATE_CASE(LOCMOE_F32, 1)
    LOCMOE_GATE_CASE(LOCMOE_BF16, 8)
    LOCMOE_GATE_CASE(LOCMOE_BF16, 4)
    LOCMOE_GATE_CASE(LOCMOE_BF16, 2)
    LOCMOE_GATE_CASE(LOCMOE_BF16, 1)
#undef LOCMOE_GATE_CASE
    return LOCMOE_ERR_DTYPE;
}

}  // namespace locmoe
