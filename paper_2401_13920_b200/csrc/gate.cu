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
#include <stdlib.h>

#include "capacity_finish.cuh"
#include "common.cuh"

namespace locmoe {

namespace {

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
    int S, logS;      // lanes cooperating on one group in the strip reduction
    int warp_floats;  // shared floats per warp
    int tab_ints;     // shared ints of the strip-offset table (one per unit of a row)
    float inv_g, sqrt_g;
    GateFuse f;       // route-stage work carried by the gate (f.src == nullptr: none)
    const int32_t* bias_src;  // per-source bias table: eps is [bias_D][E] and token t takes row bias_src[t] (nullptr: eps is [E])
    int bias_D;
    float* p_part;    // [grid][E] per-CTA column sums of the probabilities (kernels built with PS only; nullptr: none)
    int pacc_floats;  // shared floats per warp for those sums (E, or 0)
};

// The bias row of a token: eps itself, or the row of the per-source table (no bias for an impossible source).
__device__ __forceinline__ const float* bias_row(const GateArgs& a, int sd) {
    if (!a.bias_src || !a.eps) return a.eps;
    return (unsigned)sd < (unsigned)a.bias_D ? a.eps + (size_t)sd * a.E : nullptr;
}

// End of a kernel built with PS: the CTA adds up its warps' column sums in warp order and writes its row.
__device__ __forceinline__ void write_p_part(const GateArgs& a, const float* pacc_base, int wpb) {
    __syncthreads();
    for (int i = threadIdx.x; i < a.E; i += blockDim.x) {
        float s = 0.0f;
        for (int ww = 0; ww < wpb; ++ww) s += pacc_base[(size_t)ww * a.pacc_floats + i];
        a.p_part[(size_t)blockIdx.x * a.E + i] = s;
    }
}

// Lane 0 of the warp that finished token `row`: the route stage's first pass over the tokens, done here.
// sd = src[row], fetched by the caller (the specialised kernel prefetches it with the row).
__device__ __forceinline__ void gate_route_hook(const GateArgs& a, int row, int bi, float cosv, int sd) {
    if (!a.f.src) return;
    // min_sets copies of the row of minima, chosen by the token index: 1 / min_sets of the same-address atomics
    // (64 experts and 65536 tokens on one row cost 29 us of L2 atomic back-pressure)
    atomicMin(&a.f.cap_min[(size_t)(row & (a.f.min_sets - 1)) * a.E + bi], order_code(cosv));
    if ((unsigned)sd >= (unsigned)a.f.D) {
        a.f.pos[row] = -1; a.f.slot[row] = -1; a.f.drop[row] = 1;
        atomicOr(a.f.status, LOCMOE_WARN_BAD_SRC);
        return;
    }
    const int key = sd * a.E + bi;
    atomicAdd(&a.f.counts[key], 1);
    atomicAdd(&a.f.hist0[(size_t)(key & a.f.digit_mask) * a.f.hstride + (row >> a.f.tile_shift)], 1);
}

// A 16-byte vector as NP packed pairs of floats (Blackwell has two-wide fp32 add / fma).
template <int DT>
struct Vec;
template <>
struct Vec<LOCMOE_F32> {
    static constexpr int NP = 2;
    __device__ static __forceinline__ void unpack(const uint4& v, float2 (&p)[2]) {
        p[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        p[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
};
template <>
struct Vec<LOCMOE_BF16> {
    static constexpr int NP = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float2 (&p)[4]) {
        p[0] = make_float2(bf16_lo(v.x), bf16_hi(v.x));
        p[1] = make_float2(bf16_lo(v.y), bf16_hi(v.y));
        p[2] = make_float2(bf16_lo(v.z), bf16_hi(v.z));
        p[3] = make_float2(bf16_lo(v.w), bf16_hi(v.w));
    }
};

// Sum of NPAIR consecutive pairs (a balanced tree of two-wide adds, then one scalar add).
template <int NPAIR>
__device__ __forceinline__ float2 pair_tree(const float2* p) {
    if constexpr (NPAIR == 1) return p[0];
    else return __fadd2_rn(pair_tree<NPAIR / 2>(p), pair_tree<NPAIR / 2>(p + NPAIR / 2));
}

// Softmax / arg-max / cosine of one row from the raw group sums in gsum[E].
template <bool EX>
__device__ __forceinline__ void gate_epilogue(const GateArgs& a, const float* gsum, float sq, int row, int lane, float* pacc) {
    const unsigned full = 0xffffffffu;
    const float* eps = EX ? bias_row(a, a.bias_src ? a.bias_src[row] : 0) : a.eps;
    float best = -1.0f;  // every logit is >= 0 after the ReLU
    int bi = 0x7fffffff;
    for (int i = lane; i < a.E; i += kWarp) {
        float G = fmaxf(gsum[i] * a.inv_g + (eps ? eps[i] : 0.0f), 0.0f);
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
        float G = fmaxf(gsum[i] * a.inv_g + (eps ? eps[i] : 0.0f), 0.0f);
        se += __expf(G - best);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        se += __shfl_xor_sync(full, se, o);
        sq += __shfl_xor_sync(full, sq, o);
    }
    const float R = 1.0f / se;
    if (a.probs || pacc) {
        float* pr = a.probs ? a.probs + (size_t)row * a.E : nullptr;
        for (int i = lane; i < a.E; i += kWarp) {
            float G = fmaxf(gsum[i] * a.inv_g + (eps ? eps[i] : 0.0f), 0.0f);
            const float pv = __expf(G - best) * R;
            if (pr) pr[i] = pv;
            if (pacc) pacc[i] += pv;      // lane i owns column i, i + 32, ...: rows are added in the warp's row order
        }
    }
    if (lane == 0) {
        float nrm = sqrtf(sq);
        const float cosv = nrm > 0.0f ? gsum[bi] / (a.sqrt_g * nrm) : 0.0f;
        a.idx[row] = bi;
        a.gate_w[row] = R;
        a.cos_sim[row] = cosv;
        gate_route_hook(a, row, bi, cosv, a.f.src ? a.f.src[row] : 0);
    }
}

// DT: token dtype.  U: elements per unit.  CH: vectors per lane per chunk.
// EXACT: the row is a whole number of chunks (no bounds tests in the loop).
template <int DT, int U, int CH, bool EXACT, bool PS>
__global__ void __launch_bounds__(256, 4) gate_vec_kernel(const GateArgs a) {
    pdl_wait();
    pdl_trigger();
    constexpr int NP = Vec<DT>::NP;
    constexpr int VE = 2 * NP;
    constexpr int UPV = VE / U;  // units per vector
    extern __shared__ float smem[];
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int wpb = blockDim.x >> 5;
    // strip offset (in floats) of every unit of a row: unit p of group p / PU sits at p + (p / PU) * pad
    int* tab = reinterpret_cast<int*>(smem);
    {
        const int pad = a.PS - a.PU;
        for (int p = threadIdx.x; p < a.V * UPV; p += blockDim.x) tab[p] = p + (p / a.PU) * pad;
    }
    __syncthreads();
    float* part = smem + a.tab_ints + (size_t)wib * a.warp_floats;
    float* gsum = part + (size_t)a.E * a.PS;
    float* pacc_base = smem + a.tab_ints + (size_t)wpb * a.warp_floats;
    float* pacc = (PS && a.p_part) ? pacc_base + (size_t)wib * a.pacc_floats : nullptr;
    if (pacc) for (int i = lane; i < a.E; i += kWarp) pacc[i] = 0.0f;
    const int nw = gridDim.x * wpb;
    const uint4* xv = reinterpret_cast<const uint4*>(a.x);

    uint4 bufA[CH], bufB[CH];
    float2 sq2 = make_float2(0.0f, 0.0f);

    auto load = [&](uint4 (&buf)[CH], int r, int c) {
        const uint4* base = xv + (size_t)r * a.V + c * (CH * kWarp) + lane;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            if (EXACT || c * (CH * kWarp) + k * kWarp + lane < a.V) buf[k] = ld_stream(base + k * kWarp);
            else buf[k] = make_uint4(0, 0, 0, 0);
        }
    };

    auto consume = [&](const uint4 (&buf)[CH], int c) {
        const int v0 = c * (CH * kWarp) + lane;
        const int* tb = tab + v0 * UPV;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            if (EXACT || v0 + k * kWarp < a.V) {
                float2 p[NP];
                Vec<DT>::unpack(buf[k], p);
#pragma unroll
                for (int e = 0; e < NP; ++e) sq2 = __ffma2_rn(p[e], p[e], sq2);
                if constexpr (U >= 2) {
                    constexpr int PPU = U / 2;  // pairs per unit
#pragma unroll
                    for (int u = 0; u < UPV; ++u) {
                        float2 s2 = pair_tree<PPU>(p + u * PPU);
                        part[tb[k * kWarp * UPV + u]] = s2.x + s2.y;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < NP; ++e) {
                        part[tb[k * kWarp * UPV + 2 * e]] = p[e].x;
                        part[tb[k * kWarp * UPV + 2 * e + 1]] = p[e].y;
                    }
                }
            }
        }
    };

    auto finish_row = [&](int row) {  // the strip holds a whole row: reduce it group by group
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
        gate_epilogue<PS>(a, gsum, sq2.x + sq2.y, row, lane, pacc);
        __syncwarp();
        sq2 = make_float2(0.0f, 0.0f);
    };

    int row = blockIdx.x * wpb + wib, ch = 0;
    if (!PS && row >= a.T) return;
    if (row < a.T) {
        load(bufA, row, 0);
        while (true) {
            int ch2 = ch + 1, row2 = row;
            if (ch2 == a.nch) { ch2 = 0; row2 = row + nw; }
            if (row2 < a.T) load(bufB, row2, ch2);
            consume(bufA, ch);
            if (ch2 == 0) finish_row(row);
            if (row2 >= a.T) break;
            row = row2; ch = ch2;

            ch2 = ch + 1; row2 = row;
            if (ch2 == a.nch) { ch2 = 0; row2 = row + nw; }
            if (row2 < a.T) load(bufA, row2, ch2);
            consume(bufB, ch);
            if (ch2 == 0) finish_row(row);
            if (row2 >= a.T) break;
            row = row2; ch = ch2;
        }
    }
    if (PS && a.p_part) write_p_part(a, pacc_base, wpb);
}

// Specialised bf16 kernel for the common shapes: the row is a whole number of chunks, every lane owns exactly NGK
// groups (E = 32 * NGK) of PUK units each.  With PUK and NGK known at compile time the strip needs neither padding
// nor an offset table (a stride of PUK floats between lanes is at worst a 2-way bank conflict for the PUK values
// instantiated; PUK % 4 == 0 is read with 16-byte loads), the group sums and logits stay in registers, and the
// winner's raw sum for the cosine comes from a shuffle.  About half the instructions of the general kernel.
template <int PUK>
__device__ __forceinline__ float strip_sum(const float* pp) {
    if constexpr (PUK % 4 == 0) {
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < PUK / 4; ++k) {
            const float4 v = reinterpret_cast<const float4*>(pp)[k];
            s += (v.x + v.y) + (v.z + v.w);
        }
        return s;
    } else if constexpr (PUK % 2 == 0) {
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < PUK / 2; ++k) {
            const float2 v = reinterpret_cast<const float2*>(pp)[k];
            s += v.x + v.y;
        }
        return s;
    } else {
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < PUK; ++k) s += pp[k];
        return s;
    }
}

template <int U, int CH, int PUK, int NGK, bool PS>
__global__ void __launch_bounds__(256, 4) gate_fast_kernel(const GateArgs a) {
    pdl_wait();
    pdl_trigger();
    constexpr int NP = 4, VE = 8, UPV = VE / U;
    extern __shared__ float smem[];
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int wpb = blockDim.x >> 5;
    float* part = smem + (size_t)wib * a.warp_floats;
    float* pacc_base = smem + (size_t)wpb * a.warp_floats;
    float* pacc = (PS && a.p_part) ? pacc_base + (size_t)wib * a.pacc_floats : nullptr;
    if (pacc) {
#pragma unroll
        for (int m = 0; m < NGK; ++m) pacc[lane + 32 * m] = 0.0f;
    }
    const int nw = gridDim.x * wpb;
    const uint4* xv = reinterpret_cast<const uint4*>(a.x);
    constexpr float kLog2e = 1.4426950408889634f;

    uint4 bufA[CH], bufB[CH];
    float2 sq2 = make_float2(0.0f, 0.0f);
    int sd_cur = 0, sd_new = 0;   // source device of the row being reduced / of the row whose first chunk is in flight

    auto load = [&](uint4 (&buf)[CH], int r, int c) {
        const uint4* base = xv + (size_t)r * a.V + c * (CH * kWarp) + lane;
#pragma unroll
        for (int k = 0; k < CH; ++k) buf[k] = ld_stream(base + k * kWarp);
        if (c == 0) {   // source device of the row, for the route hook / the bias row
            if (a.f.src) sd_new = a.f.src[r];
            else if (PS && a.bias_src) sd_new = a.bias_src[r];
        }
    };

    auto consume = [&](const uint4 (&buf)[CH], int c) {
        float* dst = part + (c * (CH * kWarp) + lane) * UPV;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            float2 p[NP];
            Vec<LOCMOE_BF16>::unpack(buf[k], p);
#pragma unroll
            for (int e = 0; e < NP; ++e) sq2 = __ffma2_rn(p[e], p[e], sq2);
            float* d = dst + k * kWarp * UPV;
            if constexpr (U == 8) {
                const float2 s2 = pair_tree<4>(p);
                d[0] = s2.x + s2.y;
            } else if constexpr (U == 4) {
                const float2 lo = __fadd2_rn(p[0], p[1]), hi = __fadd2_rn(p[2], p[3]);
                *reinterpret_cast<float2*>(d) = make_float2(lo.x + lo.y, hi.x + hi.y);
            } else {  // U == 2
                *reinterpret_cast<float4*>(d) = make_float4(p[0].x + p[0].y, p[1].x + p[1].y, p[2].x + p[2].y, p[3].x + p[3].y);
            }
        }
    };

    auto finish_row = [&](int row) {
        __syncwarp();
        float gs[NGK];
#pragma unroll
        for (int m = 0; m < NGK; ++m) gs[m] = strip_sum<PUK>(part + (size_t)(lane + 32 * m) * PUK);
        __syncwarp();  // the strip may now be overwritten by the next row
        // the logits are recomputed in the second pass rather than kept: fewer live registers, no spills
        const float* eps = PS ? bias_row(a, sd_cur) : a.eps;   // without the extras: the caller's row, as it is
        auto logit = [&](int m) { return fmaxf(fmaf(gs[m], a.inv_g, eps ? eps[lane + 32 * m] : 0.0f), 0.0f); };
        float best = -1.0f;
        int bi = 0x7fffffff;
#pragma unroll
        for (int m = 0; m < NGK; ++m) {
            const float G = logit(m);
            if (G > best) { best = G; bi = lane + 32 * m; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(full, best, o);
            const int oi = __shfl_xor_sync(full, bi, o);
            if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
        }
        const float nb = -best * kLog2e;
        float se = 0.0f;
#pragma unroll
        for (int m = 0; m < NGK; ++m) se += exp2f(fmaf(logit(m), kLog2e, nb));
        float sq = sq2.x + sq2.y;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            se += __shfl_xor_sync(full, se, o);
            sq += __shfl_xor_sync(full, sq, o);
        }
        float cand = gs[0];
#pragma unroll
        for (int m = 1; m < NGK; ++m) if ((bi >> 5) == m) cand = gs[m];
        const float wsum = __shfl_sync(full, cand, bi & 31);
        if constexpr (PS) {
            if (a.p_part) {
                const float R = 1.0f / se;
#pragma unroll
                for (int m = 0; m < NGK; ++m) pacc[lane + 32 * m] += exp2f(fmaf(logit(m), kLog2e, nb)) * R;
            }
        }
        if (lane == 0) {
            const float nrm = sqrtf(sq);
            const float cosv = nrm > 0.0f ? wsum / (a.sqrt_g * nrm) : 0.0f;
            a.idx[row] = bi;
            a.gate_w[row] = 1.0f / se;
            a.cos_sim[row] = cosv;
            gate_route_hook(a, row, bi, cosv, sd_cur);
        }
        sq2 = make_float2(0.0f, 0.0f);
        sd_cur = sd_new;
    };

    int row = blockIdx.x * wpb + wib, ch = 0;
    if (!PS && row >= a.T) return;
    if (row < a.T) {
        load(bufA, row, 0);
        sd_cur = sd_new;
        while (true) {
            int ch2 = ch + 1, row2 = row;
            if (ch2 == a.nch) { ch2 = 0; row2 = row + nw; }
            if (row2 < a.T) load(bufB, row2, ch2);
            consume(bufA, ch);
            if (ch2 == 0) finish_row(row);
            if (row2 >= a.T) break;
            row = row2; ch = ch2;

            ch2 = ch + 1; row2 = row;
            if (ch2 == a.nch) { ch2 = 0; row2 = row + nw; }
            if (row2 < a.T) load(bufA, row2, ch2);
            consume(bufB, ch);
            if (ch2 == 0) finish_row(row);
            if (row2 >= a.T) break;
            row = row2; ch = ch2;
        }
    }
    if (PS && a.p_part) write_p_part(a, pacc_base, wpb);
}

// Fallback for rows that are not 16-byte friendly: plain element loads, one warp per row.
template <int DT, bool PS>
__global__ void __launch_bounds__(256) gate_scalar_kernel(const GateArgs a) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ float smem[];
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int wpb = blockDim.x >> 5;
    float* gsum = smem + (size_t)wib * a.warp_floats;
    float* pacc_base = smem + (size_t)wpb * a.warp_floats;
    float* pacc = (PS && a.p_part) ? pacc_base + (size_t)wib * a.pacc_floats : nullptr;
    if (pacc) for (int i = lane; i < a.E; i += kWarp) pacc[i] = 0.0f;
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
        gate_epilogue<PS>(a, gsum, sq, row, lane, pacc);
        __syncwarp();
    }
    if (PS && a.p_part) write_p_part(a, pacc_base, wpb);
}

int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

thread_local int g_last_grid = 0;   // grid of the launch just queued by this thread's call (rows of p_part); set by launch_persistent

template <typename K>
int launch_persistent(K kernel, const GateArgs& a, int max_warps, cudaStream_t st) {
    // Largest CTA (in warps) whose strips fit in shared memory, then as many CTAs as are resident.
    int wpb = max_warps;
    size_t smem = 0;
    for (; wpb >= 1; wpb >>= 1) {
        smem = ((size_t)wpb * (a.warp_floats + a.pacc_floats) + a.tab_ints) * sizeof(float);
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
    if (a.p_part && grid > LOCMOE_GATE_PARTIAL_ROWS) grid = LOCMOE_GATE_PARTIAL_ROWS;
    g_last_grid = (int)grid;
    return launch_pdl(kernel, (unsigned)grid, wpb * 32, smem, st, a);
}

}  // namespace

int gate_last_grid() { return g_last_grid; }

int launch_gate(const locmoe_shape_t& s, const void* x, const float* eps, int32_t* idx, float* gate_w,
                float* cos_sim, float* probs, cudaStream_t st, const GateFuse* fuse, const GateExtra* extra) {
    GateArgs a{};
    if (fuse) a.f = *fuse;
    const bool ps = extra && (extra->p_part || extra->bias_src);   // kernels built with the extras
    if (extra) {
        a.bias_src = extra->bias_src; a.bias_D = s.n_nodes * s.dev_per_node;
        a.p_part = extra->p_part; a.pacc_floats = extra->p_part ? ((s.E + 3) & ~3) : 0;
    }
    a.x = x; a.eps = eps; a.idx = idx; a.gate_w = gate_w; a.cos_sim = cos_sim; a.probs = probs;
    a.T = s.T; a.H = s.H; a.E = s.E; a.g = s.H / s.E;
    a.inv_g = 1.0f / (float)a.g;
    a.sqrt_g = sqrtf((float)a.g);
    const int esz = s.x_dtype == LOCMOE_F32 ? 4 : 2;
    const int VE = 16 / esz;
    const bool vec_ok = ((size_t)s.H * esz) % 16 == 0 && ((uintptr_t)x % 16) == 0 && s.H <= 65535;
    if (!vec_ok) {
        a.warp_floats = (s.E + 3) & ~3;
        if (s.x_dtype == LOCMOE_F32) return ps ? launch_persistent(gate_scalar_kernel<LOCMOE_F32, true>, a, 8, st)
                                               : launch_persistent(gate_scalar_kernel<LOCMOE_F32, false>, a, 8, st);
        return ps ? launch_persistent(gate_scalar_kernel<LOCMOE_BF16, true>, a, 8, st)
                  : launch_persistent(gate_scalar_kernel<LOCMOE_BF16, false>, a, 8, st);
    }
    const int U = gcd_int(a.g, VE);
    a.V = s.H / VE;
    a.PU = a.g / U;
    a.S = 1; a.logS = 0;
    while (a.S * 2 * s.E <= kWarp && a.S * 2 <= a.PU) { a.S *= 2; a.logS++; }
    // stride congruent to S modulo 2S keeps the strip reads of a warp in distinct banks
    a.PS = a.PU;
    if (a.PU > 1) while (a.PS % (2 * a.S) != a.S) a.PS++;
    a.warp_floats = (s.E * a.PS + s.E + 3) & ~3;
    a.tab_ints = (s.H / U + 3) & ~3;
    // chunk size: prefer one that divides the row exactly (no bounds tests in the loop)
    const int per_lane = a.V / kWarp;
    const bool whole = a.V % kWarp == 0;
    int CH = 4;
    bool exact = whole && per_lane % 4 == 0;
    if (!exact && whole && per_lane % 5 == 0) { CH = 5; exact = true; }
    a.nch = (a.V + CH * kWarp - 1) / (CH * kWarp);
    // specialised kernel for the common bf16 shapes (whole chunks, E a multiple of 32 with a known group layout);
    // LOCMOE_GATE=general keeps the general kernel (testing aid)
    if (s.x_dtype == LOCMOE_BF16 && exact && probs == nullptr && a.S == 1 && s.E % 32 == 0 &&
        !(getenv("LOCMOE_GATE") && getenv("LOCMOE_GATE")[0] == 'g')) {
        const int NG = s.E / 32;
        GateArgs f = a;
        f.warp_floats = (s.H / U + 3) & ~3;
        f.tab_ints = 0;
#define LOCMOE_FAST_CASE(UU, CC, PP, NN) \
        if (U == UU && CH == CC && a.PU == PP && NG == NN)                                      \
            return ps ? launch_persistent(gate_fast_kernel<UU, CC, PP, NN, true>, f, 8, st)     \
                      : launch_persistent(gate_fast_kernel<UU, CC, PP, NN, false>, f, 8, st);
        LOCMOE_FAST_CASE(8, 4, 10, 2)   // H = 5120, E = 64
        LOCMOE_FAST_CASE(8, 5, 10, 1)   // H = 2560, E = 32
        LOCMOE_FAST_CASE(8, 4, 4, 4)    // H = 4096, E = 128
        LOCMOE_FAST_CASE(4, 4, 5, 8)    // H = 5120, E = 256
        LOCMOE_FAST_CASE(8, 4, 8, 2)    // H = 4096, E = 64
        LOCMOE_FAST_CASE(4, 4, 7, 8)    // H = 7168, E = 256
        LOCMOE_FAST_CASE(8, 4, 16, 1)   // H = 4096, E = 32
#undef LOCMOE_FAST_CASE
    }
#define LOCMOE_GATE_CASE(DT, UU)                                                                              \
    if (s.x_dtype == DT && U == UU) {                                                                         \
        if (exact && CH == 4) return ps ? launch_persistent(gate_vec_kernel<DT, UU, 4, true, true>, a, 8, st)   \
                                        : launch_persistent(gate_vec_kernel<DT, UU, 4, true, false>, a, 8, st); \
        if (exact && CH == 5) return ps ? launch_persistent(gate_vec_kernel<DT, UU, 5, true, true>, a, 8, st)   \
                                        : launch_persistent(gate_vec_kernel<DT, UU, 5, true, false>, a, 8, st); \
        return ps ? launch_persistent(gate_vec_kernel<DT, UU, 4, false, true>, a, 8, st)                        \
                  : launch_persistent(gate_vec_kernel<DT, UU, 4, false, false>, a, 8, st);                      \
    }
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
