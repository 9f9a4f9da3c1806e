// Dispatch (row gather into the All-to-All shaped buffer) and gate-weighted
// combine (first equation of Sec. 3.2.1, top-1: y_m = R_m * expert output).
//
// Both are row movers bound by HBM: whole rows of a few KB are read with
// 16-byte streaming loads and written with coalesced 16-byte stores, several
// loads per thread in flight before their stores, and grids of many short CTAs
// (a gather of whole rows runs at the DRAM efficiency of a flat copy).
// Dispatch has a token-major kernel (default, needs slot[]), two row-major ones
// and a bulk-copy variant; combine is one warp per token.
#include <stdlib.h>

#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kCH = 4;
constexpr int kThreads = 256;

// Row-major, one warp per buffer row: buf[row] = x[inv[row]] or zeros.  V = 16-byte vectors per row.  Four loads
// per lane are issued before their stores; six CTAs (1536 threads) per SM are resident, which measured faster than
// a deeper software pipeline at half the occupancy.  Used beyond 2^32 vectors, or with LOCMOE_DISPATCH=vec.
__global__ void __launch_bounds__(kThreads, 6) dispatch_vec_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ inv,
                                                                   uint4* __restrict__ buf, long long rows, int V, int T,
                                                                   int zero_pad) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const long long nw = (long long)gridDim.x * (blockDim.x >> 5);
    long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    int t_next = row < rows ? inv[row] : -1;
    for (; row < rows; row += nw) {
        const int t = t_next;
        if (row + nw < rows) t_next = inv[row + nw];
        uint4* dst = buf + row * V;
        if (t < 0 || t >= T) {
            if (zero_pad)
                for (int v = lane; v < V; v += kWarp) st_stream(dst + v, make_uint4(0, 0, 0, 0));
            continue;
        }
        const uint4* srcp = x + (long long)t * V;
        for (int v0 = lane; v0 < V; v0 += kCH * kWarp) {
            uint4 r[kCH];
#pragma unroll
            for (int k = 0; k < kCH; ++k)
                if (v0 + k * kWarp < V) r[k] = ld_stream(srcp + v0 + k * kWarp);
#pragma unroll
            for (int k = 0; k < kCH; ++k)
                if (v0 + k * kWarp < V) st_stream(dst + v0 + k * kWarp, r[k]);
        }
    }
}

// Flat mapping of dispatch (the default when the vector count fits 32 bits): thread -> (row, vector) by index
// arithmetic, four vectors per thread a grid-stride apart; perfectly balanced whatever the mix of empty rows.
__global__ void __launch_bounds__(kThreads) dispatch_flat_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ inv,
                                                                 uint4* __restrict__ buf, unsigned total, unsigned V, int T,
                                                                 int zero_pad) {
    pdl_wait();
    pdl_trigger();
    const unsigned s = gridDim.x * blockDim.x;
    for (unsigned j = blockIdx.x * blockDim.x + threadIdx.x; j < total; j += 4 * s) {
        uint4 r[4];
        bool st[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned jj = j + k * s;
            st[k] = false;
            r[k] = make_uint4(0, 0, 0, 0);
            if (jj < total) {
                const unsigned row = jj / V, v = jj - row * V;
                const int t = __ldg(inv + row);
                if (t >= 0 && t < T) { r[k] = ld_stream(x + (size_t)t * V + v); st[k] = true; }
                else st[k] = zero_pad != 0;
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (st[k]) st_stream(buf + (size_t)(j + k * s), r[k]);
    }
}

// Token-major dispatch (used when the caller supplies slot[]): the (token, vector) items are walked in descending
// token order, every CTA a contiguous run of 8 items per thread, so that the copy starts with the tokens the gate
// read last (still in L2) and ends with the lowest tokens, whose rows a combine in ascending token order reads
// first.  Rows without a token are zero-filled by the same CTAs: CTA b looks at rows [b * zrows, (b + 1) * zrows).
constexpr int kTokIters = 2;
__global__ void __launch_bounds__(kThreads) dispatch_token_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ slot,
                                                                  const int32_t* __restrict__ inv, uint4* __restrict__ buf,
                                                                  unsigned total, unsigned V, int T, long long rows,
                                                                  int zero_pad, int zrows) {
    pdl_wait();
    pdl_trigger();
    const unsigned base = blockIdx.x * (unsigned)(kThreads * 4 * kTokIters);
#pragma unroll
    for (int it = 0; it < kTokIters; ++it) {
        uint4 r[4];
        size_t dst[4];
        bool st[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned jj = base + (unsigned)((it * 4 + k) * kThreads) + threadIdx.x;
            st[k] = false;
            if (jj < total && jj >= base) {
                const unsigned tt = jj / V, v = jj - tt * V;
                const int t = T - 1 - (int)tt;
                const int row = __ldg(slot + t);
                if (row >= 0 && row < rows) {
                    r[k] = ld_stream(x + (size_t)t * V + v);
                    dst[k] = (size_t)row * V + v;
                    st[k] = true;
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (st[k]) st_stream(buf + dst[k], r[k]);
    }
    if (zero_pad) {
        const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
        for (int i = w; i < zrows; i += kThreads / 32) {
            const long long row = (long long)blockIdx.x * zrows + i;
            if (row >= rows) break;
            const int t = __ldg(inv + row);
            if (t >= 0 && t < T) continue;
            uint4* d = buf + row * V;
            for (unsigned v = lane; v < V; v += kWarp) st_stream(d + v, make_uint4(0, 0, 0, 0));
        }
    }
}

// Device-side diagnostics word (bit 0: a bounded barrier wait gave up).  Read with locmoe_device_flags().
__device__ int g_device_flags = 0;

// Dispatch through the bulk-copy engine: global -> shared -> global, no registers in the data path.
// Shared memory holds one zero segment plus one staging segment per warp; lane 0 of every warp runs an
// independent loop over its work items (row segments): wait until its previous store has drained the stage,
// start the bulk load, wait for the mbarrier (bounded), start the bulk store.  With ~20 stages of ~10 KB per
// SM roughly 200 KB per SM are in flight, which is what the HBM latency-bandwidth product asks for.
__global__ void __launch_bounds__(1024, 1) dispatch_tma_kernel(const unsigned char* __restrict__ x,
                                                                const int32_t* __restrict__ inv,
                                                                unsigned char* __restrict__ buf, long long rows,
                                                                int nseg, uint32_t seg, long long rowbytes, int T,
                                                                int zero_pad) {
    extern __shared__ __align__(128) unsigned char smraw[];
    const int nw = blockDim.x >> 5;
    unsigned char* zero = smraw;
    unsigned char* stages = smraw + seg;
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + (size_t)nw * seg);
    for (uint32_t i = threadIdx.x * 16; i < seg; i += blockDim.x * 16) *reinterpret_cast<uint4*>(zero + i) = make_uint4(0, 0, 0, 0);
    if ((int)threadIdx.x < nw) mbar_init(&bars[threadIdx.x], 1);
    mbar_init_fence();
    fence_async_smem();
    __syncthreads();
    if ((threadIdx.x & 31) != 0) return;
    const int w = threadIdx.x >> 5;
    unsigned char* st = stages + (size_t)w * seg;
    uint64_t* bar = &bars[w];
    const long long items = rows * nseg;
    const long long stride = (long long)gridDim.x * nw;
    long long it = (long long)blockIdx.x * nw + w;
    uint32_t phase = 0;
    int t_next = it < items ? inv[it / nseg] : -1;
    for (; it < items; it += stride) {
        const int t = t_next;
        if (it + stride < items) t_next = inv[(it + stride) / nseg];
        const long long row = it / nseg;
        const long long off = (it - row * nseg) * seg;
        unsigned char* dst = buf + row * rowbytes + off;
        if (t < 0 || t >= T) {
            if (zero_pad) { bulk_s2g(dst, zero, seg); bulk_commit(); }
            continue;
        }
        bulk_wait_read<0>();  // the previous store of this lane has finished reading the stage
        mbar_expect_tx(bar, seg);
        bulk_g2s(st, x + (long long)t * rowbytes + off, seg, bar);
        if (!mbar_wait_bounded(bar, phase)) { atomicOr(&g_device_flags, 1); break; }
        phase ^= 1u;
        bulk_s2g(dst, st, seg);
        bulk_commit();
    }
    bulk_wait_all<0>();
}

// Element-wise fallback for rows that are not a multiple of 16 bytes or misaligned bases.
template <typename E>
__global__ void __launch_bounds__(kThreads) dispatch_scalar_kernel(const E* __restrict__ x, const int32_t* __restrict__ inv,
                                                                   E* __restrict__ buf, long long rows, int H, int T,
                                                                   int zero_pad) {
    const int lane = threadIdx.x & 31;
    const long long nw = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); row < rows; row += nw) {
        const int t = inv[row];
        E* dst = buf + row * H;
        if (t < 0 || t >= T) {
            if (zero_pad) for (int j = lane; j < H; j += kWarp) dst[j] = E(0);
            continue;
        }
        const E* srcp = x + (long long)t * H;
        for (int j = lane; j < H; j += kWarp) dst[j] = srcp[j];
    }
}

// ---- combine ----
// 8 consecutive elements ("octet") as four packed float pairs.
template <int DT> struct Oct;
template <> struct Oct<LOCMOE_F32> {
    __device__ static __forceinline__ void load(const void* base, long long o, float2 (&f)[4]) {
        const uint4* p = reinterpret_cast<const uint4*>(base) + o * 2;
        uint4 a = ld_stream(p), b = ld_stream(p + 1);
        f[0] = make_float2(__uint_as_float(a.x), __uint_as_float(a.y));
        f[1] = make_float2(__uint_as_float(a.z), __uint_as_float(a.w));
        f[2] = make_float2(__uint_as_float(b.x), __uint_as_float(b.y));
        f[3] = make_float2(__uint_as_float(b.z), __uint_as_float(b.w));
    }
    __device__ static __forceinline__ void store(void* base, long long o, const float2 (&f)[4]) {
        uint4* p = reinterpret_cast<uint4*>(base) + o * 2;
        st_stream(p, make_uint4(__float_as_uint(f[0].x), __float_as_uint(f[0].y), __float_as_uint(f[1].x), __float_as_uint(f[1].y)));
        st_stream(p + 1, make_uint4(__float_as_uint(f[2].x), __float_as_uint(f[2].y), __float_as_uint(f[3].x), __float_as_uint(f[3].y)));
    }
};
template <> struct Oct<LOCMOE_BF16> {
    __device__ static __forceinline__ void load(const void* base, long long o, float2 (&f)[4]) {
        uint4 a = ld_stream(reinterpret_cast<const uint4*>(base) + o);
        f[0] = make_float2(bf16_lo(a.x), bf16_hi(a.x));
        f[1] = make_float2(bf16_lo(a.y), bf16_hi(a.y));
        f[2] = make_float2(bf16_lo(a.z), bf16_hi(a.z));
        f[3] = make_float2(bf16_lo(a.w), bf16_hi(a.w));
    }
    __device__ static __forceinline__ void store(void* base, long long o, const float2 (&f)[4]) {
        st_stream(reinterpret_cast<uint4*>(base) + o,
                  make_uint4(cvt_bf16x2(f[0]), cvt_bf16x2(f[1]), cvt_bf16x2(f[2]), cvt_bf16x2(f[3])));
    }
};

// out[t] (+)= gate_w[t] * y[slot[t]]; O = octets (8 elements) per row.
template <int YDT, int ODT, bool ACC>
__global__ void __launch_bounds__(kThreads, ACC ? 4 : 6) combine_vec_kernel(const void* __restrict__ y, const int32_t* __restrict__ slot,
                                                               const float* __restrict__ gate_w, void* __restrict__ out,
                                                               int T, int O, long long rows, int tpc) {
    pdl_wait();
    pdl_trigger();
    constexpr int CH = 2;
    const int lane = threadIdx.x & 31;
    const int nch = (O + CH * kWarp - 1) / (CH * kWarp);
    // every CTA owns a contiguous run of tpc tokens, so that the grid walks the tokens in ascending order
    const long long t_lo = (long long)blockIdx.x * tpc;
    const int t_hi = (int)min((long long)T, t_lo + tpc);
    for (int t = (int)t_lo + (threadIdx.x >> 5); t < t_hi; t += blockDim.x >> 5) {
        const int s = slot[t];
        const long long obase = (long long)t * O;
        if (s < 0 || s >= rows) {
            if (!ACC) {
                const float2 z[4] = {{0, 0}, {0, 0}, {0, 0}, {0, 0}};
                for (int o = lane; o < O; o += kWarp) Oct<ODT>::store(out, obase + o, z);
            }
            continue;
        }
        const float w = gate_w[t];
        const float2 w2 = make_float2(w, w);
        const long long ybase = (long long)s * O;
        for (int c = 0; c < nch; ++c) {
            float2 f[CH][4], prev[CH][4];
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                int o = (c * CH + k) * kWarp + lane;
                if (o < O) {
                    Oct<YDT>::load(y, ybase + o, f[k]);
                    if (ACC) Oct<ODT>::load(out, obase + o, prev[k]);
                }
            }
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                int o = (c * CH + k) * kWarp + lane;
                if (o < O) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) f[k][e] = ACC ? __ffma2_rn(w2, f[k][e], prev[k][e]) : __fmul2_rn(w2, f[k][e]);
                    Oct<ODT>::store(out, obase + o, f[k]);
                }
            }
        }
    }
}

__device__ __forceinline__ float load_elem(const void* p, long long i, int dt) {
    if (dt == LOCMOE_F32) return reinterpret_cast<const float*>(p)[i];
    return __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(p)[i]) << 16);
}
__device__ __forceinline__ void store_elem(void* p, long long i, int dt, float v) {
    if (dt == LOCMOE_F32) reinterpret_cast<float*>(p)[i] = v;
    else reinterpret_cast<uint16_t*>(p)[i] = (uint16_t)f32_to_bf16_bits(v);
}

__global__ void __launch_bounds__(kThreads) combine_scalar_kernel(const void* __restrict__ y, int ydt,
                                                                  const int32_t* __restrict__ slot,
                                                                  const float* __restrict__ gate_w, void* __restrict__ out,
                                                                  int odt, int T, int H, long long rows, int acc) {
    const int lane = threadIdx.x & 31;
    const int nw = gridDim.x * (blockDim.x >> 5);
    for (int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); t < T; t += nw) {
        const int s = slot[t];
        const long long ob = (long long)t * H;
        if (s < 0 || s >= rows) {
            if (!acc) for (int j = lane; j < H; j += kWarp) store_elem(out, ob + j, odt, 0.0f);
            continue;
        }
        const float w = gate_w[t];
        const long long yb = (long long)s * H;
        for (int j = lane; j < H; j += kWarp) {
            float v = load_elem(y, yb + j, ydt);
            v = acc ? fmaf(w, v, load_elem(out, ob + j, odt)) : w * v;
            store_elem(out, ob + j, odt, v);
        }
    }
}

// Grid of the flat kernels: about two loop iterations per thread, at most 256 CTAs per SM (measured best on B200:
// many short CTAs beat a resident-only grid by 4-5 % on these copy-like kernels).
int flat_grid(unsigned long long total, int per_thread) {
    unsigned long long want = (total + (unsigned long long)kThreads * per_thread * 2 - 1) / ((unsigned long long)kThreads * per_thread * 2);
    unsigned long long cap = 256ull * sm_count();
    if (want > cap) want = cap;
    return want < 1 ? 1 : (int)want;
}

int grid_for(long long units, int warps_per_block, int blocks_per_sm) {
    long long want = (units + warps_per_block - 1) / warps_per_block;
    long long cap = (long long)blocks_per_sm * sm_count();
    if (want > cap) want = cap;
    return want < 1 ? 1 : (int)want;
}

}  // namespace

// Bulk-copy dispatch: segments of at most 16 KB that divide the row into equal multiples of 16 bytes.
// Returns 1 when the row size does not suit it.
static int launch_dispatch_tma(const locmoe_shape_t& s, int64_t rows, size_t rb, const void* x, const int32_t* inv, void* buf,
                               int zero_pad, cudaStream_t st) {
    int nseg = (int)((rb + 16383) / 16384);
    while (nseg <= 64 && (rb % ((size_t)nseg * 16) != 0)) ++nseg;
    if (nseg > 64) return 1;
    const uint32_t seg = (uint32_t)(rb / nseg);
    int nw = (int)((220 * 1024 - seg) / (seg + 8));
    if (nw > 24) nw = 24;
    if (nw < 4) return 1;
    const size_t smem = (size_t)seg * (nw + 1) + (size_t)nw * 8;
    static bool attr_done_dev[64] = {false};   // the attribute is per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_done_dev[dev & 63]) {
        if (cudaFuncSetAttribute(dispatch_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) {
            cudaGetLastError();
            return LOCMOE_ERR_CUDA;
        }
        attr_done_dev[dev & 63] = true;
    }
    const long long want = (rows * nseg + nw - 1) / nw;
    int g = sm_count();
    if (want < g) g = (int)want;
    dispatch_tma_kernel<<<g, nw * 32, smem, st>>>(static_cast<const unsigned char*>(x), inv, static_cast<unsigned char*>(buf),
                                                  rows, nseg, seg, (long long)rb, s.T, zero_pad);
    return check_launch();
}

int launch_dispatch(const locmoe_shape_t& s, int64_t rows, const void* x, const int32_t* inv, const int32_t* slot,
                    void* buf, int zero_pad, cudaStream_t st) {
    const int esz = s.x_dtype == LOCMOE_F32 ? 4 : 2;
    const size_t rb = (size_t)s.H * esz;
    const bool vec_ok = rb % 16 == 0 && (uintptr_t)x % 16 == 0 && (uintptr_t)buf % 16 == 0;
    // 16 CTAs per SM (more, shorter CTAs than are resident measured ~4 % faster than a resident-only grid)
    const int grid = grid_for(rows, kThreads / 32, 16);
    // LOCMOE_DISPATCH = tma | vec | flat forces one of the other kernels (testing aid).  The load/store kernels are
    // the default: the bulk-copy variant measured 218 us against 213 us for the warp-per-row kernel on the
    // 65536 x 5120 bf16 case.
    const char* mode = getenv("LOCMOE_DISPATCH");
    if (vec_ok && mode && mode[0] == 't') {
        const int rc = launch_dispatch_tma(s, rows, rb, x, inv, buf, zero_pad, st);
        if (rc != 1) return rc;   // 1: the row size does not suit the bulk-copy kernel, fall through
    }
    // the token-major kernel walks all T tokens: only where the buffer can hold at least half of them (with one
    // slot per (source, expert) pair, 4096 rows for 65536 tokens, its 20480 nearly empty CTAs took 80 us; the
    // row-major kernel below walks the rows instead)
    const bool dense = (unsigned long long)rows * 2 >= (unsigned long long)s.T;
    if (vec_ok && slot && dense && !mode && (unsigned long long)s.T * (rb / 16) < 0xf0000000ull) {
        const unsigned total = (unsigned)((unsigned long long)s.T * (rb / 16));
        const unsigned per = (unsigned)(kThreads * 4 * kTokIters);
        const int g = (int)((total + per - 1) / per);
        const int zrows = (int)((rows + g - 1) / g);
        return launch_pdl(dispatch_token_kernel, g, kThreads, 0, st, static_cast<const uint4*>(x), slot, inv,
                          static_cast<uint4*>(buf), total, (unsigned)(rb / 16), s.T, (long long)rows, zero_pad, zrows);
    }
    if (vec_ok && !(mode && mode[0] == 'v') && (unsigned long long)rows * (rb / 16) < 0xffffffffull) {
        const int fg = flat_grid((unsigned long long)rows * (rb / 16), 4);
        return launch_pdl(dispatch_flat_kernel, fg, kThreads, 0, st, static_cast<const uint4*>(x), inv, static_cast<uint4*>(buf),
                          (unsigned)(rows * (rb / 16)), (unsigned)(rb / 16), s.T, zero_pad);
    }
    if (vec_ok) {
        return launch_pdl(dispatch_vec_kernel, grid, kThreads, 0, st, static_cast<const uint4*>(x), inv, static_cast<uint4*>(buf),
                          (long long)rows, (int)(rb / 16), s.T, zero_pad);
    } else if (esz == 4) {
        dispatch_scalar_kernel<uint32_t><<<grid, kThreads, 0, st>>>(static_cast<const uint32_t*>(x), inv,
                                                                    static_cast<uint32_t*>(buf), rows, s.H, s.T, zero_pad);
    } else {
        dispatch_scalar_kernel<uint16_t><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), inv,
                                                                    static_cast<uint16_t*>(buf), rows, s.H, s.T, zero_pad);
    }
    return check_launch();
}

int launch_combine(const locmoe_shape_t& s, int64_t rows, const void* y, int y_dtype, const int32_t* slot,
                   const float* gate_w, void* out, int accumulate, cudaStream_t st) {
    const bool vec_ok = s.H % 8 == 0 && (uintptr_t)y % 16 == 0 && (uintptr_t)out % 16 == 0;
    // several waves of short CTAs measured fastest (~6 %); a flat (token, octet) mapping like dispatch's measured
    // 202-204 us against 197 us for this warp-per-token kernel on the 65536 x 5120 bf16 case and was dropped
    const int grid = grid_for(s.T, kThreads / 32, 32);
    // vector kernel: one token per warp in ascending order while the grid stays below 1024 CTAs per SM
    const int cgrid = grid_for(s.T, kThreads / 32, 1024);
    const int tpc = (s.T + cgrid - 1) / cgrid;
    if (!vec_ok) {
        combine_scalar_kernel<<<grid, kThreads, 0, st>>>(y, y_dtype, slot, gate_w, out, s.x_dtype, s.T, s.H, rows,
                                                         accumulate);
        return check_launch();
    }
    const int O = s.H / 8;
#define LOCMOE_COMBINE_CASE(YD, OD, AC)                                                                              \
    if (y_dtype == YD && s.x_dtype == OD && (accumulate != 0) == AC) {                                               \
        return launch_pdl(combine_vec_kernel<YD, OD, AC>, cgrid, kThreads, 0, st, y, slot, gate_w, out, s.T, O, (long long)rows, tpc); \
                                                                                     \
    }
    LOCMOE_COMBINE_CASE(LOCMOE_F32, LOCMOE_F32, false)
    LOCMOE_COMBINE_CASE(LOCMOE_F32, LOCMOE_F32, true)
    LOCMOE_COMBINE_CASE(LOCMOE_F32, LOCMOE_BF16, false)
    LOCMOE_COMBINE_CASE(LOCMOE_F32, LOCMOE_BF16, true)
    LOCMOE_COMBINE_CASE(LOCMOE_BF16, LOCMOE_F32, false)
    LOCMOE_COMBINE_CASE(LOCMOE_BF16, LOCMOE_F32, true)
    LOCMOE_COMBINE_CASE(LOCMOE_BF16, LOCMOE_BF16, false)
    LOCMOE_COMBINE_CASE(LOCMOE_BF16, LOCMOE_BF16, true)
#undef LOCMOE_COMBINE_CASE
    return LOCMOE_ERR_DTYPE;
}

int read_device_flags(int* out, cudaStream_t st) {
    if (cudaMemcpyFromSymbolAsync(out, g_device_flags, sizeof(int), 0, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    return LOCMOE_OK;
}

}  // namespace locmoe
