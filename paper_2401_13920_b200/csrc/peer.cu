// Dispatch and combine fused with the All-to-All around the experts (Sec. 3.2.4), one process per GPU.
//
// Every rank owns a contiguous block of the logical devices, routes the tokens of its own source devices in the
// receive-side layout of the WHOLE logical map (row = (e * D + r(dev(e), src)) * C + pos), and
//   dispatch: stores each kept token's row straight into the receive buffer of the GPU that hosts expert e
//             (plain 16-byte stores through a peer pointer: NVLink / NVSwitch on a multi-GPU node) and zero-fills
//             the empty rows that belong to its own source devices;
//   combine : loads the expert output row from that GPU's buffer (plain peer loads) and scales it.
// The send-side buffer and the library All-to-All disappear: a row crosses the link once, as it is produced.
// Experts are split evenly, so rank q's buffer holds the rows [q * rows_per_peer, (q + 1) * rows_per_peer).
// A call may be restricted to a window of every owner's buffer (rows [win_lo, win_hi) inside each peer's slice): the
// receive buffer can then be filled expert slice by expert slice while the experts of the slices already filled run.
// No kernel waits on another GPU; the caller separates dispatch, expert FFN and combine with a barrier across
// the ranks (all stores of a kernel are visible to the peers once its stream has been synchronised).
// Plain loads and stores only: no bulk-copy engine, no multicast.
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kThreads = 256;
constexpr int kIters = 2;
constexpr int kMaxPeers = 64;

struct PeerTable {
    uint4* base[kMaxPeers];
};

// Source device of global receive-layout row `row` (cell = row / C = e * D + r(dev(e), src)).
__device__ __forceinline__ int row_source(long long row, int C, int D, int Ed, int N, int Dn) {
    const long long cell = row / C;
    const int e = (int)(cell / D), rho = (int)(cell - (long long)e * D);
    const int a = e / Ed;
    return (((a / Dn) + rho / Dn) % N) * Dn + ((a % Dn) + rho % Dn) % Dn;
}

// Token-major copy in descending token order (as the single-GPU dispatch) into the owners' buffers, then the
// zero-fill of this rank's empty rows.
__global__ void __launch_bounds__(kThreads) dispatch_peer_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ slot,
                                                                 const int32_t* __restrict__ inv, const PeerTable peers,
                                                                 long long rows_per_peer, unsigned total, unsigned V, int T,
                                                                 long long rows, int zero_pad, int zrows, int C, int D, int Ed,
                                                                 int N, int Dn, int src_lo, int src_hi, long long win_lo,
                                                                 long long win_hi) {
    const unsigned base = blockIdx.x * (unsigned)(kThreads * 4 * kIters);
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        uint4 r[4];
        uint4* dst[4];
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
                    const int q = (int)(row / rows_per_peer);
                    const long long lr = row - q * rows_per_peer;      // row inside the owner's buffer
                    if (lr >= win_lo && lr < win_hi) {
                        r[k] = ld_stream(x + (size_t)t * V + v);
                        dst[k] = peers.base[q] + (size_t)lr * V + v;
                        st[k] = true;
                    }
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (st[k]) st_stream(dst[k], r[k]);
    }
    if (zero_pad) {
        const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
        for (int i = w; i < zrows; i += kThreads / 32) {
            const long long row = (long long)blockIdx.x * zrows + i;
            if (row >= rows) break;
            const int t = __ldg(inv + row);
            if (t >= 0 && t < T) continue;
            const int s = row_source(row, C, D, Ed, N, Dn);
            if (s < src_lo || s >= src_hi) continue;   // another rank's row
            const int q = (int)(row / rows_per_peer);
            const long long lr = row - q * rows_per_peer;
            if (lr < win_lo || lr >= win_hi) continue;         // outside the window of this call
            uint4* d = peers.base[q] + (size_t)lr * V;
            for (unsigned v = lane; v < V; v += 32) st_stream(d + v, make_uint4(0, 0, 0, 0));
        }
    }
}

// out[t] = gate_w[t] * y[slot[t]] with y spread over the peers' buffers; bf16 or fp32 rows, 16-byte vectors.
template <int YDT, int ODT>
__global__ void __launch_bounds__(kThreads) combine_peer_kernel(const PeerTable peers, long long rows_per_peer,
                                                                const int32_t* __restrict__ slot,
                                                                const float* __restrict__ gate_w, void* __restrict__ out,
                                                                int T, int O, long long rows, int tpc) {
    constexpr int YV = YDT == LOCMOE_F32 ? 2 : 1, OV = ODT == LOCMOE_F32 ? 2 : 1;   // 16-byte vectors per octet
    const int lane = threadIdx.x & 31;
    const long long t_lo = (long long)blockIdx.x * tpc;
    const int t_hi = (int)min((long long)T, t_lo + tpc);
    for (int t = (int)t_lo + (threadIdx.x >> 5); t < t_hi; t += kThreads / 32) {
        const int s = slot[t];
        uint4* orow = reinterpret_cast<uint4*>(out) + (size_t)t * O * OV;
        if (s < 0 || s >= rows) {
            for (int o = lane; o < O * OV; o += 32) st_stream(orow + o, make_uint4(0, 0, 0, 0));
            continue;
        }
        const int q = (int)(s / rows_per_peer);
        const uint4* yrow = peers.base[q] + (size_t)(s - q * rows_per_peer) * O * YV;
        const float w = gate_w[t];
        // two octets per lane in flight
        for (int o0 = lane; o0 < O; o0 += 64) {
            uint4 raw[2][2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int o = o0 + 32 * h;
                if (o < O) {
                    if (YDT == LOCMOE_F32) { raw[h][0] = ld_stream(yrow + 2 * o); raw[h][1] = ld_stream(yrow + 2 * o + 1); }
                    else raw[h][0] = ld_stream(yrow + o);
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int o = o0 + 32 * h;
                if (o >= O) continue;
                float f[8];
                if (YDT == LOCMOE_F32) {
                    const uint4 a = raw[h][0], b = raw[h][1];
                    f[0] = __uint_as_float(a.x); f[1] = __uint_as_float(a.y); f[2] = __uint_as_float(a.z); f[3] = __uint_as_float(a.w);
                    f[4] = __uint_as_float(b.x); f[5] = __uint_as_float(b.y); f[6] = __uint_as_float(b.z); f[7] = __uint_as_float(b.w);
                } else {
                    const uint4 a = raw[h][0];
                    f[0] = bf16_lo(a.x); f[1] = bf16_hi(a.x); f[2] = bf16_lo(a.y); f[3] = bf16_hi(a.y);
                    f[4] = bf16_lo(a.z); f[5] = bf16_hi(a.z); f[6] = bf16_lo(a.w); f[7] = bf16_hi(a.w);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) f[k] = __fmul_rn(w, f[k]);
                if (ODT == LOCMOE_F32) {
                    st_stream(orow + 2 * o, make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3])));
                    st_stream(orow + 2 * o + 1, make_uint4(__float_as_uint(f[4]), __float_as_uint(f[5]), __float_as_uint(f[6]), __float_as_uint(f[7])));
                } else {
                    st_stream(orow + o, make_uint4(cvt_bf16x2(make_float2(f[0], f[1])), cvt_bf16x2(make_float2(f[2], f[3])),
                                                   cvt_bf16x2(make_float2(f[4], f[5])), cvt_bf16x2(make_float2(f[6], f[7]))));
                }
            }
        }
    }
}

}  // namespace

int launch_dispatch_peer(const locmoe_shape_t& s, int C_alloc, int64_t rows, const void* x, const int32_t* inv,
                         const int32_t* slot, void* const* peer_bufs, int n_peers, int src_lo, int src_hi, int zero_pad,
                         long long win_lo, long long win_hi, cudaStream_t st) {
    PeerTable pt{};
    for (int q = 0; q < n_peers; ++q) pt.base[q] = static_cast<uint4*>(peer_bufs[q]);
    const int esz = s.x_dtype == LOCMOE_F32 ? 4 : 2;
    const size_t rb = (size_t)s.H * esz;
    const unsigned V = (unsigned)(rb / 16);
    const unsigned total = (unsigned)((unsigned long long)s.T * V);
    const unsigned per = (unsigned)(kThreads * 4 * kIters);
    int g = (int)((total + per - 1) / per);
    if (g < 1) g = 1;
    const int zrows = (int)((rows + g - 1) / g);
    const int D = s.n_nodes * s.dev_per_node;
    dispatch_peer_kernel<<<g, kThreads, 0, st>>>(static_cast<const uint4*>(x), slot, inv, pt, (long long)(rows / n_peers), total,
                                                 V, s.T, (long long)rows, zero_pad, zrows, C_alloc, D, s.E / D, s.n_nodes,
                                                 s.dev_per_node, src_lo, src_hi, win_lo, win_hi);
    return check_launch();
}

int launch_combine_peer(const locmoe_shape_t& s, int64_t rows, void* const* peer_y, int n_peers, int y_dtype,
                        const int32_t* slot, const float* gate_w, void* out, cudaStream_t st) {
    PeerTable pt{};
    for (int q = 0; q < n_peers; ++q) pt.base[q] = static_cast<uint4*>(peer_y[q]);
    long long want = ((long long)s.T + 7) / 8, cap = 1024ll * sm_count();
    const int grid = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    const int tpc = (s.T + grid - 1) / grid;
    const int O = s.H / 8;
    const long long rpp = rows / n_peers;
    if (y_dtype == LOCMOE_F32 && s.x_dtype == LOCMOE_F32)
        combine_peer_kernel<LOCMOE_F32, LOCMOE_F32><<<grid, kThreads, 0, st>>>(pt, rpp, slot, gate_w, out, s.T, O, rows, tpc);
    else if (y_dtype == LOCMOE_F32)
        combine_peer_kernel<LOCMOE_F32, LOCMOE_BF16><<<grid, kThreads, 0, st>>>(pt, rpp, slot, gate_w, out, s.T, O, rows, tpc);
    else if (s.x_dtype == LOCMOE_F32)
        combine_peer_kernel<LOCMOE_BF16, LOCMOE_F32><<<grid, kThreads, 0, st>>>(pt, rpp, slot, gate_w, out, s.T, O, rows, tpc);
    else
        combine_peer_kernel<LOCMOE_BF16, LOCMOE_BF16><<<grid, kThreads, 0, st>>>(pt, rpp, slot, gate_w, out, s.T, O, rows, tpc);
    return check_launch();
}

}  // namespace locmoe
