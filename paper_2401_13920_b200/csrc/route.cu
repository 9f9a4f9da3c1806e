// Capacity-bounded routing (Sec. 3.2.3 capacity limit, Sec. 3.2.4 exchange layout).
//
// pos[t] -- the number of earlier tokens with the same (source device, expert)
// pair -- is the rank of t inside its key class in token order.  It is
// obtained with a stable least-significant-digit radix sort of the keys
// key = src * E + expert: per pass a per-tile digit histogram, one exclusive
// scan over (digit, tile), and a stable in-tile ranking that uses warp match
// operations and per-warp digit counters.  A token's final sorted position
// minus the start of its key class is pos.  Every step is integer and order
// independent, so the result is a function of the inputs only; no kernel waits
// on another CTA.
//
// Launch sequence (P radix passes, P = 1 for up to 1024 keys, 2 up to 65536):
//   init -> [hist_p -> scan_p -> scatter_p] for p = 0..P-1
// scan_0 also turns the per-key demand counts into key-class starts and the
// count matrices (kept, send_counts, load, locality tallies).
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxRounds = 16;
constexpr int kScanThreads = 1024;

struct RouteArgs {
    const int32_t* idx;
    const int32_t* src;
    const locmoe_capacity_t* cap;
    int32_t C_alloc;
    int32_t* pos; int32_t* slot; uint8_t* drop; int32_t* inv;
    int32_t* counts; int32_t* kept; int32_t* send_counts; int32_t* load;
    unsigned long long* locality;
    int32_t* status;
    int T, E, N, Dn, D, Ed, K, layout;
    long long rows;
    int tile, rounds, ntiles;
    uint32_t* keys[2];
    int32_t* toks[2];
    int32_t* hist;       // [nbins][ntiles], digit major
    int32_t* keystart;   // [K]
    int32_t* n_valid;    // items that survive pass 0
};

__device__ __forceinline__ int dest_rank(int a, int b, int N, int Dn) {
    int dn = b / Dn - a / Dn; if (dn < 0) dn += N;
    int dl = b % Dn - a % Dn; if (dl < 0) dl += Dn;
    return dn * Dn + dl;
}

__global__ void __launch_bounds__(kThreads) route_init_kernel(const RouteArgs a) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (long long i = i0; i < a.rows; i += stride) a.inv[i] = -1;
    for (long long i = i0; i < a.K; i += stride) a.counts[i] = 0;
    for (long long i = i0; i < (long long)a.D * a.D; i += stride) a.send_counts[i] = 0;
    for (long long i = i0; i < a.E; i += stride) a.load[i] = 0;
    if (i0 < 6) a.locality[i0] = 0ull;
    if (i0 == 0) *a.status = 0;
}

// Key of token t, or -1 with a warning bit when the token cannot be routed.
__device__ __forceinline__ int token_key(const RouteArgs& a, int t, int* warn) {
    int e = a.idx[t], s = a.src[t];
    if (s < 0 || s >= a.D) { *warn |= LOCMOE_WARN_BAD_SRC; return -1; }
    if (e < 0 || e >= a.E) { *warn |= LOCMOE_WARN_BAD_IDX; return -1; }
    return s * a.E + e;
}

template <bool FIRST>
__global__ void __launch_bounds__(kThreads) route_hist_kernel(const RouteArgs a, int pass, int shift, int nbins) {
    extern __shared__ int sh[];
    for (int d = threadIdx.x; d < nbins; d += blockDim.x) sh[d] = 0;
    __syncthreads();
    const int n = FIRST ? a.T : *a.n_valid;
    const int base = blockIdx.x * a.tile;
    const uint32_t mask = (uint32_t)nbins - 1u;
    const uint32_t* kin = a.keys[(pass + 1) & 1];
    int warn = 0;
    for (int o = threadIdx.x; o < a.tile; o += blockDim.x) {
        int j = base + o;
        if (j >= n) break;
        int key;
        if (FIRST) {
            key = token_key(a, j, &warn);
            if (key < 0) continue;
            atomicAdd(&a.counts[key], 1);
        } else {
            key = (int)kin[j];
        }
        atomicAdd(&sh[((uint32_t)key >> shift) & mask], 1);
    }
    if (FIRST && warn) atomicOr(a.status, warn);
    __syncthreads();
    for (int d = threadIdx.x; d < nbins; d += blockDim.x) a.hist[(size_t)d * a.ntiles + blockIdx.x] = sh[d];
}

// In-place exclusive scan of data[0..n) by one CTA; returns the total in *total (if given).
__device__ void block_exclusive_scan(const int32_t* in, int32_t* out, int n, int32_t* total) {
    __shared__ int warp_sums[kScanThreads / 32];
    __shared__ int carry_all;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int chunk = (n + kScanThreads - 1) / kScanThreads;
    const int lo = min(tid * chunk, n), hi = min(lo + chunk, n);
    int s = 0;
    for (int i = lo; i < hi; ++i) s += in[i];
    int incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[w] = incl;
    __syncthreads();
    if (w == 0) {
        int v = warp_sums[lane];
        int iv = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_up_sync(0xffffffffu, iv, o);
            if (lane >= o) iv += u;
        }
        warp_sums[lane] = iv - v;
        if (lane == 31) carry_all = iv;
    }
    __syncthreads();
    int run = warp_sums[w] + incl - s;
    for (int i = lo; i < hi; ++i) { int v = in[i]; out[i] = run; run += v; }
    if (total && tid == 0) *total = carry_all;
}

// Block 0: offsets for this pass.  With with_stats: block 1 builds the key-class
// starts, blocks >= 2 the count matrices.
__global__ void __launch_bounds__(kScanThreads) route_scan_kernel(const RouteArgs a, int nbins, int with_stats) {
    if (blockIdx.x == 0) {
        block_exclusive_scan(a.hist, a.hist, nbins * a.ntiles, with_stats ? a.n_valid : nullptr);
        return;
    }
    if (blockIdx.x == 1) {
        block_exclusive_scan(a.counts, a.keystart, a.K, nullptr);
        return;
    }
    int C = a.cap->C_local;
    if (C > a.C_alloc) {
        C = a.C_alloc;
        if (blockIdx.x == 2 && threadIdx.x == 0) atomicOr(a.status, LOCMOE_WARN_CLAMPED);
    }
    unsigned long long raw0 = 0, raw1 = 0, raw2 = 0, kp0 = 0, kp1 = 0, kp2 = 0;
    for (int k = (blockIdx.x - 2) * blockDim.x + threadIdx.x; k < a.K; k += (gridDim.x - 2) * blockDim.x) {
        int c = a.counts[k];
        int kp = c < C ? c : C;
        a.kept[k] = kp;
        if (c == 0) continue;
        int s = k / a.E, e = k - s * a.E, b = e / a.Ed;
        if (b == s) { raw0 += c; kp0 += kp; }
        else if (b / a.Dn == s / a.Dn) { raw1 += c; kp1 += kp; }
        else { raw2 += c; kp2 += kp; }
        atomicAdd(&a.load[e], c);
        if (kp) atomicAdd(&a.send_counts[s * a.D + b], kp);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        raw0 += __shfl_xor_sync(0xffffffffu, raw0, o); raw1 += __shfl_xor_sync(0xffffffffu, raw1, o);
        raw2 += __shfl_xor_sync(0xffffffffu, raw2, o); kp0 += __shfl_xor_sync(0xffffffffu, kp0, o);
        kp1 += __shfl_xor_sync(0xffffffffu, kp1, o); kp2 += __shfl_xor_sync(0xffffffffu, kp2, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (raw0) atomicAdd(&a.locality[0], raw0);
        if (raw1) atomicAdd(&a.locality[1], raw1);
        if (raw2) atomicAdd(&a.locality[2], raw2);
        if (kp0) atomicAdd(&a.locality[3], kp0);
        if (kp1) atomicAdd(&a.locality[4], kp1);
        if (kp2) atomicAdd(&a.locality[5], kp2);
    }
}

template <bool FIRST, bool LAST>
__global__ void __launch_bounds__(kThreads) route_scatter_kernel(const RouteArgs a, int pass, int shift, int nbins) {
    extern __shared__ int cnt[];  // [kWarps][nbins]
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kWarps * nbins; i += blockDim.x) cnt[i] = 0;
    __syncthreads();

    const int n = FIRST ? a.T : *a.n_valid;
    const uint32_t mask = (uint32_t)nbins - 1u;
    const uint32_t* kin = a.keys[(pass + 1) & 1];
    const int32_t* tin = a.toks[(pass + 1) & 1];
    uint32_t* kout = a.keys[pass & 1];
    int32_t* tout = a.toks[pass & 1];
    const int wbase = blockIdx.x * a.tile + w * a.rounds * 32;
    const uint32_t lt = (1u << lane) - 1u;
    int* mycnt = cnt + w * nbins;

    int key[kMaxRounds], tok[kMaxRounds], rank[kMaxRounds];
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
        key[r] = -1; tok[r] = -1; rank[r] = 0;
        if (r < a.rounds) {
            int j = wbase + r * 32 + lane;
            if (j < n) {
                if (FIRST) {
                    int warn = 0;
                    tok[r] = j;
                    key[r] = token_key(a, j, &warn);
                    if (key[r] < 0) { a.pos[j] = -1; a.slot[j] = -1; a.drop[j] = 1; }
                } else {
                    key[r] = (int)kin[j];
                    tok[r] = tin[j];
                }
            }
            const bool valid = key[r] >= 0;
            const uint32_t d = valid ? (((uint32_t)key[r] >> shift) & mask) : 0xffffffffu;
            const uint32_t peers = __match_any_sync(0xffffffffu, d);
            int before = 0;
            if (valid) before = mycnt[d];
            __syncwarp();
            if (valid) {
                rank[r] = before + __popc(peers & lt);
                if ((peers & lt) == 0) mycnt[d] = before + __popc(peers);
            }
            __syncwarp();
        }
    }
    __syncthreads();
    // counters -> starting offsets: global (digit, tile) offset plus the earlier warps of this tile
    for (int d = threadIdx.x; d < nbins; d += blockDim.x) {
        int run = a.hist[(size_t)d * a.ntiles + blockIdx.x];
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) {
            int c = cnt[ww * nbins + d];
            cnt[ww * nbins + d] = run;
            run += c;
        }
    }
    __syncthreads();

    int C = 0;
    if (LAST) { C = a.cap->C_local; if (C > a.C_alloc) C = a.C_alloc; }
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
        if (r < a.rounds && key[r] >= 0) {
            const uint32_t d = ((uint32_t)key[r] >> shift) & mask;
            const int dest = mycnt[d] + rank[r];
            if (!LAST) {
                kout[dest] = (uint32_t)key[r];
                tout[dest] = tok[r];
            } else {
                const int k = key[r], t = tok[r];
                const int p = dest - a.keystart[k];
                const bool dropped = p >= C;
                a.pos[t] = p;
                a.drop[t] = dropped ? 1 : 0;
                int row = -1;
                if (!dropped) {
                    const int s = k / a.E, e = k - s * a.E;
                    const int b = e / a.Ed, el = e - b * a.Ed;
                    long long rr;
                    if (a.layout == LOCMOE_LAYOUT_SEND)
                        rr = (((long long)s * a.D + dest_rank(s, b, a.N, a.Dn)) * a.Ed + el) * a.C_alloc + p;
                    else
                        rr = ((long long)e * a.D + dest_rank(b, s, a.N, a.Dn)) * a.C_alloc + p;
                    row = (int)rr;
                    a.inv[row] = t;
                }
                a.slot[t] = row;
            }
        }
    }
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

int plan_route(const locmoe_shape_t& s, RoutePlan* p) {
    const long long K = (long long)s.n_nodes * s.dev_per_node * s.E;
    if (K < 1 || K > 0x7fffffffll) return LOCMOE_ERR_SHAPE;
    int kb = 1;
    while ((1ll << kb) < K) ++kb;
    p->key_bits = kb;
    p->passes = kb <= 10 ? 1 : (kb + 7) / 8;
    int left = kb;
    for (int i = 0; i < 4; ++i) p->bits[i] = 0;
    for (int i = 0; i < p->passes; ++i) {
        int b = (left + (p->passes - i) - 1) / (p->passes - i);
        p->bits[i] = b;
        left -= b;
    }
    int rounds = (int)(((long long)s.T + 65535) / 65536);
    if (rounds < 2) rounds = 2;
    if (rounds > kMaxRounds) rounds = kMaxRounds;
    p->rounds = rounds;
    p->tile = kWarps * rounds * 32;
    p->ntiles = (int)(((long long)s.T + p->tile - 1) / p->tile);
    int maxbins = 1 << p->bits[0];
    size_t off = 0;
    for (int i = 0; i < 2; ++i) {
        p->off_keys[i] = off; off += p->passes > 1 ? align256((size_t)s.T * 4) : 0;
        p->off_toks[i] = off; off += p->passes > 1 ? align256((size_t)s.T * 4) : 0;
    }
    p->off_hist = off; off += align256((size_t)maxbins * p->ntiles * 4 + 4);
    p->off_keystart = off; off += align256((size_t)K * 4);
    p->total = off;
    return LOCMOE_OK;
}

int launch_route(const locmoe_shape_t& s, const int32_t* idx, const int32_t* src, const locmoe_capacity_t* cap_dev,
                 int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                 int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                 void* ws, cudaStream_t st) {
    RoutePlan p;
    int rc = plan_route(s, &p);
    if (rc) return rc;
    RouteArgs a{};
    a.idx = idx; a.src = src; a.cap = cap_dev; a.C_alloc = C_alloc;
    a.pos = pos; a.slot = slot; a.drop = drop; a.inv = inv;
    a.counts = counts; a.kept = kept; a.send_counts = send_counts; a.load = load;
    a.locality = reinterpret_cast<unsigned long long*>(locality);
    a.status = status;
    a.T = s.T; a.E = s.E; a.N = s.n_nodes; a.Dn = s.dev_per_node; a.D = a.N * a.Dn; a.Ed = a.E / a.D;
    a.K = a.D * a.E; a.layout = s.layout;
    a.rows = (long long)a.K * C_alloc;
    a.tile = p.tile; a.rounds = p.rounds; a.ntiles = p.ntiles;
    char* w = static_cast<char*>(ws);
    for (int i = 0; i < 2; ++i) {
        a.keys[i] = reinterpret_cast<uint32_t*>(w + p.off_keys[i]);
        a.toks[i] = reinterpret_cast<int32_t*>(w + p.off_toks[i]);
    }
    a.hist = reinterpret_cast<int32_t*>(w + p.off_hist);
    a.n_valid = a.hist + (size_t)(1 << p.bits[0]) * p.ntiles;
    a.keystart = reinterpret_cast<int32_t*>(w + p.off_keystart);

    long long init_items = a.rows > a.K ? a.rows : a.K;
    int init_blocks = (int)((init_items + kThreads * 4 - 1) / (kThreads * 4));
    if (init_blocks > 4 * sm_count()) init_blocks = 4 * sm_count();
    if (init_blocks < 1) init_blocks = 1;
    route_init_kernel<<<init_blocks, kThreads, 0, st>>>(a);
    if ((rc = check_launch())) return rc;

    int stats_blocks = (a.K + kScanThreads - 1) / kScanThreads;
    if (stats_blocks > 64) stats_blocks = 64;
    int shift = 0;
    for (int pass = 0; pass < p.passes; ++pass) {
        const int nbins = 1 << p.bits[pass];
        const bool first = pass == 0, last = pass == p.passes - 1;
        if (first) route_hist_kernel<true><<<p.ntiles, kThreads, nbins * sizeof(int), st>>>(a, pass, shift, nbins);
        else route_hist_kernel<false><<<p.ntiles, kThreads, nbins * sizeof(int), st>>>(a, pass, shift, nbins);
        if ((rc = check_launch())) return rc;
        route_scan_kernel<<<first ? 2 + stats_blocks : 1, kScanThreads, 0, st>>>(a, nbins, first ? 1 : 0);
        if ((rc = check_launch())) return rc;
        const size_t sm = (size_t)kWarps * nbins * sizeof(int);
        if (first && last) route_scatter_kernel<true, true><<<p.ntiles, kThreads, sm, st>>>(a, pass, shift, nbins);
        else if (first) route_scatter_kernel<true, false><<<p.ntiles, kThreads, sm, st>>>(a, pass, shift, nbins);
        else if (last) route_scatter_kernel<false, true><<<p.ntiles, kThreads, sm, st>>>(a, pass, shift, nbins);
        else route_scatter_kernel<false, false><<<p.ntiles, kThreads, sm, st>>>(a, pass, shift, nbins);
        if ((rc = check_launch())) return rc;
        shift += p.bits[pass];
    }
    return LOCMOE_OK;
}

}  // namespace locmoe
