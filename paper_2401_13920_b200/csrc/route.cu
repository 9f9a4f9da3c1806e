// Capacity-bounded routing (Sec. 3.2.3 capacity limit, Sec. 3.2.4 exchange layout).
//
// pos[t] -- the number of earlier tokens with the same (source device, expert)
// pair -- is the rank of t inside its key class in token order.  It is
// obtained with a stable least-significant-digit radix sort of the keys
// key = src * E + expert.  A token's final sorted position minus the start of
// its key class is pos.  Every step is integer and order independent, so the
// result is a function of the inputs only; no kernel waits on another CTA.
//
// Launch sequence for P radix passes of at most 8 bits (P = 1 up to 256 keys, 2 up to 65536):
//   init      inv = -1, accumulators and later-pass histograms = 0
//   hist0     per-tile histogram of digit 0, per-key demand counts
//   scatter_p every CTA derives its own (digit, tile) offsets from the
//             histogram matrix (no separate scan launch), ranks its tile stably
//             with warp match operations and per-warp digit counters, moves
//             (key, token) to the sorted position and adds to the next pass's
//             histogram with integer atomics; the last pass emits the outputs.
//   extras    ride on the scatters as extra CTAs: key-class starts and first buffer rows (no capacity needed) on
//             the first scatter -- a launch of their own before the only scatter when P = 1 --, the count
//             matrices (kept, send_counts, load, locality tallies), which need the capacity, on the last one.
//   prescan   large batches only: one launch per pass that prefix-scans the histogram matrix along the tiles.
// In the fused call (locmoe_capacity_route) the capacity stage has no launch of its own: hist0 also takes the
// per-expert minima of the cosines of its tile, and one more extra CTA of the first scatter combines them and
// evaluates the capacity rule; the last scatter reads the record.
#include <stdlib.h>

#include "capacity_finish.cuh"
#include "common.cuh"

namespace locmoe {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxRounds = 16;
constexpr int kMaxPasses = 4;

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
    int tile, rounds, ntiles, passes;
    int bits[kMaxPasses];
    uint32_t* keys[2];
    int32_t* toks[2];
    int32_t* hist[kMaxPasses];  // [1 << bits[p]][hstride], digit major
    int32_t* counts_rep;        // [nrep][K] replicas of the demand counters (nrep > 1), summed into counts by the extras
    int nrep;
    int32_t* keystart;          // [K]
    int32_t* rowbase;           // [K] first buffer row of the key's class
    int hstride, tile_shift;    // row stride of the histogram matrices (a multiple of 4 >= ntiles); log2(tile)
    int32_t* rowtot;            // [256] per-digit totals of the pass being scattered (prescan mode)
    int prescan;                // 1: a prescan launch turned hist[p] into exclusive prefixes along the tiles
    // capacity carried along (the fused call): hist0 also takes the per-expert minima of the cosines per tile,
    // an extra CTA of the first scatter combines them and writes the capacity record the last scatter reads
    int fuse_cap, H;
    int hist_by_gate;           // the gate kernel has already taken hist[0], counts and the minima
    int cap_sets;               // rows of cap_part: tiles (hist0 took the minima) or the gate's replica count
    double lnbeta;              // ln B(1/2, (H-1)/2), from the host
    const float* cos;
    uint32_t* cap_part;         // [ntiles][E] order-preserving codes
    locmoe_capacity_rule_t rule;
    float* delta_e;
    float* theta_e;
    locmoe_capacity_t* cap_out;
};

// Row base (in units of C_alloc rows) of key k = s * E + e in the chosen layout.
__device__ __forceinline__ long long route_row_base(const RouteArgs& a, int k) {
    const int s = k / a.E, e = k - s * a.E;
    const int b = e / a.Ed, el = e - b * a.Ed;
    if (a.layout == LOCMOE_LAYOUT_SEND) return ((long long)s * a.D + dest_order(s, b, a.N, a.Dn)) * a.Ed + el;
    return (long long)e * a.D + dest_order(b, s, a.N, a.Dn);
}

// early != 0: nothing this kernel writes is touched by the kernel queued before it (the caller says so), so the
// fill runs while that kernel drains and the wait comes last -- it must still come, so that this kernel's
// completion implies its predecessor's for the kernels after it.
__global__ void __launch_bounds__(kThreads) route_init_kernel(const RouteArgs a, int early) {
    if (!early) pdl_wait();
    pdl_trigger();
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (long long i = i0; i < a.rows; i += stride) a.inv[i] = -1;
    for (long long i = i0; i < a.K; i += stride) a.counts[i] = 0;
    if (a.nrep > 1)
        for (long long i = i0; i < (long long)a.nrep * a.K; i += stride) a.counts_rep[i] = 0;
    for (long long i = i0; i < (long long)a.D * a.D; i += stride) a.send_counts[i] = 0;
    for (long long i = i0; i < a.E; i += stride) a.load[i] = 0;
    for (int p = a.hist_by_gate ? 0 : 1; p < a.passes; ++p) {
        const long long n = ((long long)a.hstride) << a.bits[p];
        for (long long i = i0; i < n; i += stride) a.hist[p][i] = 0;
    }
    if (a.hist_by_gate)
        for (long long i = i0; i < (long long)a.cap_sets * a.E; i += stride) a.cap_part[i] = 0xffffffffu;
    if (i0 < 6) a.locality[i0] = 0ull;
    if (i0 == 0) *a.status = 0;
    if (early) pdl_wait();
}

__global__ void __launch_bounds__(kThreads) route_hist0_kernel(const RouteArgs a) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ int sh[];
    const int nbins = 1 << a.bits[0];
    uint32_t* smin = reinterpret_cast<uint32_t*>(sh + nbins);   // [E] minima of this tile (fused capacity only)
    for (int d = threadIdx.x; d < nbins; d += blockDim.x) sh[d] = 0;
    if (a.fuse_cap)
        for (int e = threadIdx.x; e < a.E; e += blockDim.x) smin[e] = 0xffffffffu;
    __syncthreads();
    const int base = blockIdx.x * a.tile;
    const uint32_t mask = (uint32_t)nbins - 1u;
    int warn = 0;
    constexpr int kU = 4;   // tokens in flight per thread
    for (int o0 = threadIdx.x; o0 < a.tile; o0 += kU * kThreads) {
        int e[kU], sd[kU];
        float cv[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int o = o0 + u * kThreads, t = base + o;
            e[u] = 0; sd[u] = 0; cv[u] = 0.0f;
            if (o < a.tile && t < a.T) {
                e[u] = a.idx[t]; sd[u] = a.src[t];
                if (a.fuse_cap) cv[u] = a.cos[t];
            }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int o = o0 + u * kThreads, t = base + o;
            if (o >= a.tile || t >= a.T) continue;
            const bool bad_s = (unsigned)sd[u] >= (unsigned)a.D, bad_e = (unsigned)e[u] >= (unsigned)a.E;
            if (a.fuse_cap && !bad_e) atomicMin(&smin[e[u]], order_code(cv[u]));
            if (bad_s || bad_e) {
                warn |= bad_s ? LOCMOE_WARN_BAD_SRC : LOCMOE_WARN_BAD_IDX;
                a.pos[t] = -1; a.slot[t] = -1; a.drop[t] = 1;
                continue;
            }
            const int key = sd[u] * a.E + e[u];
            // few keys mean many adds per address (64 per key with 1024 keys and 65536 tokens, 3 us of serialised L2
            // atomics): the tiles spread theirs over nrep copies, which the first extra CTA adds up
            if (a.nrep > 1) atomicAdd(&a.counts_rep[(size_t)(blockIdx.x & (a.nrep - 1)) * a.K + key], 1);
            else atomicAdd(&a.counts[key], 1);
            atomicAdd(&sh[(uint32_t)key & mask], 1);
        }
    }
    if (warn) atomicOr(a.status, warn);
    __syncthreads();
    for (int d = threadIdx.x; d < nbins; d += blockDim.x) a.hist[0][(size_t)d * a.hstride + blockIdx.x] = sh[d];
    if (a.fuse_cap)
        for (int e = threadIdx.x; e < a.E; e += blockDim.x) a.cap_part[(size_t)blockIdx.x * a.E + e] = smin[e];
}

// Exclusive scan of in[0..n) into out[0..n) by one CTA of kThreads threads (in == out allowed).  Every warp owns a
// contiguous eighth of the array and walks it in coalesced 32-element tiles (first to total it, then to write the
// running prefix), so that the single CTA streams the array instead of chasing per-thread chunks.
__device__ void block_exclusive_scan(const int32_t* in, int32_t* out, int n) {
    __shared__ int warp_sums[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int per = ((n + kWarps - 1) / kWarps + 31) & ~31;   // multiple of 32 per warp
    const int lo = min(w * per, n), hi = min(lo + per, n);
    int s = 0;
    for (int i = lo + lane; i < hi; i += 32) s += in[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) warp_sums[w] = s;
    __syncthreads();
    int run = 0;
#pragma unroll
    for (int ww = 0; ww < kWarps; ++ww) if (ww < w) run += warp_sums[ww];
    for (int i0 = lo; i0 < hi; i0 += 128) {
        int v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { const int i = i0 + q * 32 + lane; v[q] = i < hi ? in[i] : 0; }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int incl = v[q];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += u;
            }
            const int i = i0 + q * 32 + lane;
            if (i < hi) out[i] = run + incl - v[q];
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    __syncthreads();
}

// Extra CTAs of the first scatter (index x = 0, 1, ... of nx), none of which needs the capacity: x = 0 builds the
// key-class starts, the next ones the first buffer row of every class; in the fused call the last one combines the
// per-tile minima and evaluates the capacity rule (dyn = the CTA's dynamic shared memory, at least E words).
__device__ void route_extras_a(const RouteArgs& a, int x, int nx, int* dyn) {
    if (x == 0) {
        if (a.nrep > 1 && !a.hist_by_gate) {   // the replicas' sums are the demand counts
            for (int k = threadIdx.x; k < a.K; k += kThreads) {
                int c = 0;
                for (int r = 0; r < a.nrep; ++r) c += __ldcg(a.counts_rep + (size_t)r * a.K + k);
                a.counts[k] = c;
            }
            __syncthreads();
        }
        block_exclusive_scan(a.counts, a.keystart, a.K);
        return;
    }
    if (a.fuse_cap && x == nx - 1) {
        __shared__ FinishShared fs;
        if (a.cap_sets == 1) {   // one row of minima, taken by the gate kernel with global atomics
            capacity_finish<true>(fs, a.cap_part, 1, a.T, a.E, a.H, a.D, a.lnbeta, a.rule, a.delta_e, a.theta_e, a.cap_out);
            return;
        }
        uint32_t* comb = reinterpret_cast<uint32_t*>(dyn);
        for (int e = threadIdx.x; e < a.E; e += kThreads) comb[e] = 0xffffffffu;
        __syncthreads();
        constexpr int kWorkers = kThreads, kU = 8;
        {
            const long long n = (long long)a.cap_sets * a.E;
            for (long long i0 = threadIdx.x; i0 < n; i0 += (long long)kU * kWorkers) {
                uint32_t c[kU];
#pragma unroll
                for (int u = 0; u < kU; ++u) {
                    const long long i = i0 + (long long)u * kWorkers;
                    c[u] = i < n ? __ldcg(a.cap_part + i) : 0xffffffffu;
                }
#pragma unroll
                for (int u = 0; u < kU; ++u) {
                    const long long i = i0 + (long long)u * kWorkers;
                    if (c[u] != 0xffffffffu) atomicMin(&comb[(int)(i % a.E)], c[u]);
                }
            }
        }
        __syncthreads();
        capacity_finish<false>(fs, comb, 1, a.T, a.E, a.H, a.D, a.lnbeta, a.rule, a.delta_e, a.theta_e, a.cap_out);
        return;
    }
    const int nrb = nx - 1 - (a.fuse_cap ? 1 : 0);
    for (int k = (x - 1) * kThreads + threadIdx.x; k < a.K; k += nrb * kThreads)
        a.rowbase[k] = (int)(route_row_base(a, k) * a.C_alloc);
}

// Extra CTAs of the last scatter: the count matrices, which need the capacity.
__device__ void route_extras_b(const RouteArgs& a, int x, int nx) {
    int C = a.cap->C_local;
    if (C > a.C_alloc) {
        C = a.C_alloc;
        if (x == 0 && threadIdx.x == 0) atomicOr(a.status, LOCMOE_WARN_CLAMPED);
    }
    unsigned long long raw0 = 0, raw1 = 0, raw2 = 0, kp0 = 0, kp1 = 0, kp2 = 0;
    for (int k = x * kThreads + threadIdx.x; k < a.K; k += nx * kThreads) {
        const int c = a.counts[k];
        const int kp = c < C ? c : C;
        a.kept[k] = kp;
        if (c == 0) continue;
        const int s = k / a.E, e = k - s * a.E, b = e / a.Ed;
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

// Single-pass sorts have no first scatter to ride on: the capacity-free extras get a launch of their own.
__global__ void __launch_bounds__(kThreads) route_extras_kernel(const RouteArgs a) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ int dyn[];
    route_extras_a(a, blockIdx.x, gridDim.x, dyn);
}

// Large batches only: turns every digit row of hist[pass] into its exclusive prefix along the tiles (in place)
// and stores the row totals, one warp per row, so that a scatter CTA reads one entry per digit instead of a
// whole row (total work O(bins x tiles) instead of O(bins x tiles^2)).
__global__ void __launch_bounds__(kThreads) route_prescan_kernel(const RouteArgs a, int pass) {
    pdl_wait();
    pdl_trigger();
    const int nbins = 1 << a.bits[pass];
    const int lane = threadIdx.x & 31;
    const int d = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (d >= nbins) return;
    int32_t* row = a.hist[pass] + (size_t)d * a.hstride;
    const int chunk = (a.ntiles + 31) / 32;
    const int lo = min(lane * chunk, a.ntiles), hi = min(lo + chunk, a.ntiles);
    int s = 0;
    for (int j = lo; j < hi; ++j) s += row[j];
    int incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    int run = incl - s;
    for (int j = lo; j < hi; ++j) { int v = row[j]; row[j] = run; run += v; }
    if (lane == 31) a.rowtot[d] = incl;
}

// One radix pass over one tile per CTA; CTAs beyond ntiles run the extras.  R = 32-token rounds per warp
// (compile time, so that a small batch does not carry the code of a large one).
template <bool FIRST, bool LAST, int R>
__global__ void __launch_bounds__(kThreads) route_scatter_kernel(const RouteArgs a, int pass, int shift) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ int sm[];
    if ((int)blockIdx.x >= a.ntiles) {
        if (LAST) route_extras_b(a, blockIdx.x - a.ntiles, gridDim.x - a.ntiles);
        else route_extras_a(a, blockIdx.x - a.ntiles, gridDim.x - a.ntiles, sm);
        return;
    }
    const int nbins = 1 << a.bits[pass];
    int* cnt = sm;                       // [kWarps][nbins] per-warp digit counters, then running offsets
    int* pre = sm + kWarps * nbins;      // [nbins] tokens of the digit in earlier tiles
    int* tot = pre + nbins;              // [nbins] tokens of the digit in all tiles, then digit bases
    __shared__ int wsum[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int tileid = blockIdx.x;
    for (int i = tid; i < kWarps * nbins; i += kThreads) cnt[i] = 0;

    // ---- this tile's items, loaded first so that their latency overlaps the offset computation ----
    const uint32_t mask = (uint32_t)nbins - 1u;
    const uint32_t* kin = a.keys[(pass + 1) & 1];
    const int32_t* tin = a.toks[(pass + 1) & 1];
    uint32_t* kout = a.keys[pass & 1];
    int32_t* tout = a.toks[pass & 1];
    const int wbase = tileid * a.tile + w * R * 32;
    const uint32_t lt = (1u << lane) - 1u;
    int* mycnt = cnt + w * nbins;
    int key[R], tok[R], rank[R];
    int kstart[LAST ? R : 1], rbase[LAST ? R : 1];   // last pass: class start and first buffer row of the item's key
    int C = 0;
    if (LAST) { C = a.cap->C_local; if (C > a.C_alloc) C = a.C_alloc; }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        key[r] = -1; tok[r] = -1; rank[r] = 0;
        const int j = wbase + r * 32 + lane;
        if (j < a.T) {
            if (FIRST) {
                const int e = a.idx[j], sd = a.src[j];
                tok[r] = j;
                key[r] = ((unsigned)sd < (unsigned)a.D && (unsigned)e < (unsigned)a.E) ? sd * a.E + e : -1;
            } else {
                key[r] = (int)kin[j]; tok[r] = tin[j];
            }
        }
    }
    if (LAST) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            kstart[r] = 0; rbase[r] = 0;
            if ((unsigned)key[r] < (unsigned)a.K) { kstart[r] = a.keystart[key[r]]; rbase[r] = a.rowbase[key[r]]; }
        }
    }

    // ---- this tile's offsets from the (digit, tile) histogram matrix: one warp per digit row, kRB rows per
    // batch, a row read as 16-byte pieces so that all of a batch's loads are in flight together (L2 resident) ----
    const int32_t* H = a.hist[pass];
    constexpr int kRB = 8;
    if (a.prescan) {
        for (int d = tid; d < nbins; d += kThreads) { pre[d] = H[(size_t)d * a.hstride + tileid]; tot[d] = a.rowtot[d]; }
    } else {
        const int npieces = a.hstride >> 2;
        for (int d0 = w; d0 < nbins; d0 += kWarps * kRB) {
            int before[kRB], all[kRB];
#pragma unroll
            for (int q = 0; q < kRB; ++q) { before[q] = 0; all[q] = 0; }
            for (int c = lane; c < npieces; c += 32) {
                int4 v[kRB];
#pragma unroll
                for (int q = 0; q < kRB; ++q) {
                    const int d = d0 + q * kWarps;
                    v[q] = make_int4(0, 0, 0, 0);
                    if (d < nbins) v[q] = *reinterpret_cast<const int4*>(H + (size_t)d * a.hstride + 4 * c);
                }
                const int j = 4 * c;
                const bool in0 = j < a.ntiles, in1 = j + 1 < a.ntiles, in2 = j + 2 < a.ntiles, in3 = j + 3 < a.ntiles;
                const bool b0 = j < tileid, b1 = j + 1 < tileid, b2 = j + 2 < tileid, b3 = j + 3 < tileid;
#pragma unroll
                for (int q = 0; q < kRB; ++q) {
                    all[q] += (in0 ? v[q].x : 0) + (in1 ? v[q].y : 0) + (in2 ? v[q].z : 0) + (in3 ? v[q].w : 0);
                    before[q] += (b0 ? v[q].x : 0) + (b1 ? v[q].y : 0) + (b2 ? v[q].z : 0) + (b3 ? v[q].w : 0);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int q = 0; q < kRB; ++q) {
                    before[q] += __shfl_xor_sync(0xffffffffu, before[q], o);
                    all[q] += __shfl_xor_sync(0xffffffffu, all[q], o);
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < kRB; ++q) {
                    const int d = d0 + q * kWarps;
                    if (d < nbins) { pre[d] = before[q]; tot[d] = all[q]; }
                }
            }
        }
    }
    __syncthreads();
    // exclusive scan of tot[] over the digits -> digit bases; the grand total is the number of valid items
    int n_valid;
    {
        const int chunk = (nbins + kThreads - 1) / kThreads;
        const int lo = min(tid * chunk, nbins), hi = min(lo + chunk, nbins);
        int s = 0;
        for (int i = lo; i < hi; ++i) s += tot[i];
        int incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) wsum[w] = incl;
        __syncthreads();
        int wb = 0, total = 0;
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) { if (ww < w) wb += wsum[ww]; total += wsum[ww]; }
        n_valid = total;
        int run = wb + incl - s;
        for (int i = lo; i < hi; ++i) { int v = tot[i]; tot[i] = run; run += v; }
    }
    __syncthreads();

    // ---- stable rank inside the tile ----
#pragma unroll
    for (int r = 0; r < R; ++r)
        if (!FIRST && wbase + r * 32 + lane >= n_valid) key[r] = -1;   // beyond the valid items: stale buffer contents
#pragma unroll
    for (int r = 0; r < R; ++r) {
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
    __syncthreads();
    // counters -> starting offsets: digit base + earlier tiles + earlier warps of this tile
    for (int d = tid; d < nbins; d += kThreads) {
        int run = tot[d] + pre[d];
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) {
            const int c = cnt[ww * nbins + d];
            cnt[ww * nbins + d] = run;
            run += c;
        }
    }
    __syncthreads();

    const int nshift = shift + a.bits[pass];
    const uint32_t nmask = LAST ? 0u : (uint32_t)(1 << a.bits[LAST ? pass : pass + 1]) - 1u;
    int32_t* Hn = LAST ? nullptr : a.hist[LAST ? pass : pass + 1];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (key[r] >= 0) {
            const uint32_t d = ((uint32_t)key[r] >> shift) & mask;
            const int dest = mycnt[d] + rank[r];
            if (LAST) {
                // final outputs of the token: dest is its position in the stable sort by key
                const int t = tok[r];
                const int p = dest - kstart[r];
                const bool dropped = p >= C;
                const int row = dropped ? -1 : rbase[r] + p;
                a.pos[t] = p;
                a.drop[t] = dropped ? 1 : 0;
                if (!dropped) a.inv[row] = t;
                a.slot[t] = row;
            } else {
                kout[dest] = (uint32_t)key[r];
                tout[dest] = tok[r];
                atomicAdd(&Hn[(size_t)(((uint32_t)key[r] >> nshift) & nmask) * a.hstride + (dest >> a.tile_shift)], 1);
            }
        }
    }
}

template <int R>
int launch_scatter_r(bool first, bool last, int grid, size_t smb, cudaStream_t st, const RouteArgs& a, int pass, int shift) {
    if (first && last) return launch_pdl(route_scatter_kernel<true, true, R>, grid, kThreads, smb, st, a, pass, shift);
    if (first) return launch_pdl(route_scatter_kernel<true, false, R>, grid, kThreads, smb, st, a, pass, shift);
    if (last) return launch_pdl(route_scatter_kernel<false, true, R>, grid, kThreads, smb, st, a, pass, shift);
    return launch_pdl(route_scatter_kernel<false, false, R>, grid, kThreads, smb, st, a, pass, shift);
}

int launch_scatter(int rounds, bool first, bool last, int grid, size_t smb, cudaStream_t st, const RouteArgs& a, int pass,
                   int shift) {
    switch (rounds) {
        case 2: return launch_scatter_r<2>(first, last, grid, smb, st, a, pass, shift);
        case 4: return launch_scatter_r<4>(first, last, grid, smb, st, a, pass, shift);
        case 8: return launch_scatter_r<8>(first, last, grid, smb, st, a, pass, shift);
        default: return launch_scatter_r<16>(first, last, grid, smb, st, a, pass, shift);
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
    p->passes = (kb + 7) / 8;
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
    while (rounds & (rounds - 1)) ++rounds;   // 2, 4, 8 or 16: the scatter kernel is compiled per value
    p->rounds = rounds;
    p->tile = kWarps * rounds * 32;
    p->ntiles = (int)(((long long)s.T + p->tile - 1) / p->tile);
    p->hstride = (p->ntiles + 3) & ~3;
    size_t off = 0;
    for (int i = 0; i < 2; ++i) {
        p->off_keys[i] = off; off += p->passes > 1 ? align256((size_t)s.T * 4) : 0;
        p->off_toks[i] = off; off += p->passes > 1 ? align256((size_t)s.T * 4) : 0;
    }
    for (int i = 0; i < 4; ++i) {
        p->off_hist[i] = off;
        if (i < p->passes) off += align256(((size_t)p->hstride << p->bits[i]) * 4);
    }
    p->off_keystart = off; off += align256((size_t)K * 4);
    p->off_rowbase = off; off += align256((size_t)K * 4);
    p->off_rowtot = off; off += 1024;
    p->off_cap_part = off; off += align256((size_t)(p->ntiles > 64 ? p->ntiles : 64) * s.E * 4);
    p->nrep = 1;   // enough copies to bring the adds per address down to 16 (config 2's level, where one copy is fastest)
    while (p->nrep < 8 && (long long)p->nrep * 2 * K <= 8192 && (long long)s.T > 16ll * K * p->nrep) p->nrep *= 2;
    p->off_counts_rep = off; off += p->nrep > 1 ? align256((size_t)p->nrep * K * 4) : 0;
    p->total = off;
    p->prescan = ((long long)p->ntiles << p->bits[0]) > 32768 ? 1 : 0;
    {   // testing aid: LOCMOE_PATH=grid forces the large-batch variants at any size
        const char* o = getenv("LOCMOE_PATH");
        if (o && o[0] == 'g') p->prescan = 1;
    }
    p->launches = 2 + p->passes + (p->passes == 1 ? 1 : 0) + (p->prescan ? p->passes : 0);
    return LOCMOE_OK;
}

// The route stage; with `fuse` != nullptr also the capacity stage (its minima ride on hist0, its finish on an extra
// CTA of the first scatter), writing the record to cap_dev before the last scatter reads it.
struct FusedCapacity {
    const float* cos_sim;
    locmoe_capacity_rule_t rule;
    float* delta_e;
    float* theta_e;
};
// The gate of the same step, when it carries the route stage's first pass (locmoe_gate_route).
struct FusedGate {
    const void* x;
    const float* eps;
    int32_t* idx;
    float* gate_w;
    float* cos_sim;
};

static int launch_route_impl(const locmoe_shape_t& s, const int32_t* idx, const int32_t* src, locmoe_capacity_t* cap_dev,
                             const FusedCapacity* fuse, const FusedGate* gate, int early_init, int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop,
                             int32_t* inv, int32_t* counts, int32_t* kept, int32_t* send_counts, int32_t* load,
                             int64_t* locality, int32_t* status, void* ws, cudaStream_t st) {
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
    a.tile = p.tile; a.rounds = p.rounds; a.ntiles = p.ntiles; a.passes = p.passes;
    char* w = static_cast<char*>(ws);
    for (int i = 0; i < 2; ++i) {
        a.keys[i] = reinterpret_cast<uint32_t*>(w + p.off_keys[i]);
        a.toks[i] = reinterpret_cast<int32_t*>(w + p.off_toks[i]);
    }
    for (int i = 0; i < kMaxPasses; ++i) {
        a.bits[i] = p.bits[i];
        a.hist[i] = reinterpret_cast<int32_t*>(w + p.off_hist[i]);
    }
    a.counts_rep = reinterpret_cast<int32_t*>(w + p.off_counts_rep);
    a.nrep = gate ? 1 : p.nrep;
    a.keystart = reinterpret_cast<int32_t*>(w + p.off_keystart);
    a.rowbase = reinterpret_cast<int32_t*>(w + p.off_rowbase);
    a.hstride = p.hstride;
    a.tile_shift = 0;
    while ((1 << a.tile_shift) < p.tile) ++a.tile_shift;
    a.rowtot = reinterpret_cast<int32_t*>(w + p.off_rowtot);
    a.prescan = p.prescan;
    a.fuse_cap = fuse ? 1 : 0;
    a.hist_by_gate = gate ? 1 : 0;
    a.cap_sets = p.ntiles;
    if (gate) {   // replicas of the row of minima: as many as keep sets * E within 8192 words, at most 64
        a.cap_sets = 1;
        while (a.cap_sets < 64 && (long long)a.cap_sets * 2 * s.E <= 8192) a.cap_sets *= 2;
    }
    a.H = s.H;
    if (fuse) {
        a.cos = fuse->cos_sim; a.rule = fuse->rule; a.delta_e = fuse->delta_e; a.theta_e = fuse->theta_e;
        a.cap_out = cap_dev;
        a.lnbeta = ln_beta_half(s.H);
        a.cap_part = reinterpret_cast<uint32_t*>(w + p.off_cap_part);
    }
    const size_t hist_smem = (fuse && !gate) ? (size_t)s.E * sizeof(uint32_t) : 0;           // hist0's minima of its tile
    const size_t cap_smem = (fuse && a.cap_sets > 1) ? (size_t)s.E * sizeof(uint32_t) : 0;   // the row of combined minima

    long long init_items = a.rows > a.K ? a.rows : a.K;
    int init_blocks = (int)((init_items + kThreads * 4 - 1) / (kThreads * 4));
    if (init_blocks > 4 * sm_count()) init_blocks = 4 * sm_count();
    if (init_blocks < 1) init_blocks = 1;
    if ((rc = launch_pdl(route_init_kernel, init_blocks, kThreads, 0, st, a, early_init))) return rc;

    if (gate) {
        GateFuse gf{};
        gf.src = src; gf.counts = counts; gf.hist0 = a.hist[0]; gf.cap_min = a.cap_part; gf.min_sets = a.cap_sets;
        gf.pos = pos; gf.slot = slot; gf.drop = drop; gf.status = status;
        gf.D = a.D; gf.digit_mask = (1 << p.bits[0]) - 1; gf.hstride = a.hstride; gf.tile_shift = a.tile_shift;
        if ((rc = launch_gate(s, gate->x, gate->eps, gate->idx, gate->gate_w, gate->cos_sim, nullptr, st, &gf))) return rc;
    } else if ((rc = launch_pdl(route_hist0_kernel, p.ntiles, kThreads, (sizeof(int) << p.bits[0]) + hist_smem, st, a))) {
        return rc;
    }

    int per_key = (a.K + kThreads * 4 - 1) / (kThreads * 4);   // CTAs that walk the K key classes
    if (per_key > 32) per_key = 32;
    if (per_key < 1) per_key = 1;
    const int extras_a = 1 + per_key + (fuse ? 1 : 0), extras_b = per_key;
    if (p.passes == 1) {
        if ((rc = launch_pdl(route_extras_kernel, extras_a, kThreads, cap_smem, st, a))) return rc;
    }
    int shift = 0;
    for (int pass = 0; pass < p.passes; ++pass) {
        const bool first = pass == 0, last = pass == p.passes - 1;
        if (p.prescan) {
            if ((rc = launch_pdl(route_prescan_kernel, ((1 << p.bits[pass]) + kWarps - 1) / kWarps, kThreads, 0, st, a, pass))) return rc;
        }
        size_t smb = ((size_t)(kWarps + 2) * sizeof(int)) << p.bits[pass];
        if (first && !last && cap_smem > smb) smb = cap_smem;
        const int grid = p.ntiles + (last ? extras_b : (first ? extras_a : 0));
        rc = launch_scatter(p.rounds, first, last, grid, smb, st, a, pass, shift);
        if (rc) return rc;
        shift += p.bits[pass];
    }
    return LOCMOE_OK;
}

int launch_route(const locmoe_shape_t& s, const int32_t* idx, const int32_t* src, const locmoe_capacity_t* cap_dev,
                 int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                 int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                 void* ws, cudaStream_t st) {
    return launch_route_impl(s, idx, src, const_cast<locmoe_capacity_t*>(cap_dev), nullptr, nullptr, 0, C_alloc, pos, slot, drop, inv,
                             counts, kept, send_counts, load, locality, status, ws, st);
}

bool capacity_route_fusable(const locmoe_shape_t& s) { return s.E <= 8192; }

int launch_capacity_route(const locmoe_shape_t& s, const int32_t* idx, const float* cos_sim, const int32_t* src,
                          const locmoe_capacity_rule_t& rule, float* delta_e, float* theta_e, locmoe_capacity_t* cap_dev,
                          int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                          int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                          int early_init, void* ws, cudaStream_t st) {
    if (!capacity_route_fusable(s)) {
        int rc = launch_capacity(s, idx, cos_sim, rule, delta_e, theta_e, cap_dev, ws, st);
        if (rc) return rc;
        return launch_route(s, idx, src, cap_dev, C_alloc, pos, slot, drop, inv, counts, kept, send_counts, load, locality,
                            status, ws, st);
    }
    const FusedCapacity f{cos_sim, rule, delta_e, theta_e};
    return launch_route_impl(s, idx, src, cap_dev, &f, nullptr, early_init, C_alloc, pos, slot, drop, inv, counts, kept, send_counts,
                             load, locality, status, ws, st);
}

// Gate, capacity and route as one chain: fill -> gate (which also takes the route stage's first pass over the
// tokens and the cosine minima) -> scatter passes.  Any number of experts (the minima live in global memory).
int launch_gate_route(const locmoe_shape_t& s, const void* x, const float* eps, const int32_t* src,
                      const locmoe_capacity_rule_t& rule, int32_t* idx, float* gate_w, float* cos_sim, float* delta_e,
                      float* theta_e, locmoe_capacity_t* cap_dev, int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop,
                      int32_t* inv, int32_t* counts, int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality,
                      int32_t* status, int early_init, void* ws, cudaStream_t st) {
    const FusedCapacity f{cos_sim, rule, delta_e, theta_e};
    const FusedGate g{x, eps, idx, gate_w, cos_sim};
    return launch_route_impl(s, idx, src, cap_dev, &f, &g, early_init, C_alloc, pos, slot, drop, inv, counts, kept, send_counts,
                             load, locality, status, ws, st);
}

}  // namespace locmoe
