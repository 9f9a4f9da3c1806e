/*
 * locmoe.h -- C ABI of the B200 (sm_100a) LocMoE router path.
 *
 * One MoE layer's routing, as defined in "LocMoE: A Low-Overhead MoE for Large
 * Language Model Training" (arXiv 2401.13920), split into five calls:
 *
 *   locmoe_gate      Sec. 3.2.1  GrAP gate, ReLU, softmax, top-1 and its score
 *   locmoe_capacity  abstract + Sec. 3.2.3 (Lemma 3, Theorem 1) capacity rule
 *   locmoe_route     Sec. 3.2.3 / 3.2.4  capacity-bounded placement of tokens
 *                    into an All-to-All shaped buffer, intra-node first
 *   locmoe_dispatch  row gather into that buffer
 *   locmoe_combine   first equation of Sec. 3.2.1: y_m = R_m * expert output
 *
 * Conventions
 *   - Every array pointer is a DEVICE pointer owned by the caller unless the
 *     parameter is documented as host memory.  The shape / rule structs
 *     passed by pointer are HOST memory and are read before the call returns.
 *   - The library allocates no device memory, keeps no state between calls and
 *     never synchronises (locmoe_capacity_read excepted).  All work is queued
 *     on the CUDA stream given as `stream` (a cudaStream_t cast to void*;
 *     NULL = the default stream).  Scratch memory comes from the caller:
 *     `ws` with at least locmoe_workspace_bytes() bytes, 256-byte aligned.
 *   - Return value: 0 = LOCMOE_OK, < 0 = error found on the host before any
 *     launch (nothing was queued), except LOCMOE_ERR_CUDA which reports a
 *     failed launch.  Conditions met on the device (capacity clamped, a token
 *     with an impossible source device) set LOCMOE_WARN_* bits in the
 *     caller's int32 status word; no kernel traps or asserts.
 *   - Environment variables, read at call time, select alternative kernels.
 *     They are testing aids (every choice gives the same results) and no part
 *     of the interface a program should rely on:
 *       LOCMOE_PATH=grid|cluster    capacity / route: force the multi-kernel or
 *                                   the one-cluster form regardless of size
 *       LOCMOE_GATE=general         gate: the general kernel on shapes that have
 *                                   a specialised one
 *       LOCMOE_DISPATCH=tma|vec|flat  dispatch: bulk-copy, warp-per-row or flat
 *                                   row-major kernel
 *       LOCMOE_FFN=1|w|w1|w2|2|2s   expert FFN: the 128 x 256-tile kernel for both
 *                                   GEMMs, the 256 x 256-tile kernel for both / the
 *                                   first / the second (default: chosen per GEMM by
 *                                   its reduction length), the two-SM kernel (2s:
 *                                   with one accumulator)
 *       LOCMOE_PDL=0                plain launches instead of programmatic
 *                                   dependent launches (read once per process)
 *       LOCMOE_DEBUG=1              print the CUDA error behind LOCMOE_ERR_CUDA
 *   - Row-major, densely packed arrays.  T tokens, H hidden size (the paper's
 *     d), E experts (n), g = H / E group width.  Logical devices
 *     D = n_nodes * dev_per_node; E % D == 0; expert e lives on device
 *     e / (E / D) ("expert_num_per_dp_dim x expert_parallel", Appendix D).
 */
#ifndef LOCMOE_H
#define LOCMOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { LOCMOE_F32 = 0, LOCMOE_BF16 = 1 };
enum { LOCMOE_LAYOUT_SEND = 0, LOCMOE_LAYOUT_RECV = 1 };
enum { LOCMOE_BOUND_BETA = 0, LOCMOE_BOUND_ERFC = 1, LOCMOE_BOUND_EXP = 2 };
enum {
    LOCMOE_OK = 0,
    LOCMOE_ERR_NULL = -1,      /* a required pointer is NULL                           */
    LOCMOE_ERR_SHAPE = -2,     /* T < 1, H % E != 0, E % D != 0, rows overflow int32...*/
    LOCMOE_ERR_DTYPE = -3,     /* unknown dtype / layout / bound form                  */
    LOCMOE_ERR_ALIGN = -4,     /* a pointer lacks the stated alignment                 */
    LOCMOE_ERR_WORKSPACE = -5, /* ws too small or misaligned                           */
    LOCMOE_ERR_CUDA = -6,      /* a CUDA call failed (launch error is cleared)         */
    LOCMOE_ERR_TOO_LARGE = -7  /* size beyond the built-in scratch of a no-allocation call */
};
enum {                         /* bits of the device status word                       */
    LOCMOE_WARN_CLAMPED = 1,   /* C_local > C_alloc: capacity clamped to C_alloc       */
    LOCMOE_WARN_BAD_SRC = 2,   /* a token's source device is outside [0, D): dropped   */
    LOCMOE_WARN_BAD_IDX = 4    /* a token's expert index is outside [0, E): dropped    */
};
enum {                         /* bits of locmoe_capacity_t.flags                      */
    LOCMOE_FLAG_DELTA_OVERRIDE = 1, /* delta came from the rule, not the data          */
    LOCMOE_FLAG_MIN_SATURATED = 2,  /* min_mult * ec_min >= T (or overflowed): T used  */
    LOCMOE_FLAG_MIN_BINDS = 4       /* Theorem 1's minimum set C_local                 */
};

/* Problem shape (host struct). */
typedef struct {
    int32_t T;            /* tokens in the batch, >= 1                                 */
    int32_t H;            /* hidden size d, a multiple of E                            */
    int32_t E;            /* experts n                                                 */
    int32_t n_nodes;      /* logical nodes N                                           */
    int32_t dev_per_node; /* logical devices per node Dn; D = N * Dn divides E         */
    int32_t x_dtype;      /* LOCMOE_F32 | LOCMOE_BF16: tokens, buffer and combined out */
    int32_t layout;       /* LOCMOE_LAYOUT_SEND | LOCMOE_LAYOUT_RECV                   */
} locmoe_shape_t;

/* Capacity rule (host struct).  Capacity = max(Theorem 1's minimum * min_mult,
 * conventional ec = ceil(T * capacity_factor / (D * n))), see locmoe_capacity. */
typedef struct {
    double min_mult;        /* multiplier on ec_min of Theorem 1                       */
    double capacity_factor; /* c_f of Sec. 3.2.3; 0 = use the minimum alone            */
    double delta_override;  /* < 0: measure delta from the batch; else use this value  */
    int32_t bound_form;     /* LOCMOE_BOUND_*: which form of Theorem 1                 */
    int32_t T_global;       /* 0: the batch is shape->T; > 0: tokens of the whole batch
                             * when this call sees one rank's share (with the whole
                             * batch's delta passed as delta_override)                  */
} locmoe_capacity_rule_t;

/* Capacity record (written on the device by locmoe_capacity). */
typedef struct {
    double delta;            /* cosine threshold: min over experts of delta_e, >= 0    */
    double p_delta;          /* Lemma 3: 1 - I_{delta^2}(1/2, (d-1)/2)                 */
    double ec_min;           /* Theorem 1 in the chosen form                           */
    int32_t C_expert;        /* slots per expert over all sources                      */
    int32_t C_local;         /* slots per (source device, expert) pair                 */
    int32_t n_empty_experts; /* experts that received no token                         */
    int32_t flags;           /* LOCMOE_FLAG_*                                          */
} locmoe_capacity_t;

/* Scratch size for locmoe_capacity and locmoe_route on this shape (they may
 * share one workspace; calls on one stream run in order).  `bytes` is host
 * memory.  C_alloc is the row stride the caller will pass to locmoe_route. */
int locmoe_workspace_bytes(const locmoe_shape_t *shape, int32_t C_alloc, size_t *bytes);

/*
 * GrAP gate (Sec. 3.2.1).  For each token t, with the fixed weight
 * w_i = (n/d) 1{i d/n <= j < (i+1) d/n}:
 *   mean_i = w_i . x_t (average of the i-th group of g entries, fp32 accumulation)
 *   G_i    = ReLU(mean_i + eps_i)                    (eps == NULL means 0)
 *   idx[t] = lowest i attaining max_i softmax(G)_i   (Eq. "max_expert")
 *   gate_w[t] = softmax(G)[idx[t]]                   (Eq. "gating_score")
 *   cos_sim[t] = <w_idx, x_t> / (|w_idx| |x_t|)      (Lemma 1; 0 for a zero token)
 *   probs[t][i] = softmax(G)_i                       (optional, NULL to skip)
 * Tokens are expected to be finite.  A token with an infinity or a NaN in it gets
 * unspecified score and cosine (possibly NaN) and a valid expert index in [0, E);
 * it does not disturb any other token's outputs, and nothing faults.  A NaN cosine
 * may or may not enter its expert's minimum in locmoe_capacity.
 * x: [T][H] of shape->x_dtype.  The fast path needs x 16-byte aligned and
 * H * sizeof(element) a multiple of 16; other inputs take a slower scalar path.
 * idx int32[T], gate_w / cos_sim float[T], probs float[T][E], eps float[E].
 */
int locmoe_gate(const locmoe_shape_t *shape, const void *x, const float *eps,
                int32_t *idx, float *gate_w, float *cos_sim, float *probs, void *stream);

/*
 * The gate with its optional extras (Sec. 3.2.1 for the bias eps_i, which the paper
 * leaves undefined; Sec. 3.2.2 for the P_i of the auxiliary loss).  Same outputs as
 * locmoe_gate; the options struct is HOST memory, its pointers are device pointers.
 *   eps / src_dev  with src_dev == NULL, eps is float[E] as in locmoe_gate (or NULL).
 *                  With src_dev int32[T], eps is a table float[D][E] and token t takes
 *                  the row of its source device: G_i = ReLU(mean_i + eps[src_dev[t]][i]);
 *                  a token whose source is outside [0, D) gets no bias.
 *   probs          float[T][E] or NULL, as in locmoe_gate.
 *   p_part         float[LOCMOE_GATE_PARTIAL_ROWS][E] or NULL: the column sums of the
 *                  probabilities, formed inside the gate kernel -- every CTA adds the rows
 *                  of its warps in a fixed order and writes one row of p_part -- so that
 *                  P_i and L_aux need no probability matrix (locmoe_aux_loss_partial).
 *                  The number of rows written is returned in p_rows (host field); it
 *                  depends on the shape and the device only, and so does the summation
 *                  order: the sums are deterministic.
 */
enum { LOCMOE_GATE_PARTIAL_ROWS = 2048 };
typedef struct {
    const float *eps;
    const int32_t *src_dev;
    float *probs;
    float *p_part;
    int32_t p_rows;  /* out */
} locmoe_gate_opts_t;
int locmoe_gate_ex(const locmoe_shape_t *shape, const void *x, locmoe_gate_opts_t *opts,
                   int32_t *idx, float *gate_w, float *cos_sim, void *stream);

/*
 * Angular deviation and capacity (abstract; Lemma 3; Theorem 1; Sec. 3.2.3).
 *   delta_e[e] = smallest cos_sim among tokens with idx == e (1 if none),
 *   theta_e[e] = acos(delta_e[e])  -- the largest angle between expert e's
 *                gating weight and a token assigned to it,
 *   delta      = clamp(min_e delta_e, 0, 1) or rule->delta_override,
 *   p_delta, ec_min = 1 / (n p_delta) (or the erfc / exp form),
 *   Cmin       = ceil(min(min_mult * ec_min, T)),
 *   C_expert   = clamp(max(Cmin, ceil(c_f T / n), 1), 1, T),
 *   C_local    = clamp(max(ceil(Cmin / D), ceil(c_f T / (D n)), 1), 1, T).
 * delta_e / theta_e: float[E]; cap_dev: device record; ws: see above.
 */
int locmoe_capacity(const locmoe_shape_t *shape, const int32_t *idx, const float *cos_sim,
                    const locmoe_capacity_rule_t *rule, float *delta_e, float *theta_e,
                    locmoe_capacity_t *cap_dev, void *ws, size_t ws_bytes, void *stream);

/*
 * The same computation as locmoe_capacity, for callers that cannot supply a
 * workspace.  (This entry point has no counterpart in the paper; it exists for
 * deployment reasons only.)
 *
 * Meant for host code that has no device allocator to turn to: a plug-in inside
 * a serving process that has already claimed the whole HBM for its own pools,
 * so that a cudaMalloc would fail or eat into them, or a C caller that is handed
 * nothing but the input and output buffers of an operator.  The scratch that
 * locmoe_capacity takes from `ws` is here a fixed 256 KiB array inside the
 * library's device image; the call itself performs no cudaMalloc / cudaFree and
 * uses no allocating library routine.  Inputs and outputs are the caller's, as
 * in locmoe_capacity, with the same meaning, layout and results.
 *
 * Limits and rules that follow from the built-in array:
 *   - at most 8192 experts; a larger shape->E returns LOCMOE_ERR_TOO_LARGE
 *     before anything is launched;
 *   - every GPU on which the library is used holds the 256 KiB until the
 *     process exits;
 *   - all calls on one device share the array and it keeps whatever the last
 *     call left in it.  Each call rewrites all it reads, so calls that follow
 *     one another on a stream are independent, but two calls that can overlap
 *     on the GPU (different streams, no dependency) race on it and must be
 *     ordered by the caller;
 *   - the first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and caches it; make
 *     that first call outside of, and before, any stream capture;
 *   - the cached address is that of the device's primary context at the time
 *     of the first call.  A cudaDeviceReset, or a switch to another context on
 *     the same device, makes it stale: do not call this entry point afterwards
 *     (the library cannot detect this, and kernels would write through a dead
 *     address).
 */
int locmoe_capacity_noalloc(const locmoe_shape_t *shape, const int32_t *idx, const float *cos_sim,
                            const locmoe_capacity_rule_t *rule, float *delta_e, float *theta_e,
                            locmoe_capacity_t *cap_dev, void *stream);

/* Copies the device record to host memory and waits for the stream. */
int locmoe_capacity_read(const locmoe_capacity_t *cap_dev, locmoe_capacity_t *cap_host, void *stream);

/*
 * Capacity-bounded routing (Sec. 3.2.3 capacity limit; Sec. 3.2.4 exchange).
 * Token t comes from logical device src_dev[t] and goes to expert idx[t].
 * C = min(cap_dev->C_local, C_alloc).
 *   pos[t]  = number of earlier tokens (lower t) with the same (src, expert)
 *   drop[t] = pos[t] >= C; a dropped token gets slot[t] = -1
 *   slot[t] = row of the token in the buffer of D * E * C_alloc rows:
 *     SEND layout  ((src * D + r(src, dev(e))) * Ed + e % Ed) * C_alloc + pos
 *     RECV layout  ((e * D) + r(dev(e), src)) * C_alloc + pos
 *     with r(a, b) = ((node(b) - node(a)) mod N) * Dn + ((loc(b) - loc(a)) mod Dn):
 *     a device lists itself first, then its own node, then the other nodes.
 *   inv[row] = t for an occupied row, -1 otherwise          int32[D * E * C_alloc]
 *   counts[s][e] tokens demanded, kept[s][e] = min(counts, C)      int32[D][E]
 *   send_counts[s][b] = kept tokens from s to the experts of device b  int32[D][D]
 *   load[e] = sum_s counts[s][e]                                   int32[E]
 *   locality[0][c] / locality[1][c]: tokens demanded / kept by class c
 *     (0 same device, 1 same node, 2 other node)                   int64[2][3]
 *   status: int32 word, LOCMOE_WARN_* bits are OR-ed in (it is zeroed first).
 * The result is deterministic: it depends only on the inputs.
 */
int locmoe_route(const locmoe_shape_t *shape, const int32_t *idx, const int32_t *src_dev,
                 const locmoe_capacity_t *cap_dev, int32_t C_alloc,
                 int32_t *pos, int32_t *slot, uint8_t *drop, int32_t *inv,
                 int32_t *counts, int32_t *kept, int32_t *send_counts, int32_t *load,
                 int64_t *locality, int32_t *status, void *ws, size_t ws_bytes, void *stream);

/*
 * locmoe_capacity followed by locmoe_route as ONE call with the same inputs,
 * outputs and results (Sec. 3.2.3): the per-expert minima of the cosines are
 * taken by the route stage's first pass over the tokens and the closed forms
 * are evaluated beside its first sorting pass, so the capacity stage costs no
 * launch and no pass of its own; the last sorting pass reads the record from
 * cap_dev.  Beyond 8192 experts the two stages simply run one after the other.
 * ws: at least locmoe_workspace_bytes() bytes.
 * flags: 0, or LOCMOE_ROUTE_EARLY_INIT: the caller states that the kernel queued
 * on the stream immediately before this call (typically locmoe_gate of the same
 * step) neither reads nor writes any output array or the workspace of this
 * call, and, if it was itself launched for programmatic dependent launch, that
 * it waits for its own predecessors before it lets its successor start (every
 * kernel of this library does).  The stage's fill of inv / counters may then
 * run while that kernel drains instead of after it.  Results are the same.
 */
enum { LOCMOE_ROUTE_EARLY_INIT = 1 };
int locmoe_capacity_route(const locmoe_shape_t *shape, const int32_t *idx, const float *cos_sim,
                          const int32_t *src_dev, const locmoe_capacity_rule_t *rule,
                          float *delta_e, float *theta_e, locmoe_capacity_t *cap_dev, int32_t C_alloc,
                          int32_t *pos, int32_t *slot, uint8_t *drop, int32_t *inv, int32_t *counts,
                          int32_t *kept, int32_t *send_counts, int32_t *load, int64_t *locality,
                          int32_t *status, int32_t flags, void *ws, size_t ws_bytes, void *stream);

/*
 * locmoe_gate, locmoe_capacity and locmoe_route as ONE call with the same
 * inputs, outputs and results (probabilities are not available in this form).
 * The route stage's fill kernel runs first; the gate kernel, as it finishes a
 * token, also takes that token's share of the route stage's first pass (the
 * demand count of its (source, expert) pair, the digit histogram of the first
 * sorting pass, the minimum cosine of its expert) with integer atomics; the
 * sorting passes follow, the first of them carrying the capacity rule.  Two
 * launches and one pass over the index arrays less than the separate calls.
 * flags: 0 or LOCMOE_ROUTE_EARLY_INIT, which here speaks about the kernel
 * queued before THIS call (for instance the combine of the previous step):
 * it touches none of this call's route outputs or workspace.
 */
int locmoe_gate_route(const locmoe_shape_t *shape, const void *x, const float *eps,
                      const int32_t *src_dev, const locmoe_capacity_rule_t *rule, int32_t *idx,
                      float *gate_w, float *cos_sim, float *delta_e, float *theta_e,
                      locmoe_capacity_t *cap_dev, int32_t C_alloc, int32_t *pos, int32_t *slot,
                      uint8_t *drop, int32_t *inv, int32_t *counts, int32_t *kept,
                      int32_t *send_counts, int32_t *load, int64_t *locality, int32_t *status,
                      int32_t flags, void *ws, size_t ws_bytes, void *stream);

/*
 * Dispatch: buf[row][:] = x[inv[row]][:] bit for bit for occupied rows; rows
 * with inv < 0 are zero-filled when zero_pad != 0 and left untouched otherwise.
 * x [T][H], buf [D * E * C_alloc][H], both of shape->x_dtype.
 * slot is optional (NULL allowed): int32[T] as written by locmoe_route for the
 * same routing, i.e. inv[slot[t]] == t for every kept token.  The result is the
 * same with or without it; with it the rows are copied token by token in
 * descending token order, so that the tokens the gate read last, which are
 * still in L2, are read first, and the rows written last are those a combine in
 * ascending token order reads first.  A slot array that does not belong to inv
 * gives an unspecified buffer (no out-of-range access: entries outside
 * [0, rows) are skipped).
 */
int locmoe_dispatch(const locmoe_shape_t *shape, int32_t C_alloc, const void *x,
                    const int32_t *inv, const int32_t *slot, void *buf, int32_t zero_pad,
                    void *stream);

/*
 * Combine: out[t][:] = gate_w[t] * y[slot[t]][:] for a kept token and 0 for a
 * dropped one; with accumulate != 0 the product is added to out (a dropped
 * token then leaves out unchanged).  y [D * E * C_alloc][H] of y_dtype,
 * out [T][H] of shape->x_dtype; the product (and the sum) is formed in fp32
 * and then rounded to the output type, to nearest-even.
 */
int locmoe_combine(const locmoe_shape_t *shape, int32_t C_alloc, const void *y, int32_t y_dtype,
                   const int32_t *slot, const float *gate_w, void *out, int32_t accumulate,
                   void *stream);

/*
 * Dispatch and combine fused with the exchange around the experts (Sec. 3.2.4:
 * the All-to-All before and after the expert networks), for one process per
 * GPU.  Every rank routes the tokens of its own logical source devices
 * [src_lo, src_hi) with the shape of the WHOLE logical map (n_nodes,
 * dev_per_node, E; shape->T = this rank's tokens; layout must be
 * LOCMOE_LAYOUT_RECV), so slot / inv index the global receive-side buffer of
 * D * E * C_alloc rows.  That buffer is spread over n_peers GPUs, expert-major:
 * peer q holds the rows [q * R, (q + 1) * R), R = D * E * C_alloc / n_peers
 * (n_peers divides D, at most 64).
 *
 * locmoe_dispatch_peer stores each kept token's row directly into the buffer of
 * the peer that hosts its expert (peer_bufs[q], base of peer q's R rows, a
 * pointer valid on this GPU: its own allocation or a peer mapping) and, with
 * zero_pad, zero-fills the empty rows whose source device is its own; rows of
 * other ranks' sources are left alone.  locmoe_combine_peer reads the expert
 * output row of each kept token from peer_y[q] and writes
 * out[t] = gate_w[t] * y[slot[t]] (0 for a dropped token), as locmoe_combine.
 * peer_bufs / peer_y are HOST arrays of n_peers device pointers, 16-byte
 * aligned; rows must be a multiple of 16 bytes.  Plain loads and stores only
 * (no bulk copies, no multicast).  Nothing here waits for another GPU: the
 * caller orders dispatch -> experts -> combine across ranks (a barrier after
 * the stream has been synchronised).
 */
int locmoe_dispatch_peer(const locmoe_shape_t *shape, int32_t C_alloc, const void *x,
                         const int32_t *inv, const int32_t *slot, void *const *peer_bufs,
                         int32_t n_peers, int32_t src_lo, int32_t src_hi, int32_t zero_pad,
                         void *stream);
/* locmoe_dispatch_peer restricted to a window of every owner's buffer: only rows whose index INSIDE their
 * owner's slice lies in [win_lo, win_hi) are stored or zero-filled (0 and INT64_MAX: everything).  With the
 * window of one block of experts, a caller fills the receive buffer block by block and starts the experts of
 * a block while the next one is in flight -- the overlap of the exchange with the expert computation of
 * Sec. 3.2.4. */
int locmoe_dispatch_peer_window(const locmoe_shape_t *shape, int32_t C_alloc, const void *x,
                                const int32_t *inv, const int32_t *slot, void *const *peer_bufs,
                                int32_t n_peers, int32_t src_lo, int32_t src_hi, int32_t zero_pad,
                                int64_t win_lo, int64_t win_hi, void *stream);
int locmoe_combine_peer(const locmoe_shape_t *shape, int32_t C_alloc, void *const *peer_y,
                        int32_t n_peers, int32_t y_dtype, const int32_t *slot, const float *gate_w,
                        void *out, void *stream);

/*
 * Top-k variant (the paper routes each token to its single best expert, Sec.
 * 3.2.1; routers that keep the k best are the family it departs from, Sec. 2).
 * The sum of Sec. 3.2.1's first equation then runs over the K chosen experts,
 * each with its softmax score (not renormalised over the chosen ones).
 *
 * locmoe_topk_select: probs float[T][E], idx int32[T], gate_w float[T] as written
 * by locmoe_gate.  Choice 0 of a token is idx / gate_w; choice c > 0 is the
 * expert with the largest probability among those not yet chosen, a tie going
 * to the lower index.  idx_k int32[K][T], w_k float[K][T]; 1 <= K <= min(8, E).
 *
 * Routing: run locmoe_capacity on the first choices with rule.T_global = K * T
 * and locmoe_route with a shape whose T is K * T on the K * T "virtual tokens"
 * v = c * T + t (idx_k as int32[K * T], src_dev repeated K times): all first
 * choices come before all second choices in a queue.  Then
 * locmoe_topk_fold (shape->T = T tokens, the same C_alloc) rewrites inv[row]
 * from v to the token v mod T, after which locmoe_dispatch (slot = NULL) fills
 * the buffer from x [T][H].
 *
 * locmoe_combine_topk: out[t][:] = sum over c < K of w_k[c][t] * y[slot_k[c][t]][:],
 * a dropped choice (slot < 0) having no term, accumulated in fp32 in the order
 * c = 0, 1, ... (first term a product, the others fused multiply-adds) and
 * rounded once to shape->x_dtype.  slot_k int32[K][T] is the route stage's slot
 * array of the K * T virtual tokens.  Rows must be multiples of 8 elements and
 * the pointers 16-byte aligned.
 */
int locmoe_topk_select(const locmoe_shape_t *shape, const float *probs, const int32_t *idx,
                       const float *gate_w, int32_t K, int32_t *idx_k, float *w_k, void *stream);
int locmoe_topk_fold(const locmoe_shape_t *shape, int32_t C_alloc, int32_t *inv, void *stream);
int locmoe_combine_topk(const locmoe_shape_t *shape, int32_t C_alloc, const void *y, int32_t y_dtype,
                        int32_t K, const int32_t *slot_k, const float *w_k, void *out, void *stream);

/*
 * Auxiliary load-balance loss, forward value (Sec. 3.2.2):
 *   L_aux = alpha * n * sum_i f_i * P_i,  f_i = load[i] / T (share of tokens whose
 *   arg-max is expert i),  P_i = (1/T) sum_t probs[t][i]  (the paper uses alpha = 0.01).
 * probs float[T][E] as written by locmoe_gate, load int32[E] as written by
 * locmoe_route; f_out / p_out float[E], loss_out float[1].  Sums are formed in a
 * fixed order (deterministic).  ws: at least locmoe_workspace_bytes() bytes.
 */
int locmoe_aux_loss(const locmoe_shape_t *shape, const float *probs, const int32_t *load, float alpha,
                    float *f_out, float *p_out, float *loss_out, void *ws, size_t ws_bytes, void *stream);

/* The same loss (Sec. 3.2.2) from the per-CTA column sums locmoe_gate_ex left in p_part
 * (p_rows rows of E floats): P_i = (1/T) * sum of the rows in index order, in fp64.  No
 * probability matrix and no workspace. */
int locmoe_aux_loss_partial(const locmoe_shape_t *shape, const float *p_part, int32_t p_rows,
                            const int32_t *load, float alpha, float *f_out, float *p_out,
                            float *loss_out, void *stream);

/*
 * Locality loss, forward value (Sec. 3.2.2, second loss equation):
 *   L_loc = mu * KL(D_c || D_l),
 * D_c the current assignment distribution of the batch, D_l the fully localised
 * one.  The paper gives no symbols for the two, no value of mu and no rule for
 * experts to which D_l gives no mass; this call fixes the following reading.
 * A source group s is a logical device (level = 0) or a logical node
 * (level = 1), G their number (D or N); group s hosts the E / G experts
 * [s * E / G, (s + 1) * E / G).  With n_s the tokens that group s routed and
 * T_r their sum,
 *   D_c(s, e) = counts[s][e] / T_r,
 *   D_l(s, e) = (n_s / T_r) * q_s(e),
 *   q_s(e) = (1 - smooth) / (E / G) for the experts s hosts, plus smooth / E for every e,
 *   KL(D_c || D_l) = sum_s (n_s / T_r) * KL_s,  KL_s = sum_e c_s(e) ln(c_s(e) / q_s(e)),
 *   c_s(e) = counts[s][e] / n_s, 0 ln 0 = 0, a group without tokens adds nothing.
 * smooth in [0, 1]; with smooth = 0 a single token outside its group makes the
 * value +inf.  counts int32[D][E] as written by locmoe_route (summed over the
 * devices of a node for level 1).  Outputs, all on the device: dc_out
 * float[G][E] = c_s(e); kl_out double[G] = KL_s; group_tokens int64[G] = n_s;
 * loss_out double[1].  Arithmetic in fp64, sums in a fixed order.
 */
int locmoe_loc_loss(const locmoe_shape_t *shape, const int32_t *counts, int32_t level, double mu,
                    double smooth, float *dc_out, double *kl_out, int64_t *group_tokens,
                    double *loss_out, void *stream);

/*
 * Cosine-frequency diagnostic (Sec. 4.1, the second cosine-histogram figure):
 * over the tokens t with idx[t] == expert, the histogram of cos(x_t, w_expert)
 * (the gating weight of the expert the token was routed to) and the histogram
 * of cos(x_t, w_other), where cos(x, w_i) = (sum of the i-th group of d/n
 * entries of x) / (sqrt(d/n) * |x|), 0 for a zero token.  nbins equal bins on
 * [lo, hi); a value below lo counts in the first bin, a value >= hi in the
 * last.  x [T][H] of shape->x_dtype, idx int32[T] as written by locmoe_gate.
 * Outputs on the device: hist_routed / hist_other int32[nbins], n_routed
 * int32[1] (tokens routed to `expert`); they are zeroed first.  Cosines and the
 * bin index are computed in fp32.
 */
int locmoe_cos_hist(const locmoe_shape_t *shape, const void *x, const int32_t *idx, int32_t expert,
                    int32_t other, int32_t nbins, float lo, float hi, int32_t *hist_routed,
                    int32_t *hist_other, int32_t *n_routed, void *stream);

/*
 * Expert feed-forward networks (first equation of Sec. 3.2.1):
 *   y[row] = W_out[e] . GeLU(W_in[e] . buf[row]),  GeLU(v) = v * Phi(v) (erf form),
 * for every row of the dispatched buffer, e being the expert that owns the row.
 * Needs shape->layout == LOCMOE_LAYOUT_RECV (the rows of one expert are the
 * contiguous block [e * D * C_alloc, (e + 1) * D * C_alloc)) and bf16 tokens.
 * Empty (zero) rows give zero rows.  Two grouped GEMMs on the tensor cores
 * (tcgen05, fp32 accumulation); the intermediate is rounded to bf16.
 *   buf   [D*E*C_alloc][H] bf16        w_in  [E][F][H] bf16      w_out [E][H][F] bf16
 *   h1    [D*E*C_alloc][F] bf16 scratch (caller's)               y [D*E*C_alloc][H] of y_dtype
 * H and F must be multiples of 8; all five pointers 16-byte aligned.
 */
int locmoe_expert_ffn(const locmoe_shape_t *shape, int32_t C_alloc, int32_t F, const void *buf,
                      const void *w_in, const void *w_out, void *h1, void *y, int32_t y_dtype,
                      void *stream);

/*
 * Host only, launches nothing: which kernel locmoe_expert_ffn would run each of
 * its two GEMMs with on the current device for this shape -- kernels[0] for
 * x W_in^T (+ GeLU), kernels[1] for g W_out^T.  The results do not depend on the
 * choice; a program may want to report it.
 */
enum { LOCMOE_FFN_TILE_128x256 = 0, LOCMOE_FFN_TILE_256x256 = 1, LOCMOE_FFN_TWO_SM = 2, LOCMOE_FFN_TWO_SM_SINGLE = 3 };
int locmoe_ffn_kernels(const locmoe_shape_t *shape, int32_t C_alloc, int32_t F, int32_t *kernels /* [2], host */);

/* Every device array of one MoE layer pass, for locmoe_moe_layer (host struct of device pointers;
 * sizes as documented at the individual calls). */
typedef struct {
    int32_t *idx; float *gate_w; float *cos_sim; float *delta_e; float *theta_e;
    locmoe_capacity_t *cap_dev;
    int32_t *pos; int32_t *slot; uint8_t *drop; int32_t *inv;
    int32_t *counts; int32_t *kept; int32_t *send_counts; int32_t *load; int64_t *locality; int32_t *status;
    void *ws; size_t ws_bytes;
    void *buf;   /* [D*E*C_alloc][H] of x_dtype                                   */
    void *h1;    /* [D*E*C_alloc][F] bf16, only with experts                      */
    void *y;     /* [D*E*C_alloc][H] bf16, only with experts                      */
} locmoe_layer_buffers_t;

/*
 * One whole MoE layer pass on one stream: gate -> capacity -> route -> dispatch ->
 * expert FFN -> combine (the six calls above, in order, nothing else).  With
 * w_in == NULL the experts are the identity and the dispatched buffer itself is
 * combined.  out [T][H] of x_dtype.  eps may be NULL.
 */
int locmoe_moe_layer(const locmoe_shape_t *shape, const void *x, const int32_t *src_dev, const float *eps,
                     const locmoe_capacity_rule_t *rule, int32_t C_alloc, int32_t F, const void *w_in,
                     const void *w_out, const locmoe_layer_buffers_t *bufs, void *out, void *stream);

/*
 * Host-side helpers of the capacity rule and the buffer layout: plain arithmetic
 * on host memory, nothing is launched.
 *
 * locmoe_conventional_capacity: the conventional term of the capacity rule,
 *   ec = ceil(b_s * c_f / (ep * n)) of Sec. 3.2.3 with b_s = the batch's tokens
 *   (rule->T_global if > 0, else shape->T), ep = D, at least 1 and at most b_s:
 *   the row stride a caller allocates the buffer with (C_alloc) when Theorem 1's
 *   minimum does not bind.  Rounded exactly as the device evaluates the rule.
 *
 * locmoe_batch_delta: the batch-wide cosine threshold from per-expert minima
 *   (delta_e as written by locmoe_capacity, copied to HOST memory, possibly
 *   already combined over ranks by an element-wise minimum): min over experts,
 *   clamped to [0, 1] as the device clamps it -- a negative minimum becomes 0, so
 *   that the value can be passed on as rule->delta_override, where "< 0" would
 *   mean "measure" (abstract; Lemma 3 uses delta^2).
 *
 * locmoe_dest_order: r(a, b) of the buffer layout, the position of logical
 *   device b in device a's list of destinations -- a itself, then the rest of
 *   a's node, then the other nodes cyclically (Sec. 3.2.4; abstract: inter-node
 *   traffic turned into intra-node).  Returns r >= 0, or LOCMOE_ERR_SHAPE.
 */
int locmoe_conventional_capacity(const locmoe_shape_t *shape, const locmoe_capacity_rule_t *rule,
                                 int32_t *C_alloc);
int locmoe_batch_delta(const float *delta_e_host, int32_t E, double *delta_host);
int locmoe_dest_order(const locmoe_shape_t *shape, int32_t a, int32_t b);

/* Kernels launched per call of gate, capacity, route, dispatch, combine on this
 * shape (counts[5], host memory); a bookkeeping aid for benchmarks.  The paper
 * has no counterpart. */
int locmoe_launch_counts(const locmoe_shape_t *shape, int32_t counts[5]);

/* Device-side diagnostics of this library on the current device, copied to host
 * memory after waiting for the stream: bit 0 is set if a kernel gave up a
 * bounded wait for one of its own asynchronous copies (its output is then
 * incomplete); bit 1 the same for the expert-FFN kernels.  0 in normal operation.
 * The paper has no counterpart. */
int locmoe_device_flags(int32_t *flags_host, void *stream);

/* Text for a return code of this library (host string, never NULL). */
const char *locmoe_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* LOCMOE_H */
