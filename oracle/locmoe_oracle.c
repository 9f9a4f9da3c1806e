/*
 * LocMoE router oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-threaded CPU statement of what the LocMoE router and
 * token dispatch compute, written from the paper (arXiv 2401.13920) and used
 * only to check the CUDA path and as the timed CPU baseline.  Every floating
 * point quantity is accumulated in IEEE double.  Nothing here is blocked,
 * fused, vectorised or re-ordered beyond what the cited definition states,
 * and nothing is shared with the CUDA sources.
 *
 * Stages (zero-based indices everywhere):
 *   oracle_gate      Sec. 3.2.1: G = ReLU(w_i . x + eps_i) with the fixed
 *                    grouped-average-pooling weight (the w_i formula), the
 *                    arg-max of softmax(G) (Eq. "max_expert") and the score
 *                    R = softmax(G)[i*] (Eq. "gating_score"); the cosine
 *                    between the token and the chosen gating weight
 *                    (Lemma 1 and its proof, Appendix A.1).
 *   oracle_p_delta   Lemma 3 / Appendix A.2: share of the unit sphere inside
 *                    the two symmetric caps |cos| >= delta.
 *   oracle_ec_min    Theorem 1: the three forms of the capacity lower bound.
 *   oracle_capacity  abstract (largest angle between an expert's gating weight
 *                    and the tokens routed to it), Theorem 1, and the
 *                    conventional rule ec = ceil(b_s c_f / (ep n)) of
 *                    Sec. 3.2.3.
 *   oracle_route     capacity-bounded first-come-first-served placement into
 *                    an All-to-All shaped buffer (Sec. 3.2.3 capacity limit,
 *                    Sec. 3.2.4 exchange, abstract: intra-node before
 *                    inter-node).
 *   oracle_dispatch  row copy into the buffer.
 *   oracle_combine   y_m = R_m * expert_out (first equation of Sec. 3.2.1,
 *                    top-1 so a single term; a dropped token has no term).
 *
 *   oracle_gate_topk, oracle_combine_topk
 *                    the same gate and the same sum of Sec. 3.2.1's first
 *                    equation with the k largest scores per token instead of
 *                    one (a variant: the paper itself routes top-1).
 *
 *   oracle_aux_loss  L_aux = alpha n sum_i f_i P_i (Sec. 3.2.2, first loss
 *                    equation), forward value.
 *   oracle_cos_hist  the two histograms of the second cosine-frequency figure of
 *                    Sec. 4.1: tokens routed to one expert, their cosine to that
 *                    expert's gating weight and to another expert's.
 *   oracle_loc_loss  L_loc = mu KL(D_c || D_l) (Sec. 3.2.2, second loss
 *                    equation), forward value, under the reading stated at
 *                    the function (the paper gives neither mu nor the
 *                    treatment of experts D_l gives no mass): the arithmetic
 *                    is pinned, the reading is not -- parity unpinned.
 *   oracle_ffn_rows  expert network of the same equation:
 *                    W_out . GeLU(W_in . x), GeLU(v) = v * Phi(v) with Phi the
 *                    standard Gaussian CDF (Sec. 3.2.1), in double.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py
 * (dense-weight identity, closed forms, library incomplete beta, brute force,
 * round trip).  oracle_loc_loss: its KL arithmetic is pinned (closed forms, a
 * library relative entropy), its reading of the paper's D_c / D_l is a choice:
 * PARITY UNPINNED for that function.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1

#define ORACLE_LAYOUT_SEND 0
#define ORACLE_LAYOUT_RECV 1

#define ORACLE_BOUND_BETA 0
#define ORACLE_BOUND_ERFC 1
#define ORACLE_BOUND_EXP 2

#define ORACLE_WARN_CLAMPED 1
#define ORACLE_WARN_BAD_SRC 2

#define ORACLE_FLAG_DELTA_OVERRIDE 1
#define ORACLE_FLAG_MIN_SATURATED 2
#define ORACLE_FLAG_MIN_BINDS 4

typedef struct {
    double min_mult;        /* multiplier on Theorem 1's minimum            */
    double capacity_factor; /* c_f of ec = ceil(b_s c_f / (ep n)); 0 = off  */
    double delta_override;  /* < 0: measure delta from the data             */
    int32_t bound_form;     /* ORACLE_BOUND_*                               */
} oracle_rule_t;

typedef struct {
    double delta, p_delta, ec_min;
    int32_t C_expert, C_local, n_empty_experts, flags;
} oracle_capacity_t;

/* Exact widening of one stored element to double. */
static double widen(const void *x, int dtype, int64_t i)
{
    if (dtype == ORACLE_F32) {
        return (double)((const float *)x)[i];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)x)[i]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* The GrAP weight written out literally: w[i][j] = (n/d) 1{ i d/n <= j < (i+1) d/n }.
 * Only used by tests to pin the grouped mean against a dense product. */
void oracle_grap_weight(int32_t n, int32_t d, double *w /* [n][d] */)
{
    for (int32_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d; ++j) {
            /* i d/n <= j < (i+1) d/n, in integers (n divides d) */
            int inside = ((int64_t)i * d <= (int64_t)j * n) && ((int64_t)j * n < (int64_t)(i + 1) * d);
            w[(int64_t)i * d + j] = inside ? (double)n / (double)d : 0.0;
        }
}

/*
 * Gate for tokens 0..T-1 of x[T][H].
 *   mean[i] = w_i . x      = (n/d) * sum of the i-th group of d/n entries
 *   G[i]    = max(mean[i] + eps[i], 0)
 *   idx     = lowest i attaining max_i softmax(G)_i  (softmax is monotone, so
 *             the lowest i attaining max G)
 *   R       = softmax(G)[idx] = 1 / sum_k exp(G[k] - G[idx])
 *   cos     = <w_idx, x> / (|w_idx| |x|), |w_i| = sqrt(n/d); 0 when |x| = 0
 *   gap     = largest G minus second largest G (0 when E == 1 is reported as +inf)
 * Optional outputs G_out[T][E], probs_out[T][E] may be NULL.
 * Returns 0, or -2 on a shape error.
 */
int oracle_gate(const void *x, int dtype, int64_t T, int32_t H, int32_t E, const float *eps,
                int32_t *idx, double *R, double *cosv, double *gap,
                double *G_out, double *probs_out)
{
    if (T < 0 || H <= 0 || E <= 0 || H % E != 0) return -2;
    const int32_t g = H / E;
    double *G = (double *)malloc(sizeof(double) * (size_t)E);
    double *mean = (double *)malloc(sizeof(double) * (size_t)E);
    if (!G || !mean) { free(G); free(mean); return -6; }
    for (int64_t t = 0; t < T; ++t) {
        double sq = 0.0;
        for (int32_t i = 0; i < E; ++i) {
            double s = 0.0;
            for (int32_t j = 0; j < g; ++j) {
                double v = widen(x, dtype, t * H + (int64_t)i * g + j);
                s += v;
                sq += v * v;
            }
            mean[i] = s * ((double)E / (double)H);
            double pre = mean[i] + (eps ? (double)eps[i] : 0.0);
            G[i] = pre > 0.0 ? pre : 0.0;
        }
        int32_t best = 0;
        for (int32_t i = 1; i < E; ++i)
            if (G[i] > G[best]) best = i;
        double second = -INFINITY;
        for (int32_t i = 0; i < E; ++i)
            if (i != best && G[i] > second) second = G[i];
        double denom = 0.0;
        for (int32_t i = 0; i < E; ++i) denom += exp(G[i] - G[best]);
        idx[t] = best;
        R[t] = 1.0 / denom;
        double nrm = sqrt(sq);
        double wnorm = sqrt((double)E / (double)H);
        cosv[t] = nrm > 0.0 ? mean[best] / (wnorm * nrm) : 0.0;
        gap[t] = (E > 1) ? G[best] - second : INFINITY;
        if (G_out)
            for (int32_t i = 0; i < E; ++i) G_out[t * E + i] = G[i];
        if (probs_out)
            for (int32_t i = 0; i < E; ++i) probs_out[t * E + i] = exp(G[i] - G[best]) / denom;
    }
    free(G);
    free(mean);
    return 0;
}

/*
 * p_delta of Lemma 3 by the cap-area argument of its proof (Appendix A.2):
 * the area of a cap of half-angle phi on the unit sphere in R^d is
 * A_{d-1} * integral_0^phi sin^{d-2}(theta) d theta, and p_delta is twice that
 * cap (phi = acos(delta)) over the whole sphere:
 *   p_delta = [2 Gamma(d/2) / (sqrt(pi) Gamma((d-1)/2))] * integral_0^{acos delta} sin^{d-2} theta d theta
 * which equals 1 - I_{delta^2}(1/2, (d-1)/2).  Composite Simpson rule.
 */
double oracle_p_delta(double delta, int32_t d)
{
    if (d < 2) return NAN;
    if (delta <= 0.0) return 1.0;
    if (delta >= 1.0) return 0.0;
    const double phi = acos(delta);
    const int64_t panels = 400000; /* even */
    const double h = phi / (double)panels;
    const double pw = (double)(d - 2);
    double acc = 0.0;
    for (int64_t k = 0; k <= panels; ++k) {
        double th = h * (double)k;
        double f = (d == 2) ? 1.0 : pow(sin(th), pw);
        double wgt = (k == 0 || k == panels) ? 1.0 : ((k & 1) ? 4.0 : 2.0);
        acc += wgt * f;
    }
    double integral = acc * h / 3.0;
    double lognorm = lgamma(0.5 * (double)d) - lgamma(0.5 * (double)(d - 1));
    double c = 2.0 / sqrt(M_PI) * exp(lognorm);
    return c * integral;
}

/*
 * Theorem 1: ec_min = 1 / (n p_delta)   (exact form), and the two large-d
 * forms with a = delta^2 d / (2 - delta^2):  1 / (n erfc(sqrt a)),  exp(a) / n.
 */
double oracle_ec_min(double delta, int32_t n, int32_t d, int32_t form)
{
    double a = delta * delta * (double)d / (2.0 - delta * delta);
    if (form == ORACLE_BOUND_ERFC) return 1.0 / ((double)n * erfc(sqrt(a)));
    if (form == ORACLE_BOUND_EXP) return exp(a) / (double)n;
    return 1.0 / ((double)n * oracle_p_delta(delta, d));
}

/*
 * Angular deviation and capacity.
 *   delta_e[e] = smallest cosine among the tokens routed to e (largest angle);
 *                1 for an expert with no token;  theta_e = acos(delta_e)
 *   delta      = min_e delta_e clamped to [0, 1], unless overridden
 *   ec_min     = Theorem 1 in the chosen form
 *   Cmin       = ceil(min(min_mult * ec_min, T))
 *   C_expert   = clamp(max(Cmin, ceil(c_f T / n), 1), 1, T)
 *   C_local    = clamp(max(ceil(Cmin / D), ceil(c_f T / (D n)), 1), 1, T)
 * where D = number of source devices (the "ep" of ec = ceil(b_s c_f/(ep n)),
 * with b_s = T).
 */
int oracle_capacity(const int32_t *idx, const double *cosv, int64_t T, int32_t E, int32_t d,
                    int32_t D, const oracle_rule_t *rule,
                    double *delta_e, double *theta_e, oracle_capacity_t *out)
{
    if (T <= 0 || E <= 0 || D <= 0 || d < 2) return -2;
    int32_t n_empty = 0;
    for (int32_t e = 0; e < E; ++e) delta_e[e] = INFINITY;
    for (int64_t t = 0; t < T; ++t) {
        int32_t e = idx[t];
        if (e < 0 || e >= E) return -2;
        if (cosv[t] < delta_e[e]) delta_e[e] = cosv[t];
    }
    double dmin = INFINITY;
    for (int32_t e = 0; e < E; ++e) {
        if (delta_e[e] == INFINITY) { delta_e[e] = 1.0; ++n_empty; }
        else if (delta_e[e] < dmin) dmin = delta_e[e];
        double c = delta_e[e] > 1.0 ? 1.0 : (delta_e[e] < -1.0 ? -1.0 : delta_e[e]);
        theta_e[e] = acos(c);
    }
    int32_t flags = 0;
    double delta = dmin < 0.0 ? 0.0 : (dmin > 1.0 ? 1.0 : dmin);
    if (rule->delta_override >= 0.0) {
        delta = rule->delta_override > 1.0 ? 1.0 : rule->delta_override;
        flags |= ORACLE_FLAG_DELTA_OVERRIDE;
    }
    double p = oracle_p_delta(delta, d);
    double ec = oracle_ec_min(delta, E, d, rule->bound_form);
    double m = rule->min_mult * ec;
    if (!(m < (double)T)) { m = (double)T; flags |= ORACLE_FLAG_MIN_SATURATED; }
    if (m < 0.0) m = 0.0;
    double Cmin = ceil(m);
    double cf = rule->capacity_factor;
    double conv_e = ceil(cf * (double)T / (double)E);
    double conv_l = ceil(cf * (double)T / ((double)D * (double)E));
    double ce = Cmin > conv_e ? Cmin : conv_e;
    double min_l = ceil(Cmin / (double)D);
    double cl = min_l > conv_l ? min_l : conv_l;
    if (min_l > conv_l) flags |= ORACLE_FLAG_MIN_BINDS;
    if (ce < 1.0) ce = 1.0;
    if (cl < 1.0) cl = 1.0;
    if (ce > (double)T) ce = (double)T;
    if (cl > (double)T) cl = (double)T;
    out->delta = delta;
    out->p_delta = p;
    out->ec_min = ec;
    out->C_expert = (int32_t)ce;
    out->C_local = (int32_t)cl;
    out->n_empty_experts = n_empty;
    out->flags = flags;
    return 0;
}

/* Destination rank seen from device a: itself first, then the rest of its own
 * node, then the other nodes in cyclic order ("intra-node first"). */
static int32_t dest_rank(int32_t a, int32_t b, int32_t N, int32_t Dn)
{
    int32_t dn = ((b / Dn - a / Dn) % N + N) % N;
    int32_t dl = ((b % Dn - a % Dn) % Dn + Dn) % Dn;
    return dn * Dn + dl;
}

void oracle_dest_order(int32_t N, int32_t Dn, int32_t *r /* [D][D] */)
{
    int32_t D = N * Dn;
    for (int32_t a = 0; a < D; ++a)
        for (int32_t b = 0; b < D; ++b) r[a * D + b] = dest_rank(a, b, N, Dn);
}

/* pos_t straight from its definition, O(T^2): how many earlier tokens share
 * both the source device and the chosen expert. */
void oracle_pos_bruteforce(const int32_t *idx, const int32_t *src, int64_t T, int32_t *pos)
{
    for (int64_t t = 0; t < T; ++t) {
        int32_t c = 0;
        for (int64_t u = 0; u < t; ++u)
            if (src[u] == src[t] && idx[u] == idx[t]) ++c;
        pos[t] = c;
    }
}

/*
 * Route.  E experts placed contiguously on D = N * Dn devices (Ed = E / D per
 * device).  Token t comes from device src[t] and goes to expert idx[t].
 *   pos[t]   = number of earlier tokens with the same (src, idx)
 *   drop[t]  = pos[t] >= C,  C = min(C_local, C_alloc)
 *   slot[t]  = row in the buffer (row stride C_alloc), -1 when dropped:
 *     SEND: ((src * D + r(src, dev(e))) * Ed + el) * C_alloc + pos
 *     RECV: ((dev(e) * Ed + el) * D + r(dev(e), src)) * C_alloc + pos
 *   inv[row] = t for an occupied row, else -1           [D * E * C_alloc]
 *   counts[s][e] raw demand, kept[s][e] = min(counts, C), load[e] = sum_s counts
 *   send_counts[s][b] = kept tokens from s to the experts of device b
 *   locality[0][c] raw / locality[1][c] kept token counts by class c:
 *     0 same device, 1 same node, 2 other node
 * A token whose src is outside [0, D) is dropped (pos = -1) and flagged.
 */
int oracle_route(const int32_t *idx, const int32_t *src, int64_t T, int32_t E, int32_t N, int32_t Dn,
                 int32_t C_local, int32_t C_alloc, int32_t layout,
                 int32_t *pos, int32_t *slot, uint8_t *drop, int32_t *inv,
                 int32_t *counts, int32_t *kept, int32_t *send_counts, int32_t *load,
                 int64_t *locality, int32_t *status)
{
    const int32_t D = N * Dn;
    if (T < 0 || E <= 0 || N <= 0 || Dn <= 0 || E % D != 0 || C_alloc <= 0 || C_local <= 0) return -2;
    const int32_t Ed = E / D;
    int32_t C = C_local;
    int32_t st = 0;
    if (C > C_alloc) { C = C_alloc; st |= ORACLE_WARN_CLAMPED; }
    const int64_t rows = (int64_t)D * E * C_alloc;
    for (int64_t r = 0; r < rows; ++r) inv[r] = -1;
    memset(counts, 0, sizeof(int32_t) * (size_t)D * E);
    memset(send_counts, 0, sizeof(int32_t) * (size_t)D * D);
    memset(load, 0, sizeof(int32_t) * (size_t)E);
    for (int i = 0; i < 6; ++i) locality[i] = 0;
    for (int64_t t = 0; t < T; ++t) {
        int32_t e = idx[t], s = src[t];
        if (e < 0 || e >= E) return -2;
        if (s < 0 || s >= D) {
            st |= ORACLE_WARN_BAD_SRC;
            pos[t] = -1; slot[t] = -1; drop[t] = 1;
            continue;
        }
        int32_t p = counts[s * E + e]++;
        load[e]++;
        int32_t b = e / Ed, el = e % Ed;
        int cls = (b == s) ? 0 : ((b / Dn == s / Dn) ? 1 : 2);
        locality[cls]++;
        pos[t] = p;
        if (p >= C) { drop[t] = 1; slot[t] = -1; continue; }
        drop[t] = 0;
        locality[3 + cls]++;
        send_counts[s * D + b]++;
        int64_t row;
        if (layout == ORACLE_LAYOUT_SEND)
            row = (((int64_t)s * D + dest_rank(s, b, N, Dn)) * Ed + el) * C_alloc + p;
        else
            row = (((int64_t)b * Ed + el) * D + dest_rank(b, s, N, Dn)) * C_alloc + p;
        slot[t] = (int32_t)row;
        inv[row] = (int32_t)t;
    }
    for (int64_t k = 0; k < (int64_t)D * E; ++k) kept[k] = counts[k] < C ? counts[k] : C;
    *status = st;
    return 0;
}

/* Dispatch: buf[slot[t]] = x[t] bit for bit; every other row zero. */
int oracle_dispatch(const void *x, int dtype, int64_t T, int32_t H, const int32_t *slot,
                    int64_t rows, void *buf)
{
    const size_t rb = (size_t)H * (dtype == ORACLE_F32 ? 4 : 2);
    memset(buf, 0, rb * (size_t)rows);
    for (int64_t t = 0; t < T; ++t) {
        if (slot[t] < 0) continue;
        if (slot[t] >= rows) return -2;
        memcpy((char *)buf + rb * (size_t)slot[t], (const char *)x + rb * (size_t)t, rb);
    }
    return 0;
}

/* Combine: out[t][j] = R[t] * y[slot[t]][j] (double), 0 for a dropped token;
 * with accumulate != 0 the product is added to prev[t][j] (prev in out dtype
 * semantics is the caller's business: prev is given in double). */
int oracle_combine(const void *y, int y_dtype, int64_t T, int32_t H, const int32_t *slot,
                   const double *R, const double *prev /* [T][H] or NULL */, double *out /* [T][H] */)
{
    for (int64_t t = 0; t < T; ++t)
        for (int32_t j = 0; j < H; ++j) {
            double v = 0.0;
            if (slot[t] >= 0) v = R[t] * widen(y, y_dtype, (int64_t)slot[t] * H + j);
            if (prev) v += prev[t * H + j];
            out[t * H + j] = v;
        }
    return 0;
}

/*
 * Expert FFN on `nrows` rows that all belong to one expert (first equation of Sec. 3.2.1):
 *   h[f] = sum_j W_in[f][j] x[j],   g[f] = h[f] * Phi(h[f]) = 0.5 h[f] (1 + erf(h[f] / sqrt 2)),
 *   y[i] = sum_f W_out[i][f] g[f].
 * x [nrows][H], w_in [F][H], w_out [H][F] are bf16 bit patterns, widened exactly; everything in double.
 * y [nrows][H].  spread [nrows][H] (may be NULL) receives sqrt(sum_f (W_out[i][f] g[f])^2): the tests derive
 * from it how far a result whose intermediate g was rounded to bf16 may lie from y.
 */
int oracle_ffn_rows(const uint16_t *x, int64_t nrows, int32_t H, int32_t F, const uint16_t *w_in,
                    const uint16_t *w_out, double *y, double *spread)
{
    double *g = (double *)malloc(sizeof(double) * (size_t)F);
    if (!g) return -6;
    for (int64_t r = 0; r < nrows; ++r) {
        for (int32_t f = 0; f < F; ++f) {
            double h = 0.0;
            for (int32_t j = 0; j < H; ++j)
                h += widen(w_in, ORACLE_BF16, (int64_t)f * H + j) * widen(x, ORACLE_BF16, r * H + j);
            g[f] = 0.5 * h * (1.0 + erf(h / sqrt(2.0)));
        }
        for (int32_t i = 0; i < H; ++i) {
            double acc = 0.0, sq = 0.0;
            for (int32_t f = 0; f < F; ++f) {
                double term = widen(w_out, ORACLE_BF16, (int64_t)i * F + f) * g[f];
                acc += term;
                sq += term * term;
            }
            y[r * H + i] = acc;
            if (spread) spread[r * H + i] = sqrt(sq);
        }
    }
    free(g);
    return 0;
}

/*
 * Auxiliary loss (Sec. 3.2.2): f_i = share of tokens whose arg-max is expert i, P_i = mean over tokens of
 * p_i(x) (the softmax of the gate logits), L_aux = alpha * n * sum_i f_i P_i.  probs [T][E] in double.
 */
double oracle_aux_loss(const int32_t *idx, const double *probs, int64_t T, int32_t E, double alpha,
                       double *f /* [E] */, double *P /* [E] */)
{
    for (int32_t i = 0; i < E; ++i) { f[i] = 0.0; P[i] = 0.0; }
    for (int64_t t = 0; t < T; ++t) {
        f[idx[t]] += 1.0;
        for (int32_t i = 0; i < E; ++i) P[i] += probs[t * E + i];
    }
    double s = 0.0;
    for (int32_t i = 0; i < E; ++i) {
        f[i] /= (double)T;
        P[i] /= (double)T;
        s += f[i] * P[i];
    }
    return alpha * (double)E * s;
}

/*
 * Locality loss (Sec. 3.2.2, second loss equation): L_loc = mu * KL(D_c || D_l), D_c the current assignment
 * distribution, D_l the fully localised one.  The paper defines neither distribution in symbols; the reading here:
 * both are joint distributions over (source group s, expert e) pairs, a group being a logical device (level 0) or
 * a logical node (level 1) and G their number;
 *   D_c(s, e) = counts[s][e] / T_routed                       (what the batch did),
 *   D_l(s, e) = (n_s / T_routed) * q_s(e)                     (same sources, every token on a local expert),
 *   q_s(e)    = (1 - smooth) / (E / G) on the E / G experts group s hosts, + smooth / E on every expert
 * (smooth > 0 keeps the divergence finite when a token leaves its group).  Then
 *   KL(D_c || D_l) = sum_s (n_s / T_routed) * KL_s,   KL_s = sum_e c_s(e) ln(c_s(e) / q_s(e)),  c_s = counts[s] / n_s,
 * with 0 ln 0 = 0 and a group without tokens contributing nothing.
 * counts [D][E] demanded tokens per (source device, expert); experts are laid out in blocks of E / D per device,
 * devices in blocks of Dn per node.  dc [G][E] receives c_s, kl [G] receives KL_s.  Returns L_loc.
 */
double oracle_loc_loss(const int32_t *counts, int32_t E, int32_t N, int32_t Dn, int32_t level, double mu,
                       double smooth, double *dc /* [G][E] */, double *kl /* [G] */)
{
    const int32_t D = N * Dn, G = level ? N : D, per = D / G, Eg = E / G;
    double total = 0.0, acc = 0.0;
    for (int32_t s = 0; s < G; ++s)
        for (int32_t m = 0; m < per; ++m)
            for (int32_t e = 0; e < E; ++e) total += (double)counts[(s * per + m) * E + e];
    for (int32_t s = 0; s < G; ++s) {
        double ns = 0.0;
        for (int32_t e = 0; e < E; ++e) {
            double c = 0.0;
            for (int32_t m = 0; m < per; ++m) c += (double)counts[(s * per + m) * E + e];
            dc[s * E + e] = c;
            ns += c;
        }
        double k = 0.0;
        for (int32_t e = 0; e < E; ++e) {
            const double c = ns > 0.0 ? dc[s * E + e] / ns : 0.0;
            const int local = e / Eg == s;
            const double q = (local ? (1.0 - smooth) / (double)Eg : 0.0) + smooth / (double)E;
            dc[s * E + e] = c;
            if (c > 0.0) k += c * log(c / q);
        }
        kl[s] = k;
        if (total > 0.0) acc += ns / total * k;
    }
    return mu * acc;
}

/*
 * Cosine-frequency diagnostic (Sec. 4.1, second cosine-histogram figure): over the tokens routed to expert e,
 * the histogram of cos(x, w_e) (the expert the token went to) and the histogram of cos(x, w_j) for another
 * expert j, with w_i the i-th gating weight (1 on the i-th group of d/n entries, scaled; the scale cancels):
 *   cos(x, w_i) = (sum of the i-th group of x) / (sqrt(d/n) * |x|),   0 when |x| = 0.
 * nbins equal bins on [lo, hi); a value below lo counts in the first bin, a value >= hi in the last.
 * Optional per-token outputs cos_e[T], cos_j[T] (NaN for tokens not routed to e) may be NULL.
 * Returns the number of tokens routed to e, or -2 on a bad argument.
 */
int64_t oracle_cos_hist(const void *x, int dtype, int64_t T, int32_t H, int32_t E, const int32_t *idx, int32_t e,
                        int32_t j, int32_t nbins, double lo, double hi, int64_t *hist_e, int64_t *hist_j,
                        double *cos_e, double *cos_j)
{
    if (H <= 0 || E <= 0 || H % E != 0 || e < 0 || e >= E || j < 0 || j >= E || nbins < 1 || !(hi > lo)) return -2;
    const int32_t g = H / E;
    int64_t n = 0;
    for (int32_t b = 0; b < nbins; ++b) { hist_e[b] = 0; hist_j[b] = 0; }
    for (int64_t t = 0; t < T; ++t) {
        if (cos_e) cos_e[t] = NAN;
        if (cos_j) cos_j[t] = NAN;
        if (idx[t] != e) continue;
        double sq = 0.0, se = 0.0, sj = 0.0;
        for (int32_t k = 0; k < H; ++k) {
            const double v = widen(x, dtype, t * H + k);
            sq += v * v;
            if (k / g == e) se += v;
            if (k / g == j) sj += v;
        }
        const double den = sqrt((double)g) * sqrt(sq);
        const double c[2] = { den > 0.0 ? se / den : 0.0, den > 0.0 ? sj / den : 0.0 };
        int64_t *h[2] = { hist_e, hist_j };
        for (int q = 0; q < 2; ++q) {
            double pos = floor((c[q] - lo) / (hi - lo) * (double)nbins);
            if (pos < 0.0) pos = 0.0;
            if (pos > (double)(nbins - 1)) pos = (double)(nbins - 1);
            h[q][(int32_t)pos] += 1;
        }
        if (cos_e) cos_e[t] = c[0];
        if (cos_j) cos_j[t] = c[1];
        ++n;
    }
    return n;
}

/*
 * Top-k variant of the gate (the paper routes every token to its single best expert; Sec. 2 describes top-k
 * routers as the family it departs from).  Same logits as oracle_gate: G[i] = max(mean_i + eps_i, 0).  The K
 * experts with the largest G are taken in descending order of G, a tie going to the lower index; the score of a
 * chosen expert is its softmax value R = exp(G_i) / sum_k exp(G_k) (not renormalised over the chosen ones), so
 * that y_m = sum over the chosen experts of R * expert(x) is the first equation of Sec. 3.2.1 restricted to them.
 *   idx_k[j][t], R_k[j][t]  j-th choice of token t (j = 0 is oracle_gate's idx and R)
 *   gap[t]                  smallest difference between consecutive logits among the K + 1 largest (how close the
 *                           choice, or the order of the choices, is to a tie); +inf when E == K == 1
 * Returns 0, or -2 on a bad argument.
 */
int oracle_gate_topk(const void *x, int dtype, int64_t T, int32_t H, int32_t E, const float *eps, int32_t K,
                     int32_t *idx_k /* [K][T] */, double *R_k /* [K][T] */, double *gap /* [T] */)
{
    if (T < 0 || H <= 0 || E <= 0 || H % E != 0 || K < 1 || K > E) return -2;
    const int32_t g = H / E;
    double *G = (double *)malloc(sizeof(double) * (size_t)E);
    char *taken = (char *)malloc((size_t)E);
    if (!G || !taken) { free(G); free(taken); return -6; }
    for (int64_t t = 0; t < T; ++t) {
        for (int32_t i = 0; i < E; ++i) {
            double s = 0.0;
            for (int32_t j = 0; j < g; ++j) s += widen(x, dtype, t * H + (int64_t)i * g + j);
            const double pre = s * ((double)E / (double)H) + (eps ? (double)eps[i] : 0.0);
            G[i] = pre > 0.0 ? pre : 0.0;
            taken[i] = 0;
        }
        double gmax = G[0];
        for (int32_t i = 1; i < E; ++i) if (G[i] > gmax) gmax = G[i];
        double denom = 0.0;
        for (int32_t i = 0; i < E; ++i) denom += exp(G[i] - gmax);
        double prev = 0.0, mingap = INFINITY;
        for (int32_t j = 0; j <= K && j < E; ++j) {       /* one more than K: the best expert left out */
            int32_t best = -1;
            for (int32_t i = 0; i < E; ++i)
                if (!taken[i] && (best < 0 || G[i] > G[best])) best = i;
            taken[best] = 1;
            if (j > 0 && prev - G[best] < mingap) mingap = prev - G[best];
            prev = G[best];
            if (j < K) {
                idx_k[(int64_t)j * T + t] = best;
                R_k[(int64_t)j * T + t] = exp(G[best] - gmax) / denom;
            }
        }
        gap[t] = mingap;
    }
    free(G);
    free(taken);
    return 0;
}

/* Combine of the top-k variant: out[t][j] = sum over the K choices c of R_k[c][t] * y[slot_k[c][t]][j] (double);
 * a dropped choice (slot < 0) has no term. */
int oracle_combine_topk(const void *y, int y_dtype, int64_t T, int32_t H, int32_t K, const int32_t *slot_k /* [K][T] */,
                        const double *R_k /* [K][T] */, double *out /* [T][H] */)
{
    for (int64_t t = 0; t < T; ++t)
        for (int32_t j = 0; j < H; ++j) {
            double v = 0.0;
            for (int32_t c = 0; c < K; ++c) {
                const int32_t sl = slot_k[(int64_t)c * T + t];
                if (sl >= 0) v += R_k[(int64_t)c * T + t] * widen(y, y_dtype, (int64_t)sl * H + j);
            }
            out[t * H + j] = v;
        }
    return 0;
}
