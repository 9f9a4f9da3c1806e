// C-ABI front end: argument validation on the host, then the kernel launchers.
#include <math.h>
#include <stdlib.h>

#include "common.cuh"

namespace locmoe {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return kNumSMsB200; }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = kNumSMsB200;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

bool pdl_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("LOCMOE_PDL"); v = (e && e[0] == '0') ? 0 : 1; }
    return v != 0;
}

namespace {

int check_shape(const locmoe_shape_t* s) {
    if (!s) return LOCMOE_ERR_NULL;
    if (s->T < 1 || s->H < 1 || s->E < 1 || s->n_nodes < 1 || s->dev_per_node < 1) return LOCMOE_ERR_SHAPE;
    if (s->H % s->E != 0) return LOCMOE_ERR_SHAPE;
    const long long D = (long long)s->n_nodes * s->dev_per_node;
    if (D > s->E || s->E % D != 0) return LOCMOE_ERR_SHAPE;
    if (D * s->E > 0x7fffffffll) return LOCMOE_ERR_SHAPE;
    if (s->x_dtype != LOCMOE_F32 && s->x_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    if (s->layout != LOCMOE_LAYOUT_SEND && s->layout != LOCMOE_LAYOUT_RECV) return LOCMOE_ERR_DTYPE;
    return LOCMOE_OK;
}

// Rows of the buffer for row stride C_alloc, or -1 if they do not fit an int32 row index.
long long buffer_rows(const locmoe_shape_t* s, int32_t C_alloc) {
    if (C_alloc < 1) return -1;
    const long long K = (long long)s->n_nodes * s->dev_per_node * s->E;
    const long long rows = K * C_alloc;
    return rows > 0x7fffffffll ? -1 : rows;
}

}  // namespace
}  // namespace locmoe

using namespace locmoe;

extern "C" {

int locmoe_workspace_bytes(const locmoe_shape_t* shape, int32_t C_alloc, size_t* bytes) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!bytes) return LOCMOE_ERR_NULL;
    if (buffer_rows(shape, C_alloc) < 0) return LOCMOE_ERR_SHAPE;
    RoutePlan p;
    if ((rc = plan_route(*shape, &p))) return rc;
    size_t c = capacity_ws_bytes(*shape);
    const size_t x = aux_ws_bytes(*shape);
    if (x > c) c = x;
    *bytes = p.total > c ? p.total : c;
    return LOCMOE_OK;
}

int locmoe_gate(const locmoe_shape_t* shape, const void* x, const float* eps, int32_t* idx, float* gate_w,
                float* cos_sim, float* probs, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !idx || !gate_w || !cos_sim) return LOCMOE_ERR_NULL;
    const int esz = shape->x_dtype == LOCMOE_F32 ? 4 : 2;
    if ((uintptr_t)x % esz) return LOCMOE_ERR_ALIGN;
    return launch_gate(*shape, x, eps, idx, gate_w, cos_sim, probs, static_cast<cudaStream_t>(stream));
}

int locmoe_gate_ex(const locmoe_shape_t* shape, const void* x, locmoe_gate_opts_t* opts, int32_t* idx, float* gate_w,
                   float* cos_sim, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !opts || !idx || !gate_w || !cos_sim) return LOCMOE_ERR_NULL;
    const int esz = shape->x_dtype == LOCMOE_F32 ? 4 : 2;
    if ((uintptr_t)x % esz) return LOCMOE_ERR_ALIGN;
    if (opts->src_dev && !opts->eps) return LOCMOE_ERR_NULL;   // a table is asked for but not given
    const GateExtra extra{opts->eps ? opts->src_dev : nullptr, opts->p_part};
    opts->p_rows = 0;
    rc = launch_gate(*shape, x, opts->eps, idx, gate_w, cos_sim, opts->probs, static_cast<cudaStream_t>(stream), nullptr, &extra);
    if (rc == LOCMOE_OK && opts->p_part) opts->p_rows = gate_last_grid();
    return rc;
}

int locmoe_aux_loss_partial(const locmoe_shape_t* shape, const float* p_part, int32_t p_rows, const int32_t* load,
                            float alpha, float* f_out, float* p_out, float* loss_out, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!p_part || !load || !f_out || !p_out || !loss_out) return LOCMOE_ERR_NULL;
    if (p_rows < 1 || p_rows > LOCMOE_GATE_PARTIAL_ROWS) return LOCMOE_ERR_SHAPE;
    return launch_aux_from_partials(*shape, p_part, p_rows, load, alpha, f_out, p_out, loss_out, static_cast<cudaStream_t>(stream));
}

int locmoe_capacity(const locmoe_shape_t* shape, const int32_t* idx, const float* cos_sim,
                    const locmoe_capacity_rule_t* rule, float* delta_e, float* theta_e, locmoe_capacity_t* cap_dev,
                    void* ws, size_t ws_bytes, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!idx || !cos_sim || !rule || !delta_e || !theta_e || !cap_dev) return LOCMOE_ERR_NULL;
    if (shape->H < 2) return LOCMOE_ERR_SHAPE;
    if (rule->bound_form < LOCMOE_BOUND_BETA || rule->bound_form > LOCMOE_BOUND_EXP) return LOCMOE_ERR_DTYPE;
    if (rule->T_global < 0) return LOCMOE_ERR_SHAPE;
    if (!(rule->min_mult >= 0.0) || !(rule->capacity_factor >= 0.0) || rule->delta_override != rule->delta_override)
        return LOCMOE_ERR_SHAPE;
    if (!ws || ws_bytes < capacity_ws_bytes(*shape) || (uintptr_t)ws % 256) return LOCMOE_ERR_WORKSPACE;
    if ((uintptr_t)cap_dev % 8) return LOCMOE_ERR_ALIGN;
    return launch_capacity(*shape, idx, cos_sim, *rule, delta_e, theta_e, cap_dev, ws, static_cast<cudaStream_t>(stream));
}

int locmoe_capacity_read(const locmoe_capacity_t* cap_dev, locmoe_capacity_t* cap_host, void* stream) {
    if (!cap_dev || !cap_host) return LOCMOE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(cap_host, cap_dev, sizeof(locmoe_capacity_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return LOCMOE_ERR_CUDA;
    }
    return LOCMOE_OK;
}

int locmoe_route(const locmoe_shape_t* shape, const int32_t* idx, const int32_t* src_dev,
                 const locmoe_capacity_t* cap_dev, int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop,
                 int32_t* inv, int32_t* counts, int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality,
                 int32_t* status, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!idx || !src_dev || !cap_dev || !pos || !slot || !drop || !inv || !counts || !kept || !send_counts || !load ||
        !locality || !status)
        return LOCMOE_ERR_NULL;
    if (buffer_rows(shape, C_alloc) < 0) return LOCMOE_ERR_SHAPE;
    RoutePlan p;
    if ((rc = plan_route(*shape, &p))) return rc;
    if (!ws || ws_bytes < p.total || (uintptr_t)ws % 256) return LOCMOE_ERR_WORKSPACE;
    if ((uintptr_t)locality % 8 || (uintptr_t)cap_dev % 8) return LOCMOE_ERR_ALIGN;
    return launch_route(*shape, idx, src_dev, cap_dev, C_alloc, pos, slot, drop, inv, counts, kept, send_counts, load,
                        locality, status, ws, static_cast<cudaStream_t>(stream));
}

int locmoe_capacity_route(const locmoe_shape_t* shape, const int32_t* idx, const float* cos_sim, const int32_t* src_dev,
                          const locmoe_capacity_rule_t* rule, float* delta_e, float* theta_e, locmoe_capacity_t* cap_dev,
                          int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                          int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                          int32_t flags, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!idx || !cos_sim || !src_dev || !rule || !delta_e || !theta_e || !cap_dev || !pos || !slot || !drop || !inv ||
        !counts || !kept || !send_counts || !load || !locality || !status)
        return LOCMOE_ERR_NULL;
    if (shape->H < 2) return LOCMOE_ERR_SHAPE;
    if (rule->bound_form < LOCMOE_BOUND_BETA || rule->bound_form > LOCMOE_BOUND_EXP) return LOCMOE_ERR_DTYPE;
    if (rule->T_global < 0) return LOCMOE_ERR_SHAPE;
    if (!(rule->min_mult >= 0.0) || !(rule->capacity_factor >= 0.0) || rule->delta_override != rule->delta_override)
        return LOCMOE_ERR_SHAPE;
    if (buffer_rows(shape, C_alloc) < 0) return LOCMOE_ERR_SHAPE;
    if (flags & ~LOCMOE_ROUTE_EARLY_INIT) return LOCMOE_ERR_DTYPE;
    RoutePlan p;
    if ((rc = plan_route(*shape, &p))) return rc;
    size_t need = p.total;
    if (capacity_ws_bytes(*shape) > need) need = capacity_ws_bytes(*shape);
    if (!ws || ws_bytes < need || (uintptr_t)ws % 256) return LOCMOE_ERR_WORKSPACE;
    if ((uintptr_t)locality % 8 || (uintptr_t)cap_dev % 8) return LOCMOE_ERR_ALIGN;
    return launch_capacity_route(*shape, idx, cos_sim, src_dev, *rule, delta_e, theta_e, cap_dev, C_alloc, pos, slot, drop,
                                 inv, counts, kept, send_counts, load, locality, status,
                                 (flags & LOCMOE_ROUTE_EARLY_INIT) ? 1 : 0, ws, static_cast<cudaStream_t>(stream));
}

int locmoe_gate_route(const locmoe_shape_t* shape, const void* x, const float* eps, const int32_t* src_dev,
                      const locmoe_capacity_rule_t* rule, int32_t* idx, float* gate_w, float* cos_sim, float* delta_e,
                      float* theta_e, locmoe_capacity_t* cap_dev, int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop,
                      int32_t* inv, int32_t* counts, int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality,
                      int32_t* status, int32_t flags, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !src_dev || !rule || !idx || !gate_w || !cos_sim || !delta_e || !theta_e || !cap_dev || !pos || !slot || !drop ||
        !inv || !counts || !kept || !send_counts || !load || !locality || !status)
        return LOCMOE_ERR_NULL;
    if (shape->H < 2) return LOCMOE_ERR_SHAPE;
    const int esz = shape->x_dtype == LOCMOE_F32 ? 4 : 2;
    if ((uintptr_t)x % esz) return LOCMOE_ERR_ALIGN;
    if (rule->bound_form < LOCMOE_BOUND_BETA || rule->bound_form > LOCMOE_BOUND_EXP) return LOCMOE_ERR_DTYPE;
    if (rule->T_global < 0) return LOCMOE_ERR_SHAPE;
    if (!(rule->min_mult >= 0.0) || !(rule->capacity_factor >= 0.0) || rule->delta_override != rule->delta_override)
        return LOCMOE_ERR_SHAPE;
    if (buffer_rows(shape, C_alloc) < 0) return LOCMOE_ERR_SHAPE;
    if (flags & ~LOCMOE_ROUTE_EARLY_INIT) return LOCMOE_ERR_DTYPE;
    RoutePlan p;
    if ((rc = plan_route(*shape, &p))) return rc;
    if (!ws || ws_bytes < p.total || (uintptr_t)ws % 256) return LOCMOE_ERR_WORKSPACE;
    if ((uintptr_t)locality % 8 || (uintptr_t)cap_dev % 8) return LOCMOE_ERR_ALIGN;
    return launch_gate_route(*shape, x, eps, src_dev, *rule, idx, gate_w, cos_sim, delta_e, theta_e, cap_dev, C_alloc, pos, slot,
                             drop, inv, counts, kept, send_counts, load, locality, status,
                             (flags & LOCMOE_ROUTE_EARLY_INIT) ? 1 : 0, ws, static_cast<cudaStream_t>(stream));
}

int locmoe_dispatch(const locmoe_shape_t* shape, int32_t C_alloc, const void* x, const int32_t* inv,
                    const int32_t* slot, void* buf, int32_t zero_pad, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !inv || !buf) return LOCMOE_ERR_NULL;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    const int esz = shape->x_dtype == LOCMOE_F32 ? 4 : 2;
    if ((uintptr_t)x % esz || (uintptr_t)buf % esz) return LOCMOE_ERR_ALIGN;
    return launch_dispatch(*shape, rows, x, inv, slot, buf, zero_pad, static_cast<cudaStream_t>(stream));
}

int locmoe_combine(const locmoe_shape_t* shape, int32_t C_alloc, const void* y, int32_t y_dtype, const int32_t* slot,
                   const float* gate_w, void* out, int32_t accumulate, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!y || !slot || !gate_w || !out) return LOCMOE_ERR_NULL;
    if (y_dtype != LOCMOE_F32 && y_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    if ((uintptr_t)y % (y_dtype == LOCMOE_F32 ? 4 : 2) || (uintptr_t)out % (shape->x_dtype == LOCMOE_F32 ? 4 : 2))
        return LOCMOE_ERR_ALIGN;
    return launch_combine(*shape, rows, y, y_dtype, slot, gate_w, out, accumulate, static_cast<cudaStream_t>(stream));
}

int locmoe_aux_loss(const locmoe_shape_t* shape, const float* probs, const int32_t* load, float alpha, float* f_out,
                    float* p_out, float* loss_out, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!probs || !load || !f_out || !p_out || !loss_out) return LOCMOE_ERR_NULL;
    if (!ws || ws_bytes < aux_ws_bytes(*shape) || (uintptr_t)ws % 256) return LOCMOE_ERR_WORKSPACE;
    return launch_aux_loss(*shape, probs, load, alpha, f_out, p_out, loss_out, ws, static_cast<cudaStream_t>(stream));
}

int locmoe_loc_loss(const locmoe_shape_t* shape, const int32_t* counts, int32_t level, double mu, double smooth,
                    float* dc_out, double* kl_out, int64_t* group_tokens, double* loss_out, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!counts || !dc_out || !kl_out || !group_tokens || !loss_out) return LOCMOE_ERR_NULL;
    if (level != 0 && level != 1) return LOCMOE_ERR_DTYPE;
    if (!(smooth >= 0.0 && smooth <= 1.0)) return LOCMOE_ERR_SHAPE;
    if ((uintptr_t)kl_out % 8 || (uintptr_t)group_tokens % 8 || (uintptr_t)loss_out % 8) return LOCMOE_ERR_ALIGN;
    return launch_loc_loss(*shape, counts, level, mu, smooth, dc_out, kl_out, reinterpret_cast<long long*>(group_tokens),
                           loss_out, static_cast<cudaStream_t>(stream));
}

int locmoe_cos_hist(const locmoe_shape_t* shape, const void* x, const int32_t* idx, int32_t expert, int32_t other,
                    int32_t nbins, float lo, float hi, int32_t* hist_routed, int32_t* hist_other, int32_t* n_routed,
                    void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !idx || !hist_routed || !hist_other || !n_routed) return LOCMOE_ERR_NULL;
    if (expert < 0 || expert >= shape->E || other < 0 || other >= shape->E || nbins < 1 || !(hi > lo)) return LOCMOE_ERR_SHAPE;
    const int esz = shape->x_dtype == LOCMOE_F32 ? 4 : 2;
    if ((uintptr_t)x % esz) return LOCMOE_ERR_ALIGN;
    return launch_cos_hist(*shape, x, idx, expert, other, nbins, lo, hi, hist_routed, hist_other, n_routed,
                           static_cast<cudaStream_t>(stream));
}

namespace {
// Shared checks of the two peer calls: receive-side layout, experts split evenly over at most 64 peers.
int check_peers(const locmoe_shape_t* shape, void* const* peers, int32_t n_peers) {
    if (!peers) return LOCMOE_ERR_NULL;
    if (shape->layout != LOCMOE_LAYOUT_RECV) return LOCMOE_ERR_DTYPE;
    const int D = shape->n_nodes * shape->dev_per_node;
    if (n_peers < 1 || n_peers > 64 || D % n_peers != 0) return LOCMOE_ERR_SHAPE;
    for (int q = 0; q < n_peers; ++q) {
        if (!peers[q]) return LOCMOE_ERR_NULL;
        if ((uintptr_t)peers[q] % 16) return LOCMOE_ERR_ALIGN;
    }
    return LOCMOE_OK;
}
}  // namespace

int locmoe_dispatch_peer(const locmoe_shape_t* shape, int32_t C_alloc, const void* x, const int32_t* inv,
                         const int32_t* slot, void* const* peer_bufs, int32_t n_peers, int32_t src_lo, int32_t src_hi,
                         int32_t zero_pad, void* stream) {
    return locmoe_dispatch_peer_window(shape, C_alloc, x, inv, slot, peer_bufs, n_peers, src_lo, src_hi, zero_pad, 0,
                                       INT64_MAX, stream);
}

int locmoe_dispatch_peer_window(const locmoe_shape_t* shape, int32_t C_alloc, const void* x, const int32_t* inv,
                                const int32_t* slot, void* const* peer_bufs, int32_t n_peers, int32_t src_lo, int32_t src_hi,
                                int32_t zero_pad, int64_t win_lo, int64_t win_hi, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!x || !inv || !slot) return LOCMOE_ERR_NULL;
    if ((rc = check_peers(shape, peer_bufs, n_peers))) return rc;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    const int D = shape->n_nodes * shape->dev_per_node;
    if (src_lo < 0 || src_hi > D || src_lo > src_hi) return LOCMOE_ERR_SHAPE;
    const size_t rb = (size_t)shape->H * (shape->x_dtype == LOCMOE_F32 ? 4 : 2);
    if (rb % 16 || (uintptr_t)x % 16) return LOCMOE_ERR_ALIGN;
    if ((unsigned long long)shape->T * (rb / 16) >= 0xf0000000ull) return LOCMOE_ERR_SHAPE;
    if (win_lo < 0 || win_hi < win_lo) return LOCMOE_ERR_SHAPE;
    return launch_dispatch_peer(*shape, C_alloc, rows, x, inv, slot, peer_bufs, n_peers, src_lo, src_hi, zero_pad,
                                (long long)win_lo, (long long)win_hi, static_cast<cudaStream_t>(stream));
}

int locmoe_combine_peer(const locmoe_shape_t* shape, int32_t C_alloc, void* const* peer_y, int32_t n_peers, int32_t y_dtype,
                        const int32_t* slot, const float* gate_w, void* out, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!slot || !gate_w || !out) return LOCMOE_ERR_NULL;
    if (y_dtype != LOCMOE_F32 && y_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    if ((rc = check_peers(shape, peer_y, n_peers))) return rc;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    if (shape->H % 8 || (uintptr_t)out % 16) return LOCMOE_ERR_ALIGN;
    return launch_combine_peer(*shape, rows, peer_y, n_peers, y_dtype, slot, gate_w, out, static_cast<cudaStream_t>(stream));
}

int locmoe_topk_select(const locmoe_shape_t* shape, const float* probs, const int32_t* idx, const float* gate_w, int32_t K,
                       int32_t* idx_k, float* w_k, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!probs || !idx || !gate_w || !idx_k || !w_k) return LOCMOE_ERR_NULL;
    if (K < 1 || K > 8 || K > shape->E) return LOCMOE_ERR_SHAPE;
    return launch_topk_select(*shape, probs, idx, gate_w, K, idx_k, w_k, static_cast<cudaStream_t>(stream));
}

int locmoe_topk_fold(const locmoe_shape_t* shape, int32_t C_alloc, int32_t* inv, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!inv) return LOCMOE_ERR_NULL;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    return launch_topk_fold(shape->T, rows, inv, static_cast<cudaStream_t>(stream));
}

int locmoe_combine_topk(const locmoe_shape_t* shape, int32_t C_alloc, const void* y, int32_t y_dtype, int32_t K,
                        const int32_t* slot_k, const float* w_k, void* out, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!y || !slot_k || !w_k || !out) return LOCMOE_ERR_NULL;
    if (y_dtype != LOCMOE_F32 && y_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    if (K < 1 || K > 8) return LOCMOE_ERR_SHAPE;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    if (shape->H % 8 || (uintptr_t)y % 16 || (uintptr_t)out % 16) return LOCMOE_ERR_ALIGN;
    return launch_combine_topk(*shape, rows, y, y_dtype, K, slot_k, w_k, out, static_cast<cudaStream_t>(stream));
}

int locmoe_expert_ffn(const locmoe_shape_t* shape, int32_t C_alloc, int32_t F, const void* buf, const void* w_in,
                      const void* w_out, void* h1, void* y, int32_t y_dtype, void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!buf || !w_in || !w_out || !h1 || !y) return LOCMOE_ERR_NULL;
    if (shape->layout != LOCMOE_LAYOUT_RECV || shape->x_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    if (y_dtype != LOCMOE_F32 && y_dtype != LOCMOE_BF16) return LOCMOE_ERR_DTYPE;
    if (F < 8 || F % 8 != 0 || shape->H % 8 != 0) return LOCMOE_ERR_SHAPE;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    if ((uintptr_t)buf % 16 || (uintptr_t)w_in % 16 || (uintptr_t)w_out % 16 || (uintptr_t)h1 % 16 || (uintptr_t)y % 16)
        return LOCMOE_ERR_ALIGN;
    return launch_expert_ffn(*shape, rows, F, buf, w_in, w_out, h1, y, y_dtype, static_cast<cudaStream_t>(stream));
}

int locmoe_ffn_kernels(const locmoe_shape_t* shape, int32_t C_alloc, int32_t F, int32_t* kernels) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!kernels) return LOCMOE_ERR_NULL;
    if (F < 8 || F % 8 != 0 || shape->H % 8 != 0) return LOCMOE_ERR_SHAPE;
    const long long rows = buffer_rows(shape, C_alloc);
    if (rows < 0) return LOCMOE_ERR_SHAPE;
    int k[2];
    plan_expert_ffn(*shape, rows, F, k);
    kernels[0] = k[0];
    kernels[1] = k[1];
    return LOCMOE_OK;
}

int locmoe_moe_layer(const locmoe_shape_t* shape, const void* x, const int32_t* src_dev, const float* eps,
                     const locmoe_capacity_rule_t* rule, int32_t C_alloc, int32_t F, const void* w_in,
                     const void* w_out, const locmoe_layer_buffers_t* b, void* out, void* stream) {
    if (!b) return LOCMOE_ERR_NULL;
    int warn = 0;
    int rc = locmoe_gate_route(shape, x, eps, src_dev, rule, b->idx, b->gate_w, b->cos_sim, b->delta_e, b->theta_e, b->cap_dev,
                               C_alloc, b->pos, b->slot, b->drop, b->inv, b->counts, b->kept, b->send_counts, b->load,
                               b->locality, b->status, 0, b->ws, b->ws_bytes, stream);
    if (rc < 0) return rc;
    warn |= rc;
    rc = locmoe_dispatch(shape, C_alloc, x, b->inv, b->slot, b->buf, 1, stream);
    if (rc < 0) return rc;
    warn |= rc;
    const void* ysrc = b->buf;
    int ydt = shape->x_dtype;
    if (w_in) {
        rc = locmoe_expert_ffn(shape, C_alloc, F, b->buf, w_in, w_out, b->h1, b->y, LOCMOE_BF16, stream);
        if (rc < 0) return rc;
        warn |= rc;
        ysrc = b->y;
        ydt = LOCMOE_BF16;
    }
    rc = locmoe_combine(shape, C_alloc, ysrc, ydt, b->slot, b->gate_w, out, 0, stream);
    if (rc < 0) return rc;
    return warn | rc;
}

int locmoe_conventional_capacity(const locmoe_shape_t* shape, const locmoe_capacity_rule_t* rule, int32_t* C_alloc) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!rule || !C_alloc) return LOCMOE_ERR_NULL;
    if (rule->T_global < 0 || !(rule->capacity_factor >= 0.0)) return LOCMOE_ERR_SHAPE;
    // the same sequence of individually rounded operations as the device's integer rule (host code is
    // compiled without contraction of a * b / c into fused operations: these are separate statements)
    const double dT = (double)(rule->T_global > 0 ? rule->T_global : shape->T);
    const double dD = (double)shape->n_nodes * (double)shape->dev_per_node, n = (double)shape->E;
    volatile double cfT = rule->capacity_factor * dT;
    volatile double den = dD * n;
    volatile double q = cfT / den;
    double c = ceil(q);
    c = c < 1.0 ? 1.0 : (c > dT ? dT : c);
    *C_alloc = (int32_t)c;
    return LOCMOE_OK;
}

int locmoe_batch_delta(const float* delta_e_host, int32_t E, double* delta_host) {
    if (!delta_e_host || !delta_host) return LOCMOE_ERR_NULL;
    if (E < 1) return LOCMOE_ERR_SHAPE;
    float m = delta_e_host[0];
    for (int32_t e = 0; e < E; ++e) {
        const float v = delta_e_host[e];
        if (v != v) return LOCMOE_ERR_SHAPE;   // a NaN cannot be a threshold
        if (v < m) m = v;
    }
    const double d = (double)m;
    *delta_host = d < 0.0 ? 0.0 : (d > 1.0 ? 1.0 : d);
    return LOCMOE_OK;
}

int locmoe_dest_order(const locmoe_shape_t* shape, int32_t a, int32_t b) {
    if (!shape) return LOCMOE_ERR_NULL;
    const int N = shape->n_nodes, Dn = shape->dev_per_node;
    if (N < 1 || Dn < 1 || (long long)N * Dn > 0x7fffffffll) return LOCMOE_ERR_SHAPE;
    const int D = N * Dn;
    if (a < 0 || a >= D || b < 0 || b >= D) return LOCMOE_ERR_SHAPE;
    return dest_order(a, b, N, Dn);
}

int locmoe_launch_counts(const locmoe_shape_t* shape, int32_t counts[5]) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!counts) return LOCMOE_ERR_NULL;
    RoutePlan p;
    if ((rc = plan_route(*shape, &p))) return rc;
    counts[0] = 1;
    counts[1] = capacity_cluster_eligible(*shape) ? 1 : 2;
    counts[2] = p.launches;
    counts[3] = 1;
    counts[4] = 1;
    return LOCMOE_OK;
}

int locmoe_device_flags(int32_t* flags_host, void* stream) {
    if (!flags_host) return LOCMOE_ERR_NULL;
    int v = 0, f = 0;
    int rc = read_device_flags(&v, static_cast<cudaStream_t>(stream));
    if (rc == LOCMOE_OK) rc = read_ffn_flags(&f, static_cast<cudaStream_t>(stream));
    *flags_host = v | (f << 1);
    return rc;
}

const char* locmoe_status_string(int code) {
    switch (code) {
        case LOCMOE_OK: return "ok";
        case LOCMOE_ERR_NULL: return "a required pointer is NULL";
        case LOCMOE_ERR_SHAPE: return "invalid shape or size";
        case LOCMOE_ERR_DTYPE: return "unknown dtype, layout or bound form";
        case LOCMOE_ERR_ALIGN: return "pointer alignment";
        case LOCMOE_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
        case LOCMOE_ERR_CUDA: return "a CUDA call failed";
        case LOCMOE_ERR_TOO_LARGE: return "size exceeds the built-in scratch of the no-allocation entry point";
        default: return code > 0 ? "warning bits set" : "unknown error";
    }
}

}  // extern "C"
