// Internal declarations shared by the LocMoE kernels and the C-ABI front end.
#pragma once

#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime.h>
#include <stdint.h>

#include "locmoe.h"

namespace locmoe {

constexpr int kWarp = 32;
constexpr int kNumSMsB200 = 148;

// Number of SMs of the current device (cached per process; B200 has 148).
int sm_count();

// LOCMOE_DEBUG=1 prints the CUDA error behind a LOCMOE_ERR_CUDA to stderr.
inline int check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        const char* d = getenv("LOCMOE_DEBUG");
        if (d && d[0] == '1') fprintf(stderr, "locmoe: CUDA error %d (%s)\n", (int)e, cudaGetErrorString(e));
    }
    return e == cudaSuccess ? LOCMOE_OK : LOCMOE_ERR_CUDA;
}

// ---- launchers (each queues its kernels on `st` and returns a LOCMOE_* code) ----
// What the gate also does per token when the route stage rides on it (locmoe_gate_route): the per-expert minimum
// of the cosines, the per-key demand counts and the (digit, tile) histogram of the first radix pass, all by
// integer atomics on arrays the route stage's fill kernel has initialised.  src == nullptr: nothing.
struct GateFuse {
    const int32_t* src;
    int32_t* counts;      // [D * E]
    int32_t* hist0;       // [1 << bits0][hstride]
    uint32_t* cap_min;    // [min_sets][E] order-preserving codes, 0xffffffff = no token yet
    int min_sets;         // a power of two
    int32_t* pos; int32_t* slot; uint8_t* drop; int32_t* status;   // a token with an impossible source is dropped here
    int D, digit_mask, hstride, tile_shift;
};

// Optional extras of the gate (locmoe_gate_ex): a per-source bias table and the fused column sums of the probabilities.
struct GateExtra {
    const int32_t* bias_src;   // [T]: eps is then [D][E] and token t takes row bias_src[t]; nullptr: eps is [E]
    float* p_part;             // [LOCMOE_GATE_PARTIAL_ROWS][E] or nullptr
};
int launch_gate(const locmoe_shape_t& s, const void* x, const float* eps, int32_t* idx, float* gate_w,
                float* cos_sim, float* probs, cudaStream_t st, const GateFuse* fuse = nullptr, const GateExtra* extra = nullptr);
int gate_last_grid();   // CTAs of the gate launch this thread queued last (= rows of p_part it writes)
int launch_aux_from_partials(const locmoe_shape_t& s, const float* p_part, int n_rows, const int32_t* load, float alpha,
                             float* f, float* P, float* loss, cudaStream_t st);

int launch_capacity(const locmoe_shape_t& s, const int32_t* idx, const float* cos_sim,
                    const locmoe_capacity_rule_t& rule, float* delta_e, float* theta_e,
                    locmoe_capacity_t* cap_dev, void* ws, cudaStream_t st);

struct RoutePlan {
    int key_bits;     // bits needed for keys 0..K (K = D*E is the "bad token" key)
    int passes;       // radix passes
    int bits[4];      // bits per pass, least significant first
    int tile;         // tokens per tile
    int rounds;       // 32-token rounds per warp per tile
    int ntiles;
    int hstride;      // row stride of the histogram matrices: ntiles rounded up to a multiple of 4
    int launches;     // kernel launches of one route call
    int prescan;      // 1: histogram matrices are prefix-scanned by a launch of their own (large batches)
    int nrep;         // replicas of the per-key demand counters that the first pass adds to (few keys: many adds per address)
    size_t off_keys[2], off_toks[2], off_hist[4], off_keystart, off_rowbase, off_rowtot, off_cap_part, off_counts_rep, total;
};
int plan_route(const locmoe_shape_t& s, RoutePlan* p);
size_t capacity_ws_bytes(const locmoe_shape_t& s);
bool capacity_cluster_eligible(const locmoe_shape_t& s);

int launch_route(const locmoe_shape_t& s, const int32_t* idx, const int32_t* src, const locmoe_capacity_t* cap_dev,
                 int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                 int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                 void* ws, cudaStream_t st);

bool capacity_route_fusable(const locmoe_shape_t& s);
int launch_capacity_route(const locmoe_shape_t& s, const int32_t* idx, const float* cos_sim, const int32_t* src,
                          const locmoe_capacity_rule_t& rule, float* delta_e, float* theta_e, locmoe_capacity_t* cap_dev,
                          int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop, int32_t* inv, int32_t* counts,
                          int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality, int32_t* status,
                          int early_init, void* ws, cudaStream_t st);

int launch_gate_route(const locmoe_shape_t& s, const void* x, const float* eps, const int32_t* src,
                      const locmoe_capacity_rule_t& rule, int32_t* idx, float* gate_w, float* cos_sim, float* delta_e,
                      float* theta_e, locmoe_capacity_t* cap_dev, int32_t C_alloc, int32_t* pos, int32_t* slot, uint8_t* drop,
                      int32_t* inv, int32_t* counts, int32_t* kept, int32_t* send_counts, int32_t* load, int64_t* locality,
                      int32_t* status, int early_init, void* ws, cudaStream_t st);

int launch_dispatch(const locmoe_shape_t& s, int64_t rows, const void* x, const int32_t* inv, const int32_t* slot,
                    void* buf, int zero_pad, cudaStream_t st);

int launch_combine(const locmoe_shape_t& s, int64_t rows, const void* y, int y_dtype, const int32_t* slot, const float* gate_w,
                   void* out, int accumulate, cudaStream_t st);

size_t aux_ws_bytes(const locmoe_shape_t& s);
int launch_aux_loss(const locmoe_shape_t& s, const float* probs, const int32_t* load, float alpha, float* f, float* P,
                    float* loss, void* ws, cudaStream_t st);

int launch_loc_loss(const locmoe_shape_t& s, const int32_t* counts, int level, double mu, double smooth, float* dc,
                    double* kl, long long* group_tokens, double* loss, cudaStream_t st);

int launch_cos_hist(const locmoe_shape_t& s, const void* x, const int32_t* idx, int e, int j, int nbins, float lo, float hi,
                    int32_t* hist_e, int32_t* hist_j, int32_t* n_routed, cudaStream_t st);

int launch_dispatch_peer(const locmoe_shape_t& s, int C_alloc, int64_t rows, const void* x, const int32_t* inv,
                         const int32_t* slot, void* const* peer_bufs, int n_peers, int src_lo, int src_hi, int zero_pad,
                         long long win_lo, long long win_hi, cudaStream_t st);
int launch_combine_peer(const locmoe_shape_t& s, int64_t rows, void* const* peer_y, int n_peers, int y_dtype,
                        const int32_t* slot, const float* gate_w, void* out, cudaStream_t st);

int launch_topk_select(const locmoe_shape_t& s, const float* probs, const int32_t* idx, const float* gate_w, int K,
                       int32_t* idx_k, float* w_k, cudaStream_t st);
int launch_topk_fold(int T, long long rows, int32_t* inv, cudaStream_t st);
int launch_combine_topk(const locmoe_shape_t& s, int64_t rows, const void* y, int y_dtype, int K, const int32_t* slot_k,
                        const float* w_k, void* out, cudaStream_t st);

int launch_expert_ffn(const locmoe_shape_t& s, int64_t rows, int F, const void* buf, const void* w_in,
                      const void* w_out, void* h1, void* y, int y_dtype, cudaStream_t st);
int read_ffn_flags(int* out, cudaStream_t st);
void plan_expert_ffn(const locmoe_shape_t& s, int64_t rows, int F, int kernels[2]);

// Copies the device diagnostics word to host memory (synchronises the stream).
int read_device_flags(int* out, cudaStream_t st);

// ---- programmatic dependent launch: a kernel launched with launch_pdl() may be scheduled while its predecessor
// on the stream is still draining; it must call pdl_wait() before it touches anything the predecessor wrote (all
// kernels here do so first thing), which blocks until the predecessor has completed and flushed.  pdl_trigger()
// lets the successor start its own launch early.  LOCMOE_PDL=0 in the environment turns the attribute off.
bool pdl_enabled();

template <typename... P, typename... A>
inline int launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...) != cudaSuccess) { cudaGetLastError(); return LOCMOE_ERR_CUDA; }
    return LOCMOE_OK;
}

#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// r(a, b) of the buffer layout: position of logical device b in device a's destination list (a itself, the rest
// of a's node, then the other nodes cyclically).  The one definition the kernels and the C ABI share.
__host__ __device__ __forceinline__ int dest_order(int a, int b, int N, int Dn) {
    int dn = b / Dn - a / Dn; if (dn < 0) dn += N;
    int dl = b % Dn - a % Dn; if (dl < 0) dl += Dn;
    return dn * Dn + dl;
}

// ---- small device helpers ----
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// fp32 -> bf16 bits, round to nearest even (NaN kept quiet).
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x40u;
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}

// Two floats -> packed bf16x2 (x in the low half), round to nearest even, one instruction.
__device__ __forceinline__ uint32_t cvt_bf16x2(const float2& f) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(f.y), "f"(f.x));
    return r;
}

// 16-byte accesses of the token matrices, every byte of which is touched once per kernel: streaming
// (evict-first) loads; plain stores, which measured 0.7 % faster per step than streaming stores on B200.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- bulk asynchronous copies (TMA, untiled form) and their mbarrier: the issuing CTA's shared memory only ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One poll of the barrier phase; true when the phase with this parity has completed.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` polls and returns false (the caller records the failure and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = 1u << 24) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; 16-byte aligned addresses, size a multiple of 16; completion on the mbarrier.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// shared -> global bulk copy, tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(smem_u32(src_smem)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until the sources of all but the newest N committed groups have been read (shared memory reusable).
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
// Makes generic-proxy writes to shared memory visible to the async proxy (before a bulk store reads them).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

}  // namespace locmoe
