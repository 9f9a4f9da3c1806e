/*
 * One whole step of the router path from a plain C program, tokens in pinned host memory:
 * host -> device copy, locmoe_gate, locmoe_capacity_route, locmoe_dispatch, locmoe_combine
 * (identity experts), device -> host copy, all queued on one stream.  This is the sequence the
 * end-to-end figure of the benchmark stands for; tests/test_c_step_gpu.py builds it, feeds it a
 * seeded batch and compares its output bit for bit with the Python binding's path.
 *
 *   c_step T H E n_nodes dev_per_node c_f x.bin src.bin out.bin slot.bin [graph]     (bf16 tokens)
 *
 * With the word "graph" as the last argument the four library calls are first run once eagerly, then captured
 * into a CUDA graph (the library allocates nothing and never synchronises, so its calls can be captured), the
 * outputs are overwritten with garbage, and the graph is replayed twice; the files hold the replay's result.
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "locmoe.h"

#define CK(call) do { if ((call) != cudaSuccess) { fprintf(stderr, "CUDA error at line %d\n", __LINE__); return 2; } } while (0)
#define LM(call) do { int rc_ = (call); if (rc_ < 0) { fprintf(stderr, "%s at line %d\n", locmoe_status_string(rc_), __LINE__); return 3; } } while (0)

static int read_file(const char *path, void *dst, size_t bytes) {
    FILE *f = fopen(path, "rb");
    if (!f) return 1;
    size_t n = fread(dst, 1, bytes, f);
    fclose(f);
    return n != bytes;
}

static int write_file(const char *path, const void *src, size_t bytes) {
    FILE *f = fopen(path, "wb");
    if (!f) return 1;
    size_t n = fwrite(src, 1, bytes, f);
    fclose(f);
    return n != bytes;
}

int main(int argc, char **argv) {
    if (argc != 11 && argc != 12) return 1;
    const int use_graph = argc == 12;
    locmoe_shape_t s = {atoi(argv[1]), atoi(argv[2]), atoi(argv[3]), atoi(argv[4]), atoi(argv[5]), LOCMOE_BF16, LOCMOE_LAYOUT_SEND};
    const double cf = atof(argv[6]);
    locmoe_capacity_rule_t rule = {cf, cf, -1.0, LOCMOE_BOUND_BETA, 0};
    const size_t T = (size_t)s.T, H = (size_t)s.H, E = (size_t)s.E, D = (size_t)s.n_nodes * s.dev_per_node;
    int32_t C_alloc = 0;
    size_t ws_bytes = 0;
    LM(locmoe_conventional_capacity(&s, &rule, &C_alloc));
    LM(locmoe_workspace_bytes(&s, C_alloc, &ws_bytes));
    const size_t rows = D * E * (size_t)C_alloc, xb = T * H * 2;

    void *xh, *outh; int32_t *srch, *sloth;                 /* pinned host buffers */
    CK(cudaMallocHost(&xh, xb)); CK(cudaMallocHost(&outh, xb));
    CK(cudaMallocHost((void **)&srch, T * 4)); CK(cudaMallocHost((void **)&sloth, T * 4));
    if (read_file(argv[7], xh, xb) || read_file(argv[8], srch, T * 4)) return 4;

    void *x, *out, *buf, *ws; int32_t *src, *idx, *pos, *slot, *inv, *counts, *kept, *send_counts, *load, *status;
    float *gate_w, *cos_sim, *delta_e, *theta_e; uint8_t *drop; int64_t *locality; locmoe_capacity_t *cap;
    CK(cudaMalloc(&x, xb)); CK(cudaMalloc(&out, xb)); CK(cudaMalloc(&buf, rows * H * 2)); CK(cudaMalloc(&ws, ws_bytes));
    CK(cudaMalloc((void **)&src, T * 4)); CK(cudaMalloc((void **)&idx, T * 4)); CK(cudaMalloc((void **)&pos, T * 4));
    CK(cudaMalloc((void **)&slot, T * 4)); CK(cudaMalloc((void **)&inv, rows * 4)); CK(cudaMalloc((void **)&drop, T));
    CK(cudaMalloc((void **)&counts, D * E * 4)); CK(cudaMalloc((void **)&kept, D * E * 4));
    CK(cudaMalloc((void **)&send_counts, D * D * 4)); CK(cudaMalloc((void **)&load, E * 4));
    CK(cudaMalloc((void **)&locality, 6 * 8)); CK(cudaMalloc((void **)&status, 4)); CK(cudaMalloc((void **)&cap, sizeof(*cap)));
    CK(cudaMalloc((void **)&gate_w, T * 4)); CK(cudaMalloc((void **)&cos_sim, T * 4));
    CK(cudaMalloc((void **)&delta_e, E * 4)); CK(cudaMalloc((void **)&theta_e, E * 4));

    cudaStream_t st;
    CK(cudaStreamCreate(&st));
    CK(cudaMemcpyAsync(x, xh, xb, cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(src, srch, T * 4, cudaMemcpyHostToDevice, st));
#define STEP() do { \
    LM(locmoe_gate(&s, x, NULL, idx, gate_w, cos_sim, NULL, st)); \
    LM(locmoe_capacity_route(&s, idx, cos_sim, src, &rule, delta_e, theta_e, cap, C_alloc, pos, slot, drop, inv, counts, kept, \
                             send_counts, load, locality, status, 0, ws, ws_bytes, st)); \
    LM(locmoe_dispatch(&s, C_alloc, x, inv, slot, buf, 1, st)); \
    LM(locmoe_combine(&s, C_alloc, buf, LOCMOE_BF16, slot, gate_w, out, 0, st)); } while (0)
    STEP();
    if (use_graph) {
        cudaGraph_t graph;
        cudaGraphExec_t exec;
        CK(cudaStreamSynchronize(st));
        CK(cudaStreamBeginCapture(st, cudaStreamCaptureModeGlobal));
        STEP();
        CK(cudaStreamEndCapture(st, &graph));
        CK(cudaGraphInstantiate(&exec, graph, 0));
        CK(cudaMemsetAsync(out, 0x5a, xb, st));
        CK(cudaMemsetAsync(slot, 0x5a, T * 4, st));
        CK(cudaGraphLaunch(exec, st));
        CK(cudaGraphLaunch(exec, st));
        CK(cudaStreamSynchronize(st));
        CK(cudaGraphExecDestroy(exec));
        CK(cudaGraphDestroy(graph));
    }
    CK(cudaMemcpyAsync(outh, out, xb, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(sloth, slot, T * 4, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    int32_t flags = -1;
    LM(locmoe_device_flags(&flags, st));
    if (flags != 0 || write_file(argv[9], outh, xb) || write_file(argv[10], sloth, T * 4)) return 5;
    printf("ok C_alloc=%d rows=%zu\n", C_alloc, rows);
    return 0;
}
