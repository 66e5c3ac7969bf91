/* A client of libcawn written in plain C: no Python, no PyTorch, only the C ABI of include/cawn.h
 * and the CUDA runtime for device memory.  Reads pushes, gamma, theta from a file, runs the forward
 * (with state in and out and the gate mask) and the backward, writes the results to a file.
 * File layout (little endian): int32 B, L, H, F; float eps; then the arrays in the order used below. */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "cawn.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)
#define CHECK_CAWN(x) do { int s_ = (x); if (s_ != CAWN_OK) { fprintf(stderr, "%s: %s\n", #x, cawn_status_string(s_)); return 3; } } while (0)

static void *read_array(FILE *f, size_t bytes)
{
    void *p = malloc(bytes ? bytes : 1);
    if (p && bytes && fread(p, 1, bytes, f) != bytes) { free(p); return NULL; }
    return p;
}

int main(int argc, char **argv)
{
    if (argc != 3) { fprintf(stderr, "usage: %s input.bin output.bin\n", argv[0]); return 1; }
    FILE *f = fopen(argv[1], "rb");
    if (!f) return 1;
    int32_t hdr[4];
    float eps;
    if (fread(hdr, 4, 4, f) != 4 || fread(&eps, 4, 1, f) != 1) return 1;
    const int B = hdr[0], H = hdr[2], F = hdr[3], C = H * F;
    const int64_t L = hdr[1];
    const size_t n = (size_t)B * (size_t)L * C, MW = (size_t)(C + 31) / 32;
    float *p = read_array(f, n * 8), *gamma = read_array(f, (size_t)C * 4), *theta = read_array(f, (size_t)C * 4);
    float *state_in = read_array(f, (size_t)B * C * 8), *grad_y = read_array(f, n * 8);
    fclose(f);
    if (!p || !gamma || !theta || !state_in || !grad_y) return 1;

    cawn_params prm = {0};
    prm.struct_size = sizeof(prm);
    prm.B = B; prm.L = L; prm.H = H; prm.F = F; prm.gate_eps = eps;
    size_t ws_fwd = 0, ws_bwd = 0;
    CHECK_CAWN(cawn_workspace_bytes(&prm, CAWN_OP_FWD, &ws_fwd));
    CHECK_CAWN(cawn_workspace_bytes(&prm, CAWN_OP_BWD_SAVED, &ws_bwd));

    void *d_p, *d_y, *d_gy, *d_gp, *d_si, *d_so, *d_gsi, *d_wf, *d_wb;
    float *d_g, *d_t, *d_gg, *d_gt;
    uint32_t *d_m;
    CHECK_CUDA(cudaMalloc(&d_p, n * 8)); CHECK_CUDA(cudaMalloc(&d_y, n * 8));
    CHECK_CUDA(cudaMalloc(&d_gy, n * 8)); CHECK_CUDA(cudaMalloc(&d_gp, n * 8));
    CHECK_CUDA(cudaMalloc(&d_si, (size_t)B * C * 8)); CHECK_CUDA(cudaMalloc(&d_so, (size_t)B * C * 8));
    CHECK_CUDA(cudaMalloc(&d_gsi, (size_t)B * C * 8));
    CHECK_CUDA(cudaMalloc((void **)&d_g, (size_t)C * 4)); CHECK_CUDA(cudaMalloc((void **)&d_t, (size_t)C * 4));
    CHECK_CUDA(cudaMalloc((void **)&d_gg, (size_t)C * 4)); CHECK_CUDA(cudaMalloc((void **)&d_gt, (size_t)C * 4));
    CHECK_CUDA(cudaMalloc((void **)&d_m, (size_t)B * L * MW * 4));
    CHECK_CUDA(cudaMalloc(&d_wf, ws_fwd)); CHECK_CUDA(cudaMalloc(&d_wb, ws_bwd));
    CHECK_CUDA(cudaMemcpy(d_p, p, n * 8, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(d_gy, grad_y, n * 8, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(d_g, gamma, (size_t)C * 4, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(d_t, theta, (size_t)C * 4, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(d_si, state_in, (size_t)B * C * 8, cudaMemcpyHostToDevice));
    CHECK_CAWN(cawn_workspace_init(d_wf, ws_fwd, NULL));
    CHECK_CAWN(cawn_workspace_init(d_wb, ws_bwd, NULL));

    CHECK_CAWN(cawn_phase_accumulate_fwd(&prm, d_p, d_g, d_t, NULL, NULL, NULL, NULL, d_si, d_y, d_so, d_m, d_wf, ws_fwd, NULL));
    CHECK_CAWN(cawn_poll_status(d_wf, NULL));
    CHECK_CAWN(cawn_phase_accumulate_bwd(&prm, d_y, CAWN_SAVED_STATES, d_g, d_t, d_si, d_gy, NULL, d_gp, d_gg, d_gt, d_gsi,
                                         d_wb, ws_bwd, NULL));
    CHECK_CAWN(cawn_poll_status(d_wb, NULL));

    FILE *o = fopen(argv[2], "wb");
    if (!o) return 1;
    void *host = malloc(n ? n * 8 : 1);
    if (!host) return 1;
#define DUMP(dev, bytes) do { CHECK_CUDA(cudaMemcpy(host, dev, bytes, cudaMemcpyDeviceToHost)); fwrite(host, 1, bytes, o); } while (0)
    DUMP(d_y, n * 8);
    DUMP(d_so, (size_t)B * C * 8);
    DUMP(d_m, (size_t)B * L * MW * 4);
    DUMP(d_gp, n * 8);
    DUMP(d_gg, (size_t)C * 4);
    DUMP(d_gt, (size_t)C * 4);
    DUMP(d_gsi, (size_t)B * C * 8);
    fclose(o);
    printf("ok\n");
    return 0;
}
