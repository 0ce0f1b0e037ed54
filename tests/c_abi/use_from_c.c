/* The library from plain C: include/omc.h, no C++, no Python.  Builds a plan for three variables,
 * compresses them on the GPU, runs one update round, decompresses, and prints what a caller would
 * check.  Compiled and run by tests/test_gpu_c_abi.py (needs a GPU); links libomc.so and libcudart. */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>

#include "omc.h"

#define CK(x) do { int rc_ = (x); if (rc_ != 0) { printf("FAIL %s -> %d (%s)\n", #x, rc_, omc_strerror(rc_)); return 1; } } while (0)
#define CU(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("FAIL %s -> %s\n", #x, cudaGetErrorString(e_)); return 1; } } while (0)

int main(void)
{
    omc_var_desc_t vars[3] = {{5000, OMC_KIND_WEIGHT_MATRIX, 0}, {64, OMC_KIND_BIAS, 0}, {1500, OMC_KIND_WEIGHT_MATRIX, 0}};
    omc_format_t fmt = {1, 5, 2, 0};
    omc_plan_t *plan = NULL;
    CK(omc_plan(vars, 3, fmt, 1.0, 0, NULL, OMC_PLAN_DEFAULT, &plan));
    uint64_t full, resid, packed, ws, closed;
    uint32_t nq;
    CK(omc_plan_sizes(plan, &full, &resid, &packed, &nq, &ws, &closed));
    if (nq != 2 || closed != 5000 + 8 + 1500 + 8 + 4 * 64) { printf("FAIL sizes\n"); return 1; }

    float *h = (float *)malloc(full * sizeof(float)), *hg = (float *)malloc(full * sizeof(float));
    for (uint64_t i = 0; i < full; ++i) { h[i] = 0.05f * (float)((int)(i * 2654435761u % 2001) - 1000) / 1000.f; hg[i] = 1e-3f; }
    float *d_params, *d_grads, *d_out, *d_resid, *d_sb;
    uint8_t *d_packed;
    void *d_ws;
    CU(cudaMalloc((void **)&d_params, full * 4)); CU(cudaMalloc((void **)&d_grads, full * 4)); CU(cudaMalloc((void **)&d_out, full * 4));
    CU(cudaMalloc((void **)&d_resid, (resid + 4) * 4)); CU(cudaMalloc((void **)&d_sb, 2 * nq * 4));
    CU(cudaMalloc((void **)&d_packed, packed)); CU(cudaMalloc(&d_ws, ws));
    CU(cudaMemcpy(d_params, h, full * 4, cudaMemcpyHostToDevice)); CU(cudaMemcpy(d_grads, hg, full * 4, cudaMemcpyHostToDevice));

    CK(omc_plan_prepare(plan, d_ws, NULL));
    CK(omc_compress(plan, d_params, d_packed, d_resid, d_sb, d_ws, NULL));
    CK(omc_update_recompress(plan, d_packed, d_resid, d_sb, d_grads, 0.5f, NULL, d_ws, NULL));
    CK(omc_decompress(plan, d_packed, d_resid, d_sb, 0, 3, d_out, NULL));
    uint32_t status = 7;
    CK(omc_plan_status(plan, NULL, &status));
    float *back = (float *)malloc(full * sizeof(float));
    CU(cudaMemcpy(back, d_out, full * 4, cudaMemcpyDeviceToHost));
    /* W = V - 0.5 * 1e-3; the 8-bit code keeps about two significant bits: error below 1/8 relative + step */
    double worst = 0;
    for (uint64_t i = 0; i < 5000; ++i) {
        double want = (double)h[i] - 0.5e-3, err = back[i] - want;
        if (err < 0) err = -err;
        double tol = 0.13 * (want < 0 ? -want : want) + 1e-3;
        if (err > tol) { printf("FAIL element %llu: %g vs %g\n", (unsigned long long)i, back[i], want); return 1; }
        if (err > worst) worst = err;
    }
    uint64_t off_bias = 0;
    CK(omc_plan_var(plan, 1, NULL, &off_bias, NULL, NULL, NULL, NULL));
    if (back[off_bias] != h[off_bias] - 0.5f * 1e-3f) { printf("FAIL fp32 variable\n"); return 1; }
    if (omc_compress(plan, NULL, d_packed, d_resid, d_sb, d_ws, NULL) != OMC_ERR_NULL_PTR) { printf("FAIL null check\n"); return 1; }
    CK(omc_plan_destroy(plan));
    printf("OK status=%u worst_abs_err=%g\n", status, worst);
    return status == 0 ? 0 : 1;
}
