/* The C boundary used from plain C: no Python, no C++.  Builds tiny inputs, runs the nine-argument call and the
 * explicit-argument call, and checks the result against a triple loop written here (double accumulation, the two
 * bf16 roundings of the data path).  Prints "ok" and exits 0, or prints what went wrong and exits 1.
 * Build: gcc -std=c99 abi_smoke.c -I<include> -L<dir of libgmlp.so> -lgmlp -L<cuda>/lib64 -lcudart -lm */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "gmlp.h"

static uint16_t to_bf16(float f) {                       /* round to nearest even */
    uint32_t w;
    memcpy(&w, &f, 4);
    w += 0x7FFFu + ((w >> 16) & 1u);
    return (uint16_t)(w >> 16);
}
static float from_bf16(uint16_t b) {
    uint32_t w = (uint32_t)b << 16;
    float f;
    memcpy(&f, &w, 4);
    return f;
}
static float lcg(uint32_t* s) {                          /* uniform in [-1, 1) */
    *s = *s * 1664525u + 1013904223u;
    return (float)((*s >> 8) & 0xFFFF) / 32768.0f - 1.0f;
}

int main(void) {
    enum { M = 5, DM = 64, DFF = 128 };
    static uint16_t X[M * DM], Wg[DM * DFF], Wu[DM * DFF], Wd[DFF * DM], Y[M * DM], Y2[M * DM];
    uint32_t seed = 7;
    for (int i = 0; i < M * DM; ++i) X[i] = to_bf16(lcg(&seed));
    for (int i = 0; i < DM * DFF; ++i) { Wg[i] = to_bf16(lcg(&seed) * 0.2f); Wu[i] = to_bf16(lcg(&seed) * 0.2f); }
    for (int i = 0; i < DFF * DM; ++i) Wd[i] = to_bf16(lcg(&seed) * 0.2f);

    void *dX, *dWg, *dWu, *dWd, *dY;
    if (cudaMalloc(&dX, sizeof X) || cudaMalloc(&dWg, sizeof Wg) || cudaMalloc(&dWu, sizeof Wu) ||
        cudaMalloc(&dWd, sizeof Wd) || cudaMalloc(&dY, sizeof Y)) { printf("cudaMalloc failed\n"); return 1; }
    cudaMemcpy(dX, X, sizeof X, cudaMemcpyHostToDevice);
    cudaMemcpy(dWg, Wg, sizeof Wg, cudaMemcpyHostToDevice);
    cudaMemcpy(dWu, Wu, sizeof Wu, cudaMemcpyHostToDevice);
    cudaMemcpy(dWd, Wd, sizeof Wd, cudaMemcpyHostToDevice);

    int rc = gmlp_forward(dX, dWg, dWu, dWd, dY, M, DM, DFF, GMLP_FLAG_CHECKED);
    if (rc != GMLP_OK) { printf("gmlp_forward: %d (%s)\n", rc, gmlp_status_string(rc)); return 1; }
    cudaMemcpy(Y, dY, sizeof Y, cudaMemcpyDeviceToHost);

    gmlp_args a;
    memset(&a, 0, sizeof a);
    a.struct_bytes = sizeof a;
    a.flags = GMLP_FLAG_CHECKED;
    a.X = dX; a.Wg = dWg; a.Wu = dWu; a.Wd = dWd; a.Y = dY;
    a.M = M; a.d_model = DM; a.d_ff = DFF;
    a.variant = GMLP_VARIANT_UMMA;
    a.act_beta = 1.0f;
    rc = gmlp_forward_ex(&a);
    if (rc != GMLP_OK) { printf("gmlp_forward_ex: %d (%s)\n", rc, gmlp_status_string(rc)); return 1; }
    cudaMemcpy(Y2, dY, sizeof Y2, cudaMemcpyDeviceToHost);

    double worst = 0.0;
    for (int m = 0; m < M; ++m) {
        float h[DFF];
        for (int n = 0; n < DFF; ++n) {
            double g = 0.0, u = 0.0;
            for (int k = 0; k < DM; ++k) {
                g += (double)from_bf16(X[m * DM + k]) * from_bf16(Wg[k * DFF + n]);
                u += (double)from_bf16(X[m * DM + k]) * from_bf16(Wu[k * DFF + n]);
            }
            h[n] = from_bf16(to_bf16((float)(g / (1.0 + exp(-g)) * u)));
        }
        for (int j = 0; j < DM; ++j) {
            double y = 0.0;
            for (int n = 0; n < DFF; ++n) y += (double)h[n] * from_bf16(Wd[n * DM + j]);
            const double tol = 2e-2 * (fabs(y) > 1.0 ? fabs(y) : 1.0);
            const double e1 = fabs(from_bf16(Y[m * DM + j]) - y) / tol, e2 = fabs(from_bf16(Y2[m * DM + j]) - y) / tol;
            if (e1 > worst) worst = e1;
            if (e2 > worst) worst = e2;
        }
    }
    gmlp_shutdown();
    if (!(worst <= 1.0)) { printf("max err/tol %.3f\n", worst); return 1; }
    printf("ok (max err/tol %.3f, library version %d)\n", worst, gmlp_version());
    return 0;
}
