/* Drives libef through its C ABI from plain C (no Python, no torch): reads a small problem and
 * its gradients from stdin, runs the iterations and prints every output, so that a test can
 * compare them with values worked out by hand from Algorithm 4.
 *
 * stdin:  d B  offsets[B+1]  M mu eta steps  then steps*M gradients of d floats (step-major).
 * stdout: per step and worker "W t i : words... : scales... : residual...", per step
 *         "S t : words... : scales... : residual... : x...".
 */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "ef.h"

#define CHECK(call) do { int rc_ = (call); if (rc_ != EF_OK) { \
    fprintf(stderr, "%s -> %s\n", #call, ef_strerror(rc_)); return 2; } } while (0)
#define CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_)); return 3; } } while (0)

static void print_f(const char* sep, const float* dev, long n) {
    float* h = (float*)malloc(sizeof(float) * n);
    cudaMemcpy(h, dev, sizeof(float) * n, cudaMemcpyDeviceToHost);
    printf("%s", sep);
    for (long k = 0; k < n; ++k) printf(" %.9g", h[k]);
    free(h);
}
static void print_u(const char* sep, const uint32_t* dev, long n) {
    uint32_t* h = (uint32_t*)malloc(sizeof(uint32_t) * n);
    cudaMemcpy(h, dev, sizeof(uint32_t) * n, cudaMemcpyDeviceToHost);
    printf("%s", sep);
    for (long k = 0; k < n; ++k) printf(" %u", h[k]);
    free(h);
}

int main(void) {
    long long d; int B, M, steps; float mu, eta;
    if (scanf("%lld %d", &d, &B) != 2) return 1;
    int64_t* off = (int64_t*)malloc(sizeof(int64_t) * (B + 1));
    for (int b = 0; b <= B; ++b) { long long v; if (scanf("%lld", &v) != 1) return 1; off[b] = v; }
    if (scanf("%d %f %f %d", &M, &mu, &eta, &steps) != 4) return 1;

    size_t bytes = 0;
    CHECK(ef_workspace_bytes(d, B, off, M, 0, &bytes));
    void* ws = NULL; float *g = NULL, *tmp = NULL;
    CUDA(cudaMalloc(&ws, bytes));
    CUDA(cudaMalloc((void**)&g, sizeof(float) * d));
    CUDA(cudaMalloc((void**)&tmp, sizeof(float) * d));
    ef_ctx* ctx = NULL;
    CHECK(ef_init(&ctx, d, B, off, M, mu, eta, 0, ws, bytes, NULL));
    const long W = (long)ef_num_words(ctx);
    float* hg = (float*)malloc(sizeof(float) * d);
    for (int t = 0; t < steps; ++t) {
        for (int i = 0; i < M; ++i) {
            for (long long j = 0; j < d; ++j) if (scanf("%f", &hg[j]) != 1) return 1;
            CUDA(cudaMemcpy(g, hg, sizeof(float) * d, cudaMemcpyHostToDevice));
            CHECK(ef_worker_step(ctx, i, g));
            CUDA(cudaDeviceSynchronize());
            printf("W %d %d", t, i);
            print_u(" :", ef_worker_words(ctx, i), W);
            print_f(" :", ef_worker_scales(ctx, i), B);
            CHECK(ef_get_residual(ctx, i, tmp));
            print_f(" :", tmp, d);
            printf("\n");
        }
        CHECK(ef_server_step(ctx));
        CUDA(cudaDeviceSynchronize());
        printf("S %d", t);
        print_u(" :", ef_server_words(ctx), W);
        print_f(" :", ef_server_scales(ctx), B);
        CHECK(ef_get_residual(ctx, -1, tmp));
        print_f(" :", tmp, d);
        print_f(" :", ef_params(ctx), d);
        printf("\n");
    }
    int64_t tcount = 0;
    CHECK(ef_step_count(ctx, &tcount));
    printf("T %lld\n", (long long)tcount);
    CHECK(ef_destroy(ctx));
    cudaFree(ws); cudaFree(g); cudaFree(tmp); free(off); free(hg);
    return 0;
}
