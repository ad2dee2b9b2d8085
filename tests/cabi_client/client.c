/* A plain C11 client of the C ABI (no Python, no C++): reads a seeded test case from a file, runs the momentum update
 * (Eq. 7-8) and the scale-and-quantize pass (Eq. 5 + Eq. 1) on the GPU through include/quaff.h, writes the results to
 * a file.  The test that builds and runs it compares the file with the CPU oracle.
 *
 *   in :  int32 M, K, nO, nOp; float gamma;  X[M][K] bf16;  O[nO] int32;  wmax[nO] f32;  s[nO] f32
 *   out:  s_new[nO] f32;  Xq[M][K] int8;  xq_O[M][nOp] int8;  dx[M] f32
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "quaff.h"

#define CHECK_CUDA(x)                                                                     \
    do {                                                                                  \
        cudaError_t e_ = (x);                                                             \
        if (e_ != cudaSuccess) {                                                          \
            fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_));                      \
            return 2;                                                                     \
        }                                                                                 \
    } while (0)
#define CHECK_QUAFF(x)                                                                    \
    do {                                                                                  \
        quaff_status_t s_ = (x);                                                          \
        if (s_ != QUAFF_OK) {                                                             \
            fprintf(stderr, "%s: %s\n", #x, quaff_status_string(s_));                     \
            return 3;                                                                     \
        }                                                                                 \
    } while (0)

/* device buffer of `bytes` bytes, filled from `host` unless that is NULL */
static void* upload(const void* host, size_t bytes) {
    void* d = NULL;
    if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) return NULL;
    if (host && bytes && cudaMemcpy(d, host, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return NULL;
    return d;
}

int main(int argc, char** argv) {
    if (argc != 3) {
        fprintf(stderr, "usage: %s in.bin out.bin\n", argv[0]);
        return 1;
    }
    FILE* f = fopen(argv[1], "rb");
    if (!f) return 1;
    int32_t hdr[4];
    float gamma;
    if (fread(hdr, 4, 4, f) != 4 || fread(&gamma, 4, 1, f) != 1) return 1;
    const int M = hdr[0], K = hdr[1], nO = hdr[2], nOp = hdr[3];
    const size_t nx = (size_t)M * K;
    uint16_t* X = malloc(nx * 2);
    int32_t* O = malloc((size_t)nO * 4 + 4);
    float* wmax = malloc((size_t)nO * 4 + 4);
    float* s = malloc((size_t)nO * 4 + 4);
    if (fread(X, 2, nx, f) != nx || fread(O, 4, nO, f) != (size_t)nO || fread(wmax, 4, nO, f) != (size_t)nO ||
        fread(s, 4, nO, f) != (size_t)nO)
        return 1;
    fclose(f);

    cudaStream_t st;
    CHECK_CUDA(cudaStreamCreate(&st));
    quaff_bf16* dX = upload(X, nx * 2);
    int32_t* dO = upload(O, (size_t)nO * 4);
    float* dwmax = upload(wmax, (size_t)nO * 4);
    float* ds = upload(s, (size_t)nO * 4);
    const size_t ws_bytes = quaff_workspace_bytes(QUAFF_WS_MOMENTUM, M, K, 0, nOp, 0);
    void* ws = upload(NULL, ws_bytes);
    int8_t* dXq = upload(NULL, nx);
    int8_t* dxqo = upload(NULL, (size_t)M * nOp);
    float* ddx = upload(NULL, (size_t)M * 4);
    if (!dX || !dO || !dwmax || !ds || !ws || !dXq || !dxqo || !ddx) {
        fprintf(stderr, "device allocation or upload failed\n");
        return 2;
    }

    CHECK_QUAFF(quaff_momentum_update(dX, K, M, K, dO, nO, dwmax, gamma, ds, NULL, NULL, ws, ws_bytes, st));
    CHECK_QUAFF(quaff_quant_act(dX, K, M, K, dO, nO, ds, dXq, K, dxqo, nOp, nOp, ddx, st));
    CHECK_CUDA(cudaStreamSynchronize(st));

    int8_t* Xq = malloc(nx);
    int8_t* xqo = malloc((size_t)M * nOp + 1);
    float* dx = malloc((size_t)M * 4);
    CHECK_CUDA(cudaMemcpy(s, ds, (size_t)nO * 4, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(Xq, dXq, nx, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(xqo, dxqo, (size_t)M * nOp, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(dx, ddx, (size_t)M * 4, cudaMemcpyDeviceToHost));
    f = fopen(argv[2], "wb");
    if (!f) return 1;
    fwrite(s, 4, nO, f);
    fwrite(Xq, 1, nx, f);
    fwrite(xqo, 1, (size_t)M * nOp, f);
    fwrite(dx, 4, M, f);
    fclose(f);
    return 0;
}
