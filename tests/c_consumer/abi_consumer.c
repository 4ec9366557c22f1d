/* A plain C program that uses libkop the way a non-Python caller would: CUDA runtime for memory and a
 * stream, kop.h for the kernels, nothing else. It checks results that have closed forms:
 *   softmax of a constant row is uniform and every row sums to 1;
 *   cross-entropy of constant logits is ln(V) for every row, and so is the mean;
 *   the running sum of ones is 1, 2, ..., n (exact in fp32), the reverse exclusive one n-1, ..., 0;
 *   GroupNorm output has zero mean and unit variance per group.
 * Exit code 0 and "abi consumer ok" on success. */
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "kop.h"

#define CHECK_CUDA(call)                                                                    \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            fprintf(stderr, "%s:%d: %s\n", __FILE__, __LINE__, cudaGetErrorString(e_));     \
            return 2;                                                                       \
        }                                                                                   \
    } while (0)

#define CHECK_KOP(call)                                                                     \
    do {                                                                                    \
        kop_status_t s_ = (call);                                                           \
        if (s_ != KOP_OK) {                                                                 \
            fprintf(stderr, "%s:%d: %s\n", __FILE__, __LINE__, kop_status_string(s_));      \
            return 3;                                                                       \
        }                                                                                   \
    } while (0)

#define EXPECT(cond, what)                                                                  \
    do {                                                                                    \
        if (!(cond)) {                                                                      \
            fprintf(stderr, "%s:%d: expectation failed: %s\n", __FILE__, __LINE__, what);   \
            return 4;                                                                       \
        }                                                                                   \
    } while (0)

int main(void)
{
    const int64_t rows = 37, cols = 1000;
    const size_t n = (size_t)rows * cols;
    float* h = (float*)malloc(n * sizeof(float));
    float* out = (float*)malloc(n * sizeof(float));
    if (!h || !out) return 1;
    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreate(&stream));
    float *dx, *dy;
    CHECK_CUDA(cudaMalloc((void**)&dx, n * sizeof(float)));
    CHECK_CUDA(cudaMalloc((void**)&dy, n * sizeof(float)));
    EXPECT(kop_version() >= 100, "version");

    /* softmax: row i is the constant i, plus a row-independent ramp in the last row */
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) h[i * cols + j] = (i == rows - 1) ? (float)(j % 7) : (float)i;
    CHECK_CUDA(cudaMemcpyAsync(dx, h, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    CHECK_KOP(kop_softmax_scale_bias(dx, NULL, dy, rows, cols, cols, cols, 0.5f, KOP_F32, (kop_stream_t)stream));
    CHECK_CUDA(cudaMemcpyAsync(out, dy, n * sizeof(float), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    for (int64_t i = 0; i < rows; ++i) {
        double sum = 0.0;
        for (int64_t j = 0; j < cols; ++j) sum += out[i * cols + j];
        EXPECT(fabs(sum - 1.0) < 1e-5, "softmax row sums to 1");
        if (i < rows - 1) EXPECT(fabs(out[i * cols + 3] - 1.0 / cols) < 1e-9, "softmax of a constant row is uniform");
    }

    /* cross-entropy of constant logits: ln(V) */
    int32_t* hl = (int32_t*)malloc(rows * sizeof(int32_t));
    for (int64_t i = 0; i < rows; ++i) hl[i] = (int32_t)((i * 131) % cols);
    for (size_t k = 0; k < n; ++k) h[k] = 0.25f;
    int32_t* dl;
    float *dloss, *dmean;
    int32_t* dbad;
    void* ws;
    const size_t ws_bytes = kop_ce_loss_rowwise_workspace_bytes(rows, cols, KOP_F32);
    EXPECT(ws_bytes > 0, "workspace size");
    CHECK_CUDA(cudaMalloc((void**)&dl, rows * sizeof(int32_t)));
    CHECK_CUDA(cudaMalloc((void**)&dloss, rows * sizeof(float)));
    CHECK_CUDA(cudaMalloc((void**)&dmean, sizeof(float)));
    CHECK_CUDA(cudaMalloc((void**)&dbad, sizeof(int32_t)));
    CHECK_CUDA(cudaMalloc(&ws, ws_bytes));
    CHECK_CUDA(cudaMemcpyAsync(dx, h, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    CHECK_CUDA(cudaMemcpyAsync(dl, hl, rows * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    CHECK_KOP(kop_ce_loss_rowwise(dx, dl, dloss, dmean, dbad, rows, cols, cols, ws, ws_bytes, KOP_F32,
                                  (kop_stream_t)stream));
    float hloss[64], hmean;
    int32_t hbad;
    CHECK_CUDA(cudaMemcpyAsync(hloss, dloss, rows * sizeof(float), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaMemcpyAsync(&hmean, dmean, sizeof(float), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaMemcpyAsync(&hbad, dbad, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    for (int64_t i = 0; i < rows; ++i) EXPECT(fabs(hloss[i] - log((double)cols)) < 1e-5, "CE of constant logits");
    EXPECT(fabs(hmean - log((double)cols)) < 1e-5 && hbad == 0, "CE mean and bad-label count");

    /* running sums of ones */
    for (size_t k = 0; k < n; ++k) h[k] = 1.0f;
    CHECK_CUDA(cudaMemcpyAsync(dx, h, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    CHECK_KOP(kop_cumsum_rows(dx, NULL, dy, rows, cols, cols, cols, cols, 0, 0, KOP_F32, (kop_stream_t)stream));
    CHECK_CUDA(cudaMemcpyAsync(out, dy, n * sizeof(float), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    for (int64_t j = 0; j < cols; ++j) EXPECT(out[5 * cols + j] == (float)(j + 1), "cumsum of ones");
    CHECK_KOP(kop_cumsum_rows(dx, NULL, dy, rows, cols, cols, cols, cols, 1, 1, KOP_F32, (kop_stream_t)stream));
    CHECK_CUDA(cudaMemcpyAsync(out, dy, n * sizeof(float), cudaMemcpyDeviceToHost, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    for (int64_t j = 0; j < cols; ++j) EXPECT(out[7 * cols + j] == (float)(cols - 1 - j), "reverse exclusive cumsum");

    /* GroupNorm: [2, 8, 5, 25] in 4 groups (rows * cols = 37000 floats are enough room) */
    {
        const int64_t N = 2, C = 8, H = 5, W = 25, G = 4;
        const size_t m = (size_t)(N * C * H * W);
        float *dmu, *drs;
        uint32_t lcg = 12345u;
        for (size_t k = 0; k < m; ++k) {
            lcg = lcg * 1664525u + 1013904223u;
            h[k] = (float)(lcg >> 8) * (1.0f / 16777216.0f) * 4.0f - 1.0f;
        }
        CHECK_CUDA(cudaMalloc((void**)&dmu, N * G * sizeof(float)));
        CHECK_CUDA(cudaMalloc((void**)&drs, N * G * sizeof(float)));
        CHECK_CUDA(cudaMemcpyAsync(dx, h, m * sizeof(float), cudaMemcpyHostToDevice, stream));
        CHECK_KOP(kop_groupnorm_act(dx, NULL, NULL, dy, dmu, drs, N, C, H, W, G, 0.0f, 0, KOP_F32,
                                    (kop_stream_t)stream));
        CHECK_CUDA(cudaMemcpyAsync(out, dy, m * sizeof(float), cudaMemcpyDeviceToHost, stream));
        CHECK_CUDA(cudaStreamSynchronize(stream));
        const size_t chunk = (size_t)(C / G * H * W);
        for (size_t g = 0; g < (size_t)(N * G); ++g) {
            double s = 0.0, q = 0.0;
            for (size_t k = 0; k < chunk; ++k) {
                s += out[g * chunk + k];
                q += (double)out[g * chunk + k] * out[g * chunk + k];
            }
            EXPECT(fabs(s / chunk) < 1e-5 && fabs(q / chunk - 1.0) < 1e-4, "GroupNorm output moments");
        }
        unsigned int timeouts = 99;
        CHECK_KOP(kop_groupnorm_wait_timeouts(&timeouts));
        EXPECT(timeouts == 0, "no bulk-copy wait ran out");
        cudaFree(dmu);
        cudaFree(drs);
    }

    /* validation happens before any launch */
    EXPECT(kop_cumsum_rows(NULL, NULL, dy, rows, cols, cols, cols, cols, 0, 0, KOP_F32, (kop_stream_t)stream) ==
               KOP_ERR_NULL_POINTER, "NULL input is rejected");
    EXPECT(kop_softmax_scale_bias(dx, NULL, dy, rows, cols, cols - 1, cols, 1.0f, KOP_F32, (kop_stream_t)stream) ==
               KOP_ERR_BAD_STRIDE, "short stride is rejected");

    cudaFree(dx); cudaFree(dy); cudaFree(dl); cudaFree(dloss); cudaFree(dmean); cudaFree(dbad); cudaFree(ws);
    cudaStreamDestroy(stream);
    free(h); free(out); free(hl);
    printf("abi consumer ok\n");
    return 0;
}
