/* A plain C program that uses libkop the way a non-Python caller would: CUDA runtime for memory and a
 * stream, kop.h for the kernels, nothing else. It checks results that have closed forms:
 *   softmax of a constant row is uniform and every row sums to 1;
 *   cross-entropy of constant logits is ln(V) for every row, and so is the mean;
 *   the running sum of ones is 1, 2, ..., n (exact in fp32), the reverse exclusive one n-1, ..., 0;
 *   GroupNorm output has zero mean and unit variance per group;
 *   the MLP segment (vendor GEMMs kept) on constant rows and constant weights collapses to
 *   out = c + 2 s silu(s), s = c / sqrt(c^2 + eps), with a handle the library creates and with a cuBLAS handle
 *   this program owns.
 * Exit code 0 and "abi consumer ok" on success. */
#include <cublas_v2.h>
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

    /* MLP segment: rows of constant c_i, RMSNorm weight 1, gate rows of W1 = 1/H, up rows = 2/H, W2 = 1/I */
    {
        const int64_t M = 6, H = 16, I = 24;
        const float eps = 1e-6f;
        float *dh, *dw, *dW1, *dW2, *dout;
        void* mws;
        const size_t need = kop_rmsnorm_swiglu_residual_workspace_bytes(M, H, I, KOP_F32);
        EXPECT(need > 0, "MLP workspace size");
        CHECK_CUDA(cudaMalloc((void**)&dh, M * H * sizeof(float)));
        CHECK_CUDA(cudaMalloc((void**)&dout, M * H * sizeof(float)));
        CHECK_CUDA(cudaMalloc((void**)&dw, H * sizeof(float)));
        CHECK_CUDA(cudaMalloc((void**)&dW1, 2 * I * H * sizeof(float)));
        CHECK_CUDA(cudaMalloc((void**)&dW2, H * I * sizeof(float)));
        CHECK_CUDA(cudaMalloc(&mws, need));
        for (int64_t i = 0; i < M; ++i)
            for (int64_t j = 0; j < H; ++j) h[i * H + j] = (float)(i - 2) * 0.75f + 0.25f;
        CHECK_CUDA(cudaMemcpy(dh, h, M * H * sizeof(float), cudaMemcpyHostToDevice));
        for (int64_t j = 0; j < H; ++j) out[j] = 1.0f;
        CHECK_CUDA(cudaMemcpy(dw, out, H * sizeof(float), cudaMemcpyHostToDevice));
        for (int64_t r = 0; r < 2 * I; ++r)
            for (int64_t j = 0; j < H; ++j) out[r * H + j] = (r < I ? 1.0f : 2.0f) / (float)H;
        CHECK_CUDA(cudaMemcpy(dW1, out, 2 * I * H * sizeof(float), cudaMemcpyHostToDevice));
        for (int64_t k = 0; k < H * I; ++k) out[k] = 1.0f / (float)I;
        CHECK_CUDA(cudaMemcpy(dW2, out, H * I * sizeof(float), cudaMemcpyHostToDevice));
        cublasHandle_t mine;
        EXPECT(cublasCreate(&mine) == CUBLAS_STATUS_SUCCESS, "cublasCreate");
        for (int pass = 0; pass < 2; ++pass) {
            void* mh = NULL;
            if (pass == 0) CHECK_KOP(kop_mlp_handle_create(&mh));
            else CHECK_KOP(kop_mlp_handle_wrap((void*)mine, &mh));      /* the caller-owned vendor handle */
            CHECK_CUDA(cudaMemsetAsync(dout, 0, M * H * sizeof(float), stream));
            CHECK_KOP(kop_rmsnorm_swiglu_residual(mh, dh, dw, dW1, dW2, dout, M, H, I, eps, mws, need, KOP_F32,
                                                  (kop_stream_t)stream));
            CHECK_CUDA(cudaMemcpyAsync(out, dout, M * H * sizeof(float), cudaMemcpyDeviceToHost, stream));
            CHECK_CUDA(cudaStreamSynchronize(stream));
            for (int64_t i = 0; i < M; ++i) {
                const double c = (double)h[i * H];
                const double sgn = c / sqrt(c * c + (double)eps);
                const double want = c + 2.0 * sgn * (sgn / (1.0 + exp(-sgn)));
                for (int64_t j = 0; j < H; ++j)
                    EXPECT(fabs((double)out[i * H + j] - want) <= 1e-5 * fmax(1.0, fabs(want)), "MLP segment closed form");
            }
            CHECK_KOP(kop_mlp_handle_destroy(mh));
        }
        /* the wrapper's destruction left this program's handle alive */
        int ver = 0;
        EXPECT(cublasGetVersion(mine, &ver) == CUBLAS_STATUS_SUCCESS && ver > 0, "caller's cuBLAS handle still valid");
        EXPECT(cublasDestroy(mine) == CUBLAS_STATUS_SUCCESS, "cublasDestroy");
        EXPECT(kop_mlp_handle_wrap(NULL, NULL) == KOP_ERR_NULL_POINTER, "NULL handle is rejected");
        cudaFree(dh); cudaFree(dout); cudaFree(dw); cudaFree(dW1); cudaFree(dW2); cudaFree(mws);
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
