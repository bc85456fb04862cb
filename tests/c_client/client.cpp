// A caller of the C ABI that knows nothing about Python or PyTorch: plain cudaMalloc'ed buffers, the functions of
// include/w8a8_linear.h, and a check of the result against values worked out by hand.
//
// Weights are 2 * identity (N = K): per-channel absmax is 2, so qw = 127 * I and s_ch = 2 / 127. Activations are
// small integers (exact in bf16), row m holding m % 7 - 3 shifted by the column parity, with one entry of each row
// set to 127 so that every per-token scale is exactly 1 and the codes equal the values. Then
// out[m,n] = bf16(((127 * A[m,n]) * 1) * (2 / 127) + bias[n]), evaluated here in float in the same order.
#include "../../include/w8a8_linear.h"

#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

static uint16_t f2bf(float f) {            // round to nearest even
    uint32_t u;
    std::memcpy(&u, &f, 4);
    u += 0x7fffu + ((u >> 16) & 1u);
    return static_cast<uint16_t>(u >> 16);
}
static float bf2f(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

#define CK(x) do { if ((x) != cudaSuccess) { std::printf("CUDA error at line %d\n", __LINE__); return 2; } } while (0)
#define W8(x) do { int st_ = (x); if (st_ != W8A8_OK) { std::printf("line %d: %s\n", __LINE__, int8_status_string(st_)); return 3; } } while (0)

int main() {
    const int64_t M = 300, K = 256, N = 256;
    std::vector<float> W(N * K, 0.f), bias(N);
    for (int64_t n = 0; n < N; ++n) { W[n * K + n] = 2.f; bias[n] = 0.25f * static_cast<float>(n % 5); }
    std::vector<float> Af(M * K);
    std::vector<uint16_t> A(M * K);
    for (int64_t m = 0; m < M; ++m)
        for (int64_t k = 0; k < K; ++k) {
            float v = static_cast<float>(m % 7 - 3 + (k & 1));
            if (k == (m * 3) % K) v = 127.f;
            Af[m * K + k] = v;
            A[m * K + k] = f2bf(v);
        }
    float *dW, *dbias, *ds_ch;
    int8_t* dqw;
    void *dA, *dout, *dws;
    CK(cudaMalloc(&dW, W.size() * 4)); CK(cudaMalloc(&dbias, N * 4)); CK(cudaMalloc(&ds_ch, N * 4));
    CK(cudaMalloc(&dqw, N * K)); CK(cudaMalloc(&dA, A.size() * 2)); CK(cudaMalloc(&dout, M * N * 2));
    const size_t ws_bytes = int8_linear_workspace_bytes(M, N, K, W8A8_ACT_BF16);
    CK(cudaMalloc(&dws, ws_bytes));
    CK(cudaMemcpy(dW, W.data(), W.size() * 4, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dbias, bias.data(), N * 4, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dA, A.data(), A.size() * 2, cudaMemcpyHostToDevice));
    cudaStream_t st;
    CK(cudaStreamCreate(&st));
    W8(int8_quantize_weight_per_channel(dW, N, K, K, dqw, ds_ch, st));
    W8(int8_linear_fused(dA, W8A8_ACT_BF16, K, nullptr, dqw, ds_ch, dbias, dout, N, M, N, K, dws, ws_bytes, st));
    W8(int8_check_status(dws, st));
    std::vector<uint16_t> out(M * N);
    std::vector<int8_t> qw(N * K);
    CK(cudaMemcpy(out.data(), dout, out.size() * 2, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(qw.data(), dqw, qw.size(), cudaMemcpyDeviceToHost));
    long bad = 0;
    const float s_ch = 2.f / 127.f;
    for (int64_t n = 0; n < N && bad == 0; ++n)
        for (int64_t k = 0; k < K; ++k)
            if (qw[n * K + k] != (n == k ? 127 : 0)) { ++bad; break; }
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            float t = 127.f * Af[m * K + n];     // the accumulator: only k == n contributes
            t = t * 1.0f;
            t = t * s_ch;
            t = t + bias[n];
            if (out[m * N + n] != f2bf(t)) ++bad;
        }
    // The same linear once more through the entry that also reports the largest magnitude written per token, then
    // the one-pass quantizer on that output with those maxima: scales are rowmax / 127 (one float division) and the
    // codes rne(x / s), both recomputed here in plain float arithmetic from the values worked out above.
    float *drowmax, *ds2;
    int8_t* dq2;
    CK(cudaMalloc(&drowmax, M * 4)); CK(cudaMalloc(&ds2, M * 4)); CK(cudaMalloc(&dq2, M * N));
    W8(int8_linear_fused_rowmax(dA, W8A8_ACT_BF16, K, nullptr, dqw, ds_ch, dbias, dout, N, drowmax, M, N, K, dws, ws_bytes, st));
    W8(int8_check_status(dws, st));
    W8(int8_quantize_act_per_token_given_absmax(dout, M, N, N, drowmax, dq2, ds2, st));
    W8(int8_sticky_status(1, st));
    std::vector<float> rowmax(M), s2(M);
    std::vector<int8_t> q2(M * N);
    CK(cudaMemcpy(rowmax.data(), drowmax, M * 4, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(s2.data(), ds2, M * 4, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(q2.data(), dq2, q2.size(), cudaMemcpyDeviceToHost));
    for (int64_t m = 0; m < M; ++m) {
        float want_max = 0.f;
        for (int64_t n = 0; n < N; ++n) want_max = std::fmax(want_max, std::fabs(bf2f(out[m * N + n])));
        const float want_s = want_max > 0.f ? want_max / 127.0f : 1.0f;
        if (rowmax[m] != want_max || s2[m] != want_s) { ++bad; continue; }
        for (int64_t n = 0; n < N; ++n) {
            const volatile float quot = bf2f(out[m * N + n]) / want_s;      // volatile: one rounded float division
            if (q2[m * N + n] != static_cast<int8_t>(std::nearbyintf(quot))) ++bad;   // default rounding mode: ties to even
        }
    }
    cudaFree(drowmax); cudaFree(ds2); cudaFree(dq2);
    std::printf(bad == 0 ? "c client ok: %ld x %ld x %ld through the C ABI, every output as worked out by hand\n"
                         : "c client FAILED (%ld x %ld x %ld)\n", static_cast<long>(M), static_cast<long>(K), static_cast<long>(N));
    if (bad) std::printf("%ld mismatches\n", bad);
    cudaFree(dW); cudaFree(dbias); cudaFree(ds_ch); cudaFree(dqw); cudaFree(dA); cudaFree(dout); cudaFree(dws);
    cudaStreamDestroy(st);
    return bad == 0 ? 0 : 1;
}
