// Host-side launch functions shared by the translation units of the library.
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace w8a8 {

// Device-side status codes written into the workspace status word (low byte
// is a w8a8_status value, the next byte says which wait gave up).
constexpr int kStatusTimeout = 7;

// ---- quantize.cu
// status_to_clear: workspace status word the kernel resets (or nullptr).
// mult: per-input-channel factors fp32 [K] multiplied into the operand first (SmoothQuant hook), or nullptr.
cudaError_t launch_quantize_bf16(const void* A, int64_t lda, int M, int K, const float* mult, int8_t* qa, float* s_tok,
                                 int* status_to_clear, cudaStream_t st);
cudaError_t launch_quantize_f32(const float* W, int64_t ldw, int N, int K, const float* mult, int8_t* qw, float* s_ch,
                                cudaStream_t st);

// ---- gemm_simt.cu : CUDA-core (dp4a) path, used for skinny M and as a cross-check
struct GemmArgs {
    const int8_t* qa;      // [M,K], row stride lda_q bytes
    int64_t lda_q;
    const float* s_tok;    // [M]
    const int8_t* qw;      // [N,K] dense
    const float* s_ch;     // [N]
    const float* bias;     // [N] or nullptr
    void* out;             // bf16 [M,N] (row stride ldo) or int32 [M,N] dense when raw_i32
    int64_t ldo;
    int M, N, K;
    bool raw_i32;
    int* status;           // workspace status word
    bool after_quantizer;  // launched behind the quantizer with programmatic dependent launch
};
cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t st);

// ---- gemm_tc.cu : tcgen05 path
int tc_num_configs();
const char* tc_config_name(int id);
// Picks a configuration for the shape (or `forced` if >= 0) and launches. Returns a w8a8_status.
int launch_gemm_tc(const GemmArgs& a, int forced, cudaStream_t st);

} // namespace w8a8
