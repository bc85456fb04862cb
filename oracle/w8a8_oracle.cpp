// CPU oracle for the fused W8A8 linear layer. TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain statement of what the path computes. It is
// called by the tests, by the smoke check and by the benchmark's cpu_baseline
// leg; the product (the CUDA library) never links, imports or calls it, and it
// shares no code with the CUDA sources.
//
// What is followed (paper, Method section):
//   * "The quantization recipe (reused)": per-channel int8 weights and
//     per-token dynamic int8 activations, symmetric, scale = row absmax / 127.
//   * "The fused kernel": int8 x int8 -> int32 accumulation, then, off the
//     int32 accumulator, per-token scale, per-channel scale, plus bias.
// The paper prints no formula for the roundings, so the readings below are
// the ones this build fixes (all IEEE binary32, round-to-nearest-even, no
// fused multiply-add, no flush-to-zero):
//     s    = amax > 0 ? amax / 127 : 1          one fp32 division per row
//     q[k] = clamp(rne(x[k] / s), -127, 127)    one fp32 division per element
//     acc  = sum_k qa[m,k] * qw[n,k]            exact integer
//     t    = float(acc); t = t * s_tok[m]; t = t * s_ch[n]; t = t + bias[n]
//     out  = bf16_rne(t)
// The roundings to integer (codes) and to bf16 (outputs) are done on values / bit
// patterns directly. The arithmetic itself (/, *, +, and the int32 -> fp32
// conversion float(acc)) is the compiler's IEEE binary32 in the default
// round-to-nearest-even mode, with contraction off; the 2^24 and 2^31 edge
// vectors in the pins check that conversion.
//
// Pins (see tests/test_oracle_pins.py): hand tie vectors for the quantizer,
// scaling / sign / permutation invariants, brute force over tiny shapes,
// identity and one-hot weights, the K*127^2 < 2^31 edge in closed form,
// K-split additivity, fp64 bound for the epilogue, convergence to the float
// matmul as outliers vanish. Parity against the authors' own tensors is
// unpinned: the paper prints no tensor values.
//
// Build: g++ -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC (build() in oracle/__init__.py)

#include <cstdint>
#include <cstring>
#include <cmath>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline float bits_to_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }
inline uint32_t f32_to_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

// bf16 -> fp32 is exact: the 16 bits are the top half of the binary32 word.
inline float bf16_to_f32(uint16_t h) { return bits_to_f32(uint32_t(h) << 16); }

// fp32 -> bf16, round to nearest, ties to even, on the bit pattern.
inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u)            // NaN: keep it a quiet NaN
        return uint16_t((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;                             // carries into the exponent when needed
    return uint16_t(u >> 16);
}

// Round a finite float with |v| < 2^23 to the nearest integer, ties to even.
inline int32_t rne_to_int(float v) {
    float fl = std::floor(v);                       // exact
    float d = v - fl;                               // exact for |v| < 2^23
    int32_t i = int32_t(fl);
    if (d > 0.5f) return i + 1;
    if (d < 0.5f) return i;
    return (i & 1) ? i + 1 : i;                     // tie: pick the even neighbour
}

inline int32_t clamp127(int32_t q) { return q > 127 ? 127 : (q < -127 ? -127 : q); }

// max_k |x[k]| of one row (exact; 0 for an empty or all-zero row).
float row_absmax(const float* x, int64_t K) {
    float amax = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
        float a = std::fabs(x[k]);
        if (a > amax) amax = a;
    }
    return amax;
}

// The second half of the quantizer: scale and codes of one row from an absmax that is handed in. With the row's
// own absmax this is the whole quantizer; with a larger one the codes use less of the range; with a smaller one the
// clamp binds.
void quant_row_given(const float* x, int64_t K, float amax, int8_t* q, float* s_out) {
    float s = (amax > 0.0f) ? amax / 127.0f : 1.0f;
    for (int64_t k = 0; k < K; ++k) {
        float r = x[k] / s;
        q[k] = int8_t(clamp127(rne_to_int(r)));
    }
    *s_out = s;
}

// One row of the symmetric absmax quantizer on fp32 values.
void quant_row(const float* x, int64_t K, int8_t* q, float* s_out) {
    quant_row_given(x, K, row_absmax(x, K), q, s_out);
}

} // namespace

extern "C" {

// Per-output-channel weight quantization. W is fp32 [N, K] with row stride ldw
// (elements); qw is int8 [N, K] dense; s_ch is fp32 [N].
void oracle_quantize_weight_per_channel(const float* W, int64_t N, int64_t K, int64_t ldw,
                                        int8_t* qw, float* s_ch) {
    #pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        quant_row(W + n * ldw, K, qw + n * K, s_ch + n);
}

// SmoothQuant hook (the paper's recipe names SmoothQuant, alpha = 0.5; Method, "The quantization recipe"):
// a per-input-channel factor is multiplied into the operand before quantization, x'[k] = x[k] * mult[k]
// (one fp32 multiply, rounded), activations by 1/s_k and weights by s_k, so that the product is unchanged.
// How s is calibrated is outside this path; the factors are inputs. mult == NULL means no smoothing.
void oracle_quantize_weight_per_channel_smooth(const float* W, int64_t N, int64_t K, int64_t ldw, const float* mult,
                                               int8_t* qw, float* s_ch) {
    #pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        float* row = new float[K > 0 ? K : 1];
        for (int64_t k = 0; k < K; ++k) row[k] = mult ? W[n * ldw + k] * mult[k] : W[n * ldw + k];
        quant_row(row, K, qw + n * K, s_ch + n);
        delete[] row;
    }
}

void oracle_quantize_act_per_token_smooth(const uint16_t* A, int64_t M, int64_t K, int64_t lda, const float* mult,
                                          int8_t* qa, float* s_tok) {
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float* row = new float[K > 0 ? K : 1];
        for (int64_t k = 0; k < K; ++k) {
            const float x = bf16_to_f32(A[m * lda + k]);
            row[k] = mult ? x * mult[k] : x;
        }
        quant_row(row, K, qa + m * K, s_tok + m);
        delete[] row;
    }
}

// Per-token activation quantization. A is bf16 (raw 16-bit patterns) [M, K]
// with row stride lda (elements); qa is int8 [M, K] dense; s_tok is fp32 [M].
void oracle_quantize_act_per_token(const uint16_t* A, int64_t M, int64_t K, int64_t lda,
                                   int8_t* qa, float* s_tok) {
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float* row = new float[K > 0 ? K : 1];
        for (int64_t k = 0; k < K; ++k) row[k] = bf16_to_f32(A[m * lda + k]);
        quant_row(row, K, qa + m * K, s_tok + m);
        delete[] row;
    }
}

// The quantizer fused into its producer (the paper's Method: per-token scales are dynamic, computed online from the
// activations; nothing says in how many passes). Two pieces:
//   * the producer of an activation matrix also reports, per token, the largest magnitude it wrote:
//     rowmax[m] = max_n |X[m,n]| over the bf16 values as stored (exact, order-free);
//   * the quantizer takes that number instead of searching for it (one pass over the row).
// With rowmax equal to the row's absmax the result is, by construction, that of oracle_quantize_act_per_token.
void oracle_row_absmax_bf16(const uint16_t* X, int64_t M, int64_t N, int64_t ld, float* rowmax) {
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float amax = 0.0f;
        for (int64_t n = 0; n < N; ++n) {
            float a = std::fabs(bf16_to_f32(X[m * ld + n]));
            if (a > amax) amax = a;
        }
        rowmax[m] = amax;
    }
}

void oracle_quantize_act_per_token_given_absmax(const uint16_t* A, int64_t M, int64_t K, int64_t lda, const float* rowmax,
                                                int8_t* qa, float* s_tok) {
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float* row = new float[K > 0 ? K : 1];
        for (int64_t k = 0; k < K; ++k) row[k] = bf16_to_f32(A[m * lda + k]);
        quant_row_given(row, K, rowmax[m], qa + m * K, s_tok + m);
        delete[] row;
    }
}

// acc[m,n] = sum_k qa[m,k] * qw[n,k], stored as int32.
// For K <= 131071 no int8 inputs can overflow an int32 sum (K * 128 * 128 < 2^31),
// so the sum is taken in int32. For larger K it is taken in int64 and checked.
// Returns the number of outputs whose exact sum does not fit in int32 (always 0
// when K * 127^2 < 2^31 and no code is -128).
int64_t oracle_gemm_i32(const int8_t* qa, const int8_t* qw, int32_t* acc,
                        int64_t M, int64_t N, int64_t K) {
    int64_t bad = 0;
    if (K <= 131071) {
        #pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            for (int64_t n = 0; n < N; ++n) {
                int32_t s = 0;
                for (int64_t k = 0; k < K; ++k)
                    s += int32_t(qa[m * K + k]) * int32_t(qw[n * K + k]);
                acc[m * N + n] = s;
            }
        }
        return 0;
    }
    #pragma omp parallel for schedule(static) reduction(+:bad)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += int64_t(qa[m * K + k]) * int64_t(qw[n * K + k]);
            if (s > INT32_MAX || s < INT32_MIN) ++bad;
            acc[m * N + n] = int32_t(s);
        }
    }
    return bad;
}

// out[m,n] = bf16(((float(acc) * s_tok[m]) * s_ch[n]) + bias[n]); bias may be NULL.
void oracle_epilogue(const int32_t* acc, const float* s_tok, const float* s_ch,
                     const float* bias, uint16_t* out, int64_t M, int64_t N) {
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            float t = float(acc[m * N + n]);        // int32 -> fp32, round to nearest even
            t = t * s_tok[m];
            t = t * s_ch[n];
            if (bias) t = t + bias[n];
            out[m * N + n] = f32_to_bf16_rne(t);
        }
    }
}

// The whole path on bf16 activations: quantize, multiply, dequantize.
// qa, s_tok and acc are caller-provided scratch that also returns the
// intermediate tensors. Returns oracle_gemm_i32's overflow count.
int64_t oracle_linear_fused_bf16(const uint16_t* A, int64_t lda,
                                 const int8_t* qw, const float* s_ch, const float* bias,
                                 uint16_t* out, int64_t M, int64_t N, int64_t K,
                                 int8_t* qa, float* s_tok, int32_t* acc) {
    oracle_quantize_act_per_token(A, M, K, lda, qa, s_tok);
    int64_t bad = oracle_gemm_i32(qa, qw, acc, M, N, K);
    oracle_epilogue(acc, s_tok, s_ch, bias, out, M, N);
    return bad;
}

int oracle_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

} // extern "C"
