// Row-wise symmetric absmax int8 quantizer (per-token for activations,
// per-channel for weights): HBM-bound, one pass over the row held in registers.
//
//   s    = amax > 0 ? amax / 127 : 1          (IEEE division)
//   q[k] = clamp(rne(x[k] / s), -127, 127)    (IEEE division, round half to even)
//
// A row is split into 16-element chunks. WARPS warps share one row; every lane
// keeps up to CPL chunks in registers between the absmax pass and the
// quantize pass, so the input is read from memory exactly once. Loads are
// 128-bit, the int8 codes leave as one 128-bit store per chunk.
#include "internal.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace w8a8 {
namespace {

template <typename T> struct Chunk;   // 16 consecutive elements of a row

template <> struct Chunk<__nv_bfloat16> {
    uint4 lo, hi;                      // 8 + 8 bf16
    __device__ __forceinline__ void load(const __nv_bfloat16* p) {
        const uint4* q = reinterpret_cast<const uint4*>(p);
        lo = __ldg(q);
        hi = __ldg(q + 1);
    }
    __device__ __forceinline__ void zero() { lo = make_uint4(0, 0, 0, 0); hi = lo; }
    // bf16 -> fp32 is exact: the 16 bits become the high half of the word
    __device__ __forceinline__ void unpack(float (&f)[16]) const {
        const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ __forceinline__ float absmax() const {
        // |x| ordering of bf16 equals the ordering of the 15-bit magnitudes
        const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        uint32_t m = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            m = max(m, w[i] & 0x7fffu);
            m = max(m, (w[i] >> 16) & 0x7fffu);
        }
        return __uint_as_float(m << 16);
    }
};

template <> struct Chunk<float> {
    float4 v[4];
    __device__ __forceinline__ void load(const float* p) {
        const float4* q = reinterpret_cast<const float4*>(p);
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = __ldg(q + i);
    }
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __device__ __forceinline__ void unpack(float (&f)[16]) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[4 * i] = v[i].x; f[4 * i + 1] = v[i].y; f[4 * i + 2] = v[i].z; f[4 * i + 3] = v[i].w; }
    }
    __device__ __forceinline__ float absmax() const {
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) m = fmaxf(fmaxf(m, fmaxf(fabsf(v[i].x), fabsf(v[i].y))), fmaxf(fabsf(v[i].z), fabsf(v[i].w)));
        return m;
    }
};

__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, float s) {
    int qa = max(-127, min(127, __float2int_rn(__fdiv_rn(a, s))));
    int qb = max(-127, min(127, __float2int_rn(__fdiv_rn(b, s))));
    int qc = max(-127, min(127, __float2int_rn(__fdiv_rn(c, s))));
    int qd = max(-127, min(127, __float2int_rn(__fdiv_rn(d, s))));
    return (uint32_t(qa) & 0xffu) | ((uint32_t(qb) & 0xffu) << 8) | ((uint32_t(qc) & 0xffu) << 16) | (uint32_t(qd) << 24);
}

template <typename T>
__device__ __forceinline__ uint4 quant_chunk(const Chunk<T>& c, float s) {
    float f[16];
    c.unpack(f);
    uint4 o;
    o.x = quant4(f[0], f[1], f[2], f[3], s);
    o.y = quant4(f[4], f[5], f[6], f[7], s);
    o.z = quant4(f[8], f[9], f[10], f[11], s);
    o.w = quant4(f[12], f[13], f[14], f[15], s);
    return o;
}

// WARPS warps per row, ROWS rows per block, up to CPL register-resident chunks
// per lane. If a row has more chunks than WARPS*32*CPL the surplus is streamed
// twice (absmax pass, then quantize pass) from memory/L2.
template <typename T, int WARPS, int ROWS, int CPL>
__global__ void __launch_bounds__(WARPS * ROWS * 32)
quant_rows_kernel(const T* __restrict__ x, int64_t ld, int rows, int K,
                  int8_t* __restrict__ q, float* __restrict__ s_out, int* status_to_clear) {
    // let a dependent kernel (the GEMM) start its own prologue right away
    grid_dep_launch_dependents();
    if (status_to_clear != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *status_to_clear = 0;

    __shared__ float s_red[ROWS][WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r_in_blk = warp / WARPS, w_in_row = warp % WARPS;
    const int row = blockIdx.x * ROWS + r_in_blk;
    const bool live = row < rows;
    const int nchunks = K >> 4;
    constexpr int STRIDE = WARPS * 32;
    const int c0 = w_in_row * 32 + lane;
    const T* xr = x + static_cast<int64_t>(live ? row : 0) * ld;

    Chunk<T> reg[CPL];
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const int c = c0 + i * STRIDE;
        if (live && c < nchunks) reg[i].load(xr + c * 16); else reg[i].zero();
    }
#pragma unroll
    for (int i = 0; i < CPL; ++i) amax = fmaxf(amax, reg[i].absmax());
    if (live) {
        for (int c = c0 + CPL * STRIDE; c < nchunks; c += STRIDE) {   // surplus chunks (very long rows)
            Chunk<T> t;
            t.load(xr + c * 16);
            amax = fmaxf(amax, t.absmax());
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (WARPS > 1) {
        if (lane == 0) s_red[r_in_blk][w_in_row] = amax;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < WARPS; ++w) amax = fmaxf(amax, s_red[r_in_blk][w]);
    }
    if (!live) return;
    const float s = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 1.0f;
    if (w_in_row == 0 && lane == 0) s_out[row] = s;

    int8_t* qr = q + static_cast<int64_t>(row) * K;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const int c = c0 + i * STRIDE;
        if (c < nchunks) *reinterpret_cast<uint4*>(qr + c * 16) = quant_chunk(reg[i], s);
    }
    for (int c = c0 + CPL * STRIDE; c < nchunks; c += STRIDE) {
        Chunk<T> t;
        t.load(xr + c * 16);
        *reinterpret_cast<uint4*>(qr + c * 16) = quant_chunk(t, s);
    }
}

template <typename T, int WARPS, int ROWS, int CPL>
cudaError_t launch(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status_to_clear, cudaStream_t st) {
    const int grid = (rows + ROWS - 1) / ROWS;
    quant_rows_kernel<T, WARPS, ROWS, CPL><<<grid, WARPS * ROWS * 32, 0, st>>>(x, ld, rows, K, q, s, status_to_clear);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status_to_clear, cudaStream_t st) {
    const int nchunks = K / 16;
    constexpr int CPL = 4;
    // fewest warps per row that keep the whole row in registers (<= CPL chunks per lane)
    if (nchunks <= 32 * CPL)      return launch<T, 1, 8, CPL>(x, ld, rows, K, q, s, status_to_clear, st);
    if (nchunks <= 64 * CPL)      return launch<T, 2, 4, CPL>(x, ld, rows, K, q, s, status_to_clear, st);
    if (nchunks <= 128 * CPL)     return launch<T, 4, 2, CPL>(x, ld, rows, K, q, s, status_to_clear, st);
    return launch<T, 8, 1, CPL>(x, ld, rows, K, q, s, status_to_clear, st);
}

} // namespace

cudaError_t launch_quantize_bf16(const void* A, int64_t lda, int M, int K, int8_t* qa, float* s_tok,
                                 int* status_to_clear, cudaStream_t st) {
    return dispatch<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(A), lda, M, K, qa, s_tok, status_to_clear, st);
}

cudaError_t launch_quantize_f32(const float* W, int64_t ldw, int N, int K, int8_t* qw, float* s_ch, cudaStream_t st) {
    return dispatch<float>(W, ldw, N, K, qw, s_ch, nullptr, st);
}

} // namespace w8a8
