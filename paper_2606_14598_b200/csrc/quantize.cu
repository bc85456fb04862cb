// Row-wise symmetric absmax int8 quantizer (per-token for activations,
// per-channel for weights): HBM-bound, one pass over the row held in registers.
//
//   s    = amax > 0 ? amax / 127 : 1          (IEEE division)
//   q[k] = clamp(rne(x[k] / s), -127, 127)    (IEEE division, round half to even)
//
// A persistent CTA of 16 warps works on RPC = 16 / WPR rows at a time (WPR warps share one
// row); in sweep i the CTAs of the grid together cover the consecutive rows
// [i * grid * RPC, (i + 1) * grid * RPC), so rows finish in ascending order. A row is split into
// 16-element chunks and every lane keeps CPL chunks in registers between the absmax pass and the
// quantize pass, so the input is read from memory exactly once. Loads are 128-bit, the int8 codes
// leave as one 128-bit store per chunk.
//
// When the caller passes a flag array, the CTA publishes, after each sweep, the call's 64-bit
// epoch into flags[row] of the rows it finished, with release semantics. The GEMM that follows
// (launched with programmatic dependent launch, so that it is already resident next to this
// kernel) acquires the flags of a row block before it loads it, and so starts on the first rows
// while later rows are still being quantized.
#include "internal.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

#include <mutex>

namespace w8a8 {
namespace {

constexpr int WARPS = 16;                 // warps per CTA
constexpr int CPL = 3;                    // register-resident 16-element chunks per lane

template <typename T> struct Chunk;       // 16 consecutive elements of a row

template <> struct Chunk<__nv_bfloat16> {
    uint4 lo, hi;                          // 8 + 8 bf16
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
        // packed bf16x2 |x| and max, then the larger half
        const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        __nv_bfloat162 m = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[0]));
#pragma unroll
        for (int i = 1; i < 8; ++i) m = __hmax2(m, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
        const uint32_t mb = *reinterpret_cast<const uint32_t*>(&m);
        return fmaxf(__uint_as_float(mb << 16), __uint_as_float(mb & 0xffff0000u));
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

// q = clamp(rne(x / s)) with the IEEE quotient, the definition.
__device__ __forceinline__ int quant_exact(float x, float s) {
    return max(-127, min(127, __float2int_rn(__fdiv_rn(x, s))));
}
__device__ __forceinline__ uint32_t quant4_exact(float a, float b, float c, float d, float s) {
    return (uint32_t(quant_exact(a, s)) & 0xffu) | ((uint32_t(quant_exact(b, s)) & 0xffu) << 8) |
           ((uint32_t(quant_exact(c, s)) & 0xffu) << 16) | (uint32_t(quant_exact(d, s)) << 24);
}

// The IEEE quotient without a division instruction. With inv = RN(1 / s) (correctly rounded, once
// per row), q0 = RN(x * inv) is within 1.5 ulp of x / s; one fma pair (remainder r0 = x - s * q0,
// exact; q1 = RN(q0 + r0 * inv)) makes it faithful, and by Markstein's theorem a second pair then
// yields exactly RN(x / s): if the reciprocal is correctly rounded and q is faithful, RN(q + r * inv)
// with the exact remainder r is the correctly rounded quotient (no over/underflow; scales outside
// [1e-30, 1e30] take the division instead). Adding 1.5 * 2^23 rounds the quotient to the nearest
// integer, ties to even, and leaves the code in the low byte of the sum; |x / s| <= 127 * (1 + 2^-23)
// so the clamp to [-127, 127] cannot bind.
struct RowScale {
    float s, inv;
    bool fast;      // false for degenerate scales: every element takes the division
};
__device__ __forceinline__ RowScale make_row_scale(float amax) {
    RowScale r;
    r.s = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 1.0f;
    r.inv = __frcp_rn(r.s);
    r.fast = r.s >= 1e-30f && r.s <= 1e30f;
    return r;
}
constexpr float MAGIC = 12582912.0f;               // 1.5 * 2^23

// the code of x in the low byte of the result (upper bytes are don't-care)
__device__ __forceinline__ uint32_t quant1(float x, const RowScale& rs) {
    const float q0 = __fmul_rn(x, rs.inv);
    const float r0 = __fmaf_rn(-rs.s, q0, x);
    const float q1 = __fmaf_rn(r0, rs.inv, q0);
    const float r1 = __fmaf_rn(-rs.s, q1, x);
    const float q2 = __fmaf_rn(r1, rs.inv, q1);
    return __float_as_uint(__fadd_rn(q2, MAGIC));
}
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, const RowScale& rs) {
    if (rs.fast) {
        const uint32_t lo = __byte_perm(quant1(a, rs), quant1(b, rs), 0x0040);
        const uint32_t hi = __byte_perm(quant1(c, rs), quant1(d, rs), 0x0040);
        return __byte_perm(lo, hi, 0x5410);
    }
    return quant4_exact(a, b, c, d, rs.s);
}

template <typename T>
__device__ __forceinline__ uint4 quant_chunk(const Chunk<T>& c, const RowScale& rs) {
    float f[16];
    c.unpack(f);
    uint4 o;
    o.x = quant4(f[0], f[1], f[2], f[3], rs);
    o.y = quant4(f[4], f[5], f[6], f[7], rs);
    o.z = quant4(f[8], f[9], f[10], f[11], rs);
    o.w = quant4(f[12], f[13], f[14], f[15], rs);
    return o;
}

// WPR warps per row (a power of two <= 16). Rows with more than WPR*32*CPL chunks
// stream the surplus twice (absmax pass, then quantize pass) from memory / L2.
template <typename T, int WPR>
__global__ void __launch_bounds__(WARPS * 32, sizeof(T) == 2 ? 2 : 1)   // bf16: <= 64 registers, so a GEMM CTA fits beside it
quant_rows_kernel(const T* __restrict__ x, int64_t ld, int rows, int K,
                  int8_t* __restrict__ q, float* __restrict__ s_out,
                  int* status_to_clear, unsigned long long* flags, unsigned long long epoch,
                  int burst_sweeps, int stay_ctas) {
    // a dependent kernel (the GEMM) may become resident right away; it synchronizes through `flags`
    grid_dep_launch_dependents();
    if (status_to_clear != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *status_to_clear = 0;

    constexpr int RPC = WARPS / WPR;                 // rows a CTA works on at a time
    constexpr int STRIDE = WPR * 32;
    __shared__ float s_red[WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot = warp / WPR, w_in_row = warp % WPR;
    const int nchunks = K >> 4;
    const int c0 = w_in_row * 32 + lane;
    // The first `burst_sweeps` sweeps are done by the whole grid; after them only the first `stay_ctas`
    // CTAs carry on (the others leave, which makes room on their SMs for the GEMM that follows).
    int sweep = 0;
    int sweep_rows = gridDim.x * RPC;
    int sweep_base = 0;

#pragma unroll 1
    for (;; ++sweep) {
        if (sweep == burst_sweeps) {
            if (static_cast<int>(blockIdx.x) >= stay_ctas) break;
            sweep_rows = stay_ctas * RPC;
        }
        if (sweep_base >= rows) break;
        const int base = sweep_base + blockIdx.x * RPC;
        sweep_base += sweep_rows;
        const int row = base + slot;
        const bool live = row < rows;
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
        if (WPR > 1) {
            if (lane == 0) s_red[warp] = amax;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < WPR; ++w) amax = fmaxf(amax, s_red[slot * WPR + w]);
        }
        if (live) {
            const RowScale s = make_row_scale(amax);
            if (w_in_row == 0 && lane == 0) s_out[row] = s.s;
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
        if (flags != nullptr || WPR > 1) __syncthreads();    // stores of the sweep are done; s_red may be reused
        if (flags != nullptr && threadIdx.x < RPC && base + threadIdx.x < rows) {
            // every thread's stores of this sweep happen before the flags become visible
            __threadfence();
            asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(flags + base + threadIdx.x), "l"(epoch) : "memory");
        }
    }
}

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

template <typename T, int WPR>
cudaError_t launch(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status_to_clear,
                   unsigned long long* flags, unsigned long long epoch, int burst_rows, cudaStream_t st) {
    constexpr int RPC = WARPS / WPR;
    const int units = (rows + RPC - 1) / RPC;
    const int cap = sm_count() * 2;                  // two CTAs of 16 warps fill an SM's register file
    const int grid = units < cap ? units : cap;
    // burst_rows < 0: the whole grid does every sweep. Otherwise the full grid only produces the first
    // burst_rows rows (at least), then one CTA per SM carries on.
    int burst_sweeps = 1 << 30, stay = grid;
    if (burst_rows >= 0 && grid > sm_count()) {
        burst_sweeps = (burst_rows + grid * RPC - 1) / (grid * RPC);
        stay = sm_count();
    }
    // keep the SM's L1/shared split at maximum shared memory while this kernel runs: the GEMM CTA that
    // joins it needs almost all of it, and the split only changes on an idle SM
    static std::once_flag once;
    std::call_once(once, [] {
        cudaFuncSetAttribute(quant_rows_kernel<T, WPR>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
    });
    quant_rows_kernel<T, WPR><<<grid, WARPS * 32, 0, st>>>(x, ld, rows, K, q, s, status_to_clear, flags, epoch,
                                                           burst_sweeps, stay);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status_to_clear,
                     unsigned long long* flags, unsigned long long epoch, int burst_rows, cudaStream_t st) {
    const int nchunks = K / 16;
    // fewest warps per row that keep the whole row in registers (<= CPL chunks per lane)
    if (nchunks <= 32 * CPL)  return launch<T, 1>(x, ld, rows, K, q, s, status_to_clear, flags, epoch, burst_rows, st);
    if (nchunks <= 64 * CPL)  return launch<T, 2>(x, ld, rows, K, q, s, status_to_clear, flags, epoch, burst_rows, st);
    if (nchunks <= 128 * CPL) return launch<T, 4>(x, ld, rows, K, q, s, status_to_clear, flags, epoch, burst_rows, st);
    if (nchunks <= 256 * CPL) return launch<T, 8>(x, ld, rows, K, q, s, status_to_clear, flags, epoch, burst_rows, st);
    return launch<T, 16>(x, ld, rows, K, q, s, status_to_clear, flags, epoch, burst_rows, st);
}

} // namespace

cudaError_t launch_quantize_bf16(const void* A, int64_t lda, int M, int K, int8_t* qa, float* s_tok,
                                 int* status_to_clear, unsigned long long* flags, unsigned long long epoch,
                                 int burst_rows, cudaStream_t st) {
    return dispatch<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(A), lda, M, K, qa, s_tok, status_to_clear, flags,
                                   epoch, burst_rows, st);
}

cudaError_t launch_quantize_f32(const float* W, int64_t ldw, int N, int K, int8_t* qw, float* s_ch, cudaStream_t st) {
    return dispatch<float>(W, ldw, N, K, qw, s_ch, nullptr, nullptr, 0ull, -1, st);
}

} // namespace w8a8
