// CUDA-core (dp4a) W8A8 GEMM + epilogue. Two uses:
//   * skinny M (a handful of tokens, e.g. the adaLN modulation linear): the
//     work is streaming the int8 weights once from HBM, which this does with
//     128-bit loads, several rows in flight per warp;
//   * an exact second implementation of acc / out for any shape (slow), used
//     to cross-check the tensor-core path on the device.
// Each warp owns NPW consecutive output channels and MB rows of A; lanes split K.
#include "internal.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace w8a8 {
namespace {

__device__ __forceinline__ int dot16(const uint4& a, const uint4& b, int acc) {
    acc = __dp4a(static_cast<int>(a.x), static_cast<int>(b.x), acc);
    acc = __dp4a(static_cast<int>(a.y), static_cast<int>(b.y), acc);
    acc = __dp4a(static_cast<int>(a.z), static_cast<int>(b.z), acc);
    acc = __dp4a(static_cast<int>(a.w), static_cast<int>(b.w), acc);
    return acc;
}

template <int MB, int NPW, int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
gemm_simt_kernel(const int8_t* qa, int64_t lda_q, const float* s_tok,
                 const int8_t* __restrict__ qw, const float* __restrict__ s_ch, const float* __restrict__ bias,
                 void* __restrict__ out, int64_t ldo, int M, int N, int K, int raw_i32, int after_quantizer, int* status,
                 float* rowmax) {
    grid_dep_launch_dependents();      // a following kernel launched to allow it may set itself up early
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = (blockIdx.x * WARPS + warp) * NPW;
    const int m0 = blockIdx.y * MB;
    if (n0 >= N) return;

    int acc[MB][NPW];
#pragma unroll
    for (int i = 0; i < MB; ++i)
#pragma unroll
        for (int j = 0; j < NPW; ++j) acc[i][j] = 0;

    const int8_t* wrow[NPW];
#pragma unroll
    for (int j = 0; j < NPW; ++j) wrow[j] = qw + static_cast<int64_t>(min(n0 + j, N - 1)) * K;
    const int8_t* arow[MB];
#pragma unroll
    for (int i = 0; i < MB; ++i) arow[i] = qa + static_cast<int64_t>(min(m0 + i, M - 1)) * lda_q;

    // always launched so that it may start while the kernel ahead of it is finishing: wait for that kernel's results
    grid_dep_wait();
    // no quantizer ahead of this kernel to clear the status word: do it here (this kernel has no waits that could set it)
    if (!after_quantizer && status != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && warp == 0 && lane == 0) *status = 0;

#pragma unroll 2
    for (int k = lane * 16; k < K; k += 32 * 16) {      // unrolled: several 512-byte slices of each weight row in flight
        uint4 w[NPW], a[MB];
#pragma unroll
        for (int j = 0; j < NPW; ++j) w[j] = __ldg(reinterpret_cast<const uint4*>(wrow[j] + k));
#pragma unroll
        // Coherent loads (the quantizer ahead may have written these rows while this kernel was already resident).
        // One or two rows: plain, L1-cached ones, since every warp of the CTA re-reads them and nothing of them was
        // touched before the wait above, so no line in this SM's L1 can predate the quantizer's writes (12.1 against
        // 14.3-18.7 us at M = 1-2 with L2-only loads); more rows: L2-only loads, which leave L1 to the weight
        // stream (15.5 against 17.2 us at M = 4).
        for (int i = 0; i < MB; ++i)
            a[i] = MB <= 2 ? *reinterpret_cast<const uint4*>(arow[i] + k) : __ldcg(reinterpret_cast<const uint4*>(arow[i] + k));
#pragma unroll
        for (int i = 0; i < MB; ++i)
#pragma unroll
            for (int j = 0; j < NPW; ++j) acc[i][j] = dot16(a[i], w[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < MB; ++i)
#pragma unroll
        for (int j = 0; j < NPW; ++j)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[i][j] += __shfl_xor_sync(0xffffffffu, acc[i][j], o);

    // lane l finishes output (i, j) with i * NPW + j == l
    int mine = 0;
#pragma unroll
    for (int i = 0; i < MB; ++i)
#pragma unroll
        for (int j = 0; j < NPW; ++j)
            if (lane == i * NPW + j) mine = acc[i][j];
    if (lane < MB * NPW) {
        const int m = m0 + lane / NPW, n = n0 + lane % NPW;
        if (m < M && n < N) {
            if (raw_i32) {
                static_cast<int32_t*>(out)[static_cast<int64_t>(m) * ldo + n] = mine;
            } else {
                float t = __int2float_rn(mine);
                t = __fmul_rn(t, __ldcg(s_tok + m));      // plain loads for what the quantizer ahead of this kernel wrote
                t = __fmul_rn(t, s_ch[n]);
                if (bias != nullptr) t = __fadd_rn(t, bias[n]);
                const __nv_bfloat16 o = __float2bfloat16_rn(t);
                static_cast<__nv_bfloat16*>(out)[static_cast<int64_t>(m) * ldo + n] = o;
                if (rowmax != nullptr) {      // side output: largest magnitude written to row m (non-negative floats order like their bits)
                    const uint32_t bits = (static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(&o)) & 0x7fffu) << 16;
                    if (bits != 0u) atomicMax(reinterpret_cast<unsigned int*>(rowmax) + m, bits);
                }
            }
        }
    }
}

template <int MB, int NPW, int WARPS>
cudaError_t launch(const GemmArgs& a, cudaStream_t st) {
    dim3 grid((a.N + WARPS * NPW - 1) / (WARPS * NPW), (a.M + MB - 1) / MB);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(WARPS * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_simt_kernel<MB, NPW, WARPS>, a.qa, a.lda_q, a.s_tok, a.qw, a.s_ch, a.bias,
                              a.out, a.ldo, a.M, a.N, a.K, a.raw_i32 ? 1 : 0, a.after_quantizer ? 1 : 0, a.status,
                              a.raw_i32 ? static_cast<float*>(nullptr) : a.rowmax);
}

} // namespace

cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t st) {
    if (a.M <= 2) return launch<2, 8, 4>(a, st);     // 8 weight rows per warp: more bytes in flight per SM
    if (a.M <= 4) return launch<4, 8, 4>(a, st);
    return launch<8, 4, 4>(a, st);
}

} // namespace w8a8
