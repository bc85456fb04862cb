// One-kernel path of the fused W8A8 linear for small problems (at most 128 tokens, K <= 1024, one wave of CTAs):
// per-token quantization, int8 GEMM and dequantizing epilogue in a single launch, for sm_100a.
//
// The paper's fused kernel leaves the activation quantizer to a kernel of its own ("The fused kernel": per-token
// scales are computed online, ahead of the GEMM). For a problem of one or a few tiles that second launch, and the
// trip of the codes through global memory, are most of the time. Here every CTA owns 32 output channels, and the
// CTAs of a cluster (up to 4) share the quantizer's work through distributed shared memory:
//   1. a CTA requests its 32 x K slice of the int8 weights (plain 16-byte loads; the weights do not depend on the
//      kernel ahead, so they are requested before the dependency wait) and, after the wait, its share of the rows
//      of A (row r belongs to the CTA of rank r mod cluster size): both fetches are in flight together;
//   2. the weights go to shared memory in the 128-byte-swizzled K-major layout tcgen05.mma reads; every row of A is
//      quantized by one warp, which writes the codes in the same layout into the operand tile of EVERY CTA of the
//      cluster (st.shared::cluster), and the row's scale likewise; the first cluster also writes codes and scales
//      to the workspace, where the two-kernel path leaves them for the caller;
//   3. after a cluster barrier one thread issues the MMAs (M = 128, N = 32, K = 32 each) into 32 TMEM columns;
//   4. the four warps that can read the accumulator dequantize and store bf16 rows directly.
// The arithmetic is that of the other paths, operation for operation: scale = absmax / 127, q = RNE(x / s) exactly,
// out = bf16(((float(acc) * s_tok) * s_ch) + bias).
// No CTA waits on a flag of another one: the only exchanges are the hardware cluster barrier and an mbarrier wait
// for the CTA's own MMAs, which is bounded like every other wait of the library.
#include "../../include/w8a8_linear.h"
#include "internal.h"
#include "ptx.cuh"
#include "quant_math.cuh"

#include <cuda_bf16.h>

namespace w8a8 {
namespace {

constexpr int SF_THREADS = 512;            // 16 warps: one warp quantizes a row at a time
constexpr int SF_WARPS = SF_THREADS / 32;
constexpr int SF_BM = 128;                 // rows of the MMA (TMEM lanes); M <= 128
constexpr int SF_BN = 32;                  // output channels per CTA = TMEM columns
constexpr int SF_BK = 128;                 // bytes of K per k-block: one swizzled row
constexpr int SF_A_KB_BYTES = SF_BM * SF_BK;     // 16 KB
constexpr int SF_W_KB_BYTES = SF_BN * SF_BK;     // 4 KB

struct SmallArgs {
    const __nv_bfloat16* A;     // [M, K], row stride lda elements
    int64_t lda;
    const float* amax_in;       // absmax of every row handed in, or nullptr
    const int8_t* qw;           // [N, K] dense
    const float* s_ch;
    const float* bias;          // or nullptr
    __nv_bfloat16* out;         // [M, N], row stride ldo
    int64_t ldo;
    int8_t* qa_out;             // workspace: codes [M, K]
    float* s_tok_out;           // workspace: scales [M]
    float* rowmax;              // or nullptr
    int M, N, K;
    int* status;
    int* sticky;
    uint64_t wait_limit_ns;
    int starve;                 // test hook: the MMAs are never committed, so the epilogue's bounded wait runs out
};

__device__ __forceinline__ void st_cluster_v2(uint32_t cluster_addr, const uint2& v) {
    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// byte offset of the 16-byte chunk `c` of row `r` inside a k-block stored as 128-byte rows with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int r, int c) {
    return static_cast<uint32_t>((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4));
}

// KV: 16-byte units (8 bf16) of a row per lane (K <= 256 * KV); CS: CTAs per cluster
template <int KV, int CS>
__global__ void __launch_bounds__(SF_THREADS, 1)
small_fused_kernel(const SmallArgs p) {
    grid_dep_launch_dependents();      // a following kernel launched to allow it may set itself up early
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const int K = p.K, M = p.M, N = p.N;
    const int num_kb = (K + SF_BK - 1) / SF_BK;
    const uint32_t a_base = base;
    const uint32_t w_off = num_kb * SF_A_KB_BYTES;
    const uint32_t w_base = base + w_off;
    const uint32_t tail_off = num_kb * (SF_A_KB_BYTES + SF_W_KB_BYTES);
    float* s_tok_s = reinterpret_cast<float*>(base_ptr + tail_off);  // [128]
    float* s_ch_s = s_tok_s + SF_BM;                                 // [32]
    float* bias_s = s_ch_s + SF_BN;                                  // [32]
    const uint32_t bar = smem_u32(bias_s + SF_BN);                   // 8 bytes
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bias_s + SF_BN + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    __shared__ int dummy_status;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * SF_BN;
    const bool active = n0 < N;        // the grid is padded to whole clusters: a CTA past N only quantizes its share
    const uint32_t rank = CS > 1 ? cluster_ctarank() : 0u;

    if (warp == 0 && active) {
        tmem_alloc(smem_u32(tmem_slot), SF_BN);
        tmem_relinquish();
    }
    if (threadIdx.x == 32) {
        mbar_init(bar, 1);
        *abort_flag = 0;
        dummy_status = 0;
        fence_mbar_init();
    }
    // ---- request the CTA's weights: 32 rows x K bytes in 16-byte chunks (at most four per thread), zero beyond N and
    // beyond K (which is what makes the bytes of A past K harmless). Weights are complete before the call is
    // enqueued: no need to wait for the kernel ahead.
    const int chunks_per_row = num_kb * 8;
    const int w_chunks = active ? SF_BN * chunks_per_row : 0;
    uint4 wv[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int i = threadIdx.x + t * SF_THREADS;
        wv[t] = make_uint4(0, 0, 0, 0);
        if (i < w_chunks) {
            const int n = i / chunks_per_row, ck = i - n * chunks_per_row;
            if (n0 + n < N && ck * 16 < K)
                wv[t] = __ldg(reinterpret_cast<const uint4*>(p.qw + static_cast<int64_t>(n0 + n) * K + ck * 16));
        }
    }
    float my_sch = 0.f, my_bias = 0.f;
    if (threadIdx.x < SF_BN && active) {
        const int n = min(n0 + static_cast<int>(threadIdx.x), N - 1);
        my_sch = __ldg(p.s_ch + n);
        my_bias = p.bias != nullptr ? __ldg(p.bias + n) : 0.f;
    }
    // This kernel may have been launched while the kernel ahead of it was still running (programmatic dependent
    // launch): the activations (and a handed-in absmax) are read only after that kernel is complete.
    grid_dep_wait();
    if (p.status != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *p.status = 0;

    // ---- quantize this CTA's share of the rows of A into the operand tile of every CTA of the cluster.
    // Row r belongs to rank r % CS; within a rank, warp w takes its rows w, w + 16, ...
    {
        constexpr int RPW = SF_BM / SF_WARPS / CS;                       // rows per warp: 8 / CS
        constexpr int RB = RPW * KV <= 8 ? RPW : 8 / KV;                 // rows whose loads are in flight together
        const bool writer = blockIdx.x < CS;                             // the first cluster fills the workspace
        uint32_t a_remote[CS], s_remote[CS];
#pragma unroll
        for (int c = 0; c < CS; ++c) {
            a_remote[c] = CS > 1 ? mapa_shared(a_base, c) : a_base;
            s_remote[c] = CS > 1 ? mapa_shared(smem_u32(s_tok_s), c) : smem_u32(s_tok_s);
        }
#pragma unroll 1
        for (int b0 = 0; b0 < RPW; b0 += RB) {
            uint4 v[RB][KV];
            float given[RB];
#pragma unroll
            for (int b = 0; b < RB; ++b) {
                const int r = (warp + SF_WARPS * (b0 + b)) * CS + static_cast<int>(rank);
                given[b] = (p.amax_in != nullptr && r < M) ? *(p.amax_in + r) : 0.f;
#pragma unroll
                for (int j = 0; j < KV; ++j) {
                    const int k0 = (j * 32 + lane) * 8;
                    v[b][j] = make_uint4(0, 0, 0, 0);
                    if (r < M && k0 < K)      // plain coherent load: the kernel ahead may have produced A
                        v[b][j] = *reinterpret_cast<const uint4*>(p.A + static_cast<int64_t>(r) * p.lda + k0);
                }
            }
            if (b0 == 0) {
                // the weights requested above land while the rows of A are on their way
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int i = threadIdx.x + t * SF_THREADS;
                    if (i < w_chunks) {
                        const int n = i / chunks_per_row, ck = i - n * chunks_per_row;
                        *reinterpret_cast<uint4*>(base_ptr + w_off + (ck >> 3) * SF_W_KB_BYTES + sw128(n, ck & 7)) = wv[t];
                    }
                }
                if (threadIdx.x < SF_BN) {
                    s_ch_s[threadIdx.x] = my_sch;
                    bias_s[threadIdx.x] = my_bias;
                }
            }
#pragma unroll
            for (int b = 0; b < RB; ++b) {
                const int r = (warp + SF_WARPS * (b0 + b)) * CS + static_cast<int>(rank);
                if (r >= M) continue;                         // warp-uniform
                float amax;
                if (p.amax_in != nullptr) {
                    amax = given[b];
                } else {
                    __nv_bfloat162 m2 = __float2bfloat162_rn(0.f);
#pragma unroll
                    for (int j = 0; j < KV; ++j) m2 = absmax8(v[b][j], m2);
                    amax = unpack_max(m2);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                }
                const RowScale rs = make_row_scale(amax);
                const RowScale2 r2 = make_row_scale2(rs);
                if (lane == 0 && writer) p.s_tok_out[r] = rs.s;
#pragma unroll
                for (int c = 0; c < CS; ++c)
                    if (lane == c) st_cluster_f32(s_remote[c] + 4u * r, rs.s);
#pragma unroll
                for (int j = 0; j < KV; ++j) {
                    const int k0 = (j * 32 + lane) * 8;
                    if (k0 < K) {
                        const uint2 q = quant8(v[b][j], rs, r2);
                        const uint32_t off = (k0 >> 7) * SF_A_KB_BYTES + sw128(r, (k0 & 127) >> 4) + ((k0 >> 3) & 1) * 8;
#pragma unroll
                        for (int c = 0; c < CS; ++c) st_cluster_v2(a_remote[c] + off, q);
                        if (writer) *reinterpret_cast<uint2*>(p.qa_out + static_cast<int64_t>(r) * K + k0) = q;
                    }
                }
            }
        }
    }
    // generic-proxy writes of the operand tiles (local and remote) -> visible to the tensor cores' async-proxy reads
    fence_proxy_async_all();
    tc_fence_before();
    if (CS > 1) cluster_sync_all(); else __syncthreads();
    fence_proxy_async_all();
    tc_fence_after();
    if (!active) return;               // nothing of this CTA is touched by another one after the barrier
    const uint32_t tmem = *tmem_slot;
    const WaitCtl ctl{abort_flag, p.status != nullptr ? p.status : &dummy_status, p.sticky, p.wait_limit_ns};

    if (threadIdx.x == 0) {
        constexpr uint32_t idesc = make_i8_idesc(SF_BM, SF_BN);
        for (int kb = 0; kb < num_kb; ++kb) {
            const uint64_t da = make_kmajor_sw128_desc(a_base + kb * SF_A_KB_BYTES);
            const uint64_t db = make_kmajor_sw128_desc(w_base + kb * SF_W_KB_BYTES);
            const int left = K - kb * SF_BK;
            const int ksteps = min(SF_BK, left + 31) / 32;
            for (int k = 0; k < ksteps; ++k)      // advancing K by 32 bytes inside the swizzled row: +2 in 16-byte units
                mma_i8_ss(tmem, da + 2 * k, db + 2 * k, idesc, (kb == 0 && k == 0) ? 0u : 1u);
        }
        if (!p.starve) tc_commit(bar);            // test hook: without the commit the wait below runs out
    }
    if (warp < 4) {
        // ---- epilogue: warp w reads TMEM lanes 32w .. 32w+31 (thread = row), all 32 columns
        __syncwarp();
        bool ok = mbar_wait(bar, 0, ctl, 4, kStatusTimeout);
        ok = __all_sync(0xffffffffu, ok) != 0;
        if (ok) {
            tc_fence_after();
            uint32_t acc[32];
            tmem_ld_32x32b_x32(tmem + (static_cast<uint32_t>(warp * 32) << 16), acc);
            tmem_wait_ld();
            const int m = warp * 32 + lane;
            if (m < M) {
                const float st = s_tok_s[m];
                uint32_t packed[16];
                uint32_t mx = 0;
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float t0 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(acc[j])), st), s_ch_s[j]);
                    float t1 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(acc[j + 1])), st), s_ch_s[j + 1]);
                    if (p.bias != nullptr) {
                        t0 = __fadd_rn(t0, bias_s[j]);
                        t1 = __fadd_rn(t1, bias_s[j + 1]);
                    }
                    const __nv_bfloat162 o = __floats2bfloat162_rn(t0, t1);
                    packed[j >> 1] = *reinterpret_cast<const uint32_t*>(&o);
                }
                __nv_bfloat16* orow = p.out + static_cast<int64_t>(m) * p.ldo + n0;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (n0 + 8 * g < N) {
                        *reinterpret_cast<uint4*>(orow + 8 * g) =
                            make_uint4(packed[4 * g], packed[4 * g + 1], packed[4 * g + 2], packed[4 * g + 3]);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {       // largest magnitude written (non-negative floats order like their bits)
                            const uint32_t w = packed[4 * g + i] & 0x7fff7fffu;
                            mx = max(mx, max(w << 16, w & 0xffff0000u));
                        }
                    }
                }
                if (p.rowmax != nullptr && mx != 0u) atomicMax(reinterpret_cast<unsigned int*>(p.rowmax) + m, mx);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, SF_BN);
}

template <int KV, int CS>
cudaError_t launch_kv_cs(const SmallArgs& p, int smem, cudaStream_t st) {
    static PerDeviceOnce smem_opt_in;
    const cudaError_t attr_err = smem_opt_in.run([] {
        return cudaFuncSetAttribute(small_fused_kernel<KV, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    });
    if (attr_err != cudaSuccess) return attr_err;
    const int ctas = (p.N + SF_BN - 1) / SF_BN;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((ctas + CS - 1) / CS * CS);      // whole clusters
    cfg.blockDim = dim3(SF_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = CS;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CS > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, small_fused_kernel<KV, CS>, p);
}

// The largest cluster (a power of two up to 4) the CTAs of the problem fill at least once. Clusters of 8 were
// measured no faster on one-tile problems (5.4 us either way at M = 128, K = N = 256) and much slower once the
// grid is a good part of the GPU (eight free SMs of one GPC per cluster).
template <int KV>
cudaError_t launch_kv(const SmallArgs& p, int smem, cudaStream_t st) {
    const int ctas = (p.N + SF_BN - 1) / SF_BN;
    if (ctas >= 4) return launch_kv_cs<KV, 4>(p, smem, st);
    if (ctas >= 2) return launch_kv_cs<KV, 2>(p, smem, st);
    return launch_kv_cs<KV, 1>(p, smem, st);
}

} // namespace

// What the kernel can run at all: one MMA tile of rows, operand tiles of a whole K in shared memory.
bool small_fused_eligible(int64_t M, int64_t N, int64_t K) {
    return M >= 1 && M <= SF_BM && K <= 1024 && N >= 1;
}

// Where it is the faster path (GPU time per call inside a CUDA graph of 50 calls, against the two-kernel path): more
// than a handful of tokens (fewer go to the weight-streaming kernel, which is as fast there) and at most 64, at most
// 32 CTAs, and at most 8 Ki elements of A to quantize per CTA (every cluster repeats the quantizer's work).
// One kernel / two kernels: M = 16, K = 512, N = 1024 4.5 / 5.3 us; (32, 256, 256) 3.9 / 4.7; (64, 512, 512) 5.1 / 5.5;
// (32, 1024, 1024) 6.1 / 6.6; but (64, 1024, 1024) 7.1 / 6.8, (128, 256, 256) 5.5 / 5.2, (128, 1024, 1024) 9.4 / 6.9.
bool small_fused_preferred(int64_t M, int64_t N, int64_t K) {
    if (!small_fused_eligible(M, N, K) || M <= kSkinnyM || M > kSmallFusedMaxTokens) return false;
    const int64_t ctas = (N + SF_BN - 1) / SF_BN;
    const int64_t cs = ctas >= 4 ? 4 : ctas >= 2 ? 2 : 1;
    return ctas <= kSmallFusedMaxCtas && M * K <= kSmallFusedMaxElemsPerCta * cs;
}

cudaError_t launch_small_fused(const void* A_bf16, int64_t lda, const float* amax_in, const GemmArgs& g, int8_t* qa_out,
                               float* s_tok_out, cudaStream_t st) {
    SmallArgs p{};
    p.A = static_cast<const __nv_bfloat16*>(A_bf16); p.lda = lda; p.amax_in = amax_in;
    p.qw = g.qw; p.s_ch = g.s_ch; p.bias = g.bias;
    p.out = static_cast<__nv_bfloat16*>(g.out); p.ldo = g.ldo;
    p.qa_out = qa_out; p.s_tok_out = s_tok_out; p.rowmax = g.rowmax;
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.status = g.status; p.sticky = sticky_status_word(); p.wait_limit_ns = wait_limit_ns();
    p.starve = starve_mode() == kStarveGemm ? 1 : 0;
    const int num_kb = (g.K + SF_BK - 1) / SF_BK;
    const int smem = num_kb * (SF_A_KB_BYTES + SF_W_KB_BYTES) + (SF_BM + 2 * SF_BN) * 4 + 16 + 1024;
    if (g.K <= 256) return launch_kv<1>(p, smem, st);
    if (g.K <= 512) return launch_kv<2>(p, smem, st);
    return launch_kv<4>(p, smem, st);
}

} // namespace w8a8
