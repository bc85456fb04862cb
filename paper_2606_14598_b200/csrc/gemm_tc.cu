// Tensor-core W8A8 GEMM with the dequantizing epilogue, for sm_100a.
//
//   acc[m,n] = sum_k qa[m,k] * qw[n,k]        tcgen05.mma.kind::i8, int32 in TMEM
//   out[m,n] = bf16(((float(acc) * s_tok[m]) * s_ch[n]) + bias[n])
//
// One persistent CTA per SM walks output tiles of 128 x BN. Warp roles:
//   warp 0    TMA producer: loads the 128 x 128-byte A tile and the BN x 128-byte
//             W tile of each k-block into a ring of shared-memory stages
//             (128-byte swizzle, K-major: both operands are row-major over K)
//   warp 1    allocates TMEM and issues the MMAs (one thread), 4 per k-block
//             (K = 32 each); tcgen05.commit releases the stage / publishes the tile
//   warps 2-5 epilogue: tcgen05.ld the accumulator (lane = row, so s_tok is one
//             scalar per thread; s_ch and bias are per-column broadcasts from
//             shared memory), dequantize, pack to bf16, stage in swizzled shared
//             memory, TMA-store 32 x 64 boxes (TMA clips ragged M and N)
// Two accumulators of BN columns alternate in TMEM so that the epilogue of one
// tile overlaps the k-loop of the next.
//
// Every mbarrier wait is bounded: on expiry the CTA records W8A8_ERR_TIMEOUT in
// the workspace status word, all roles unwind, TMEM is freed and the kernel
// returns.
#include "internal.h"
#include "ptx.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>
#include <unordered_map>

namespace w8a8 {
namespace {

constexpr int BM = 128;            // rows of A per tile (= TMEM lanes)
constexpr int BK = 128;            // int8 elements (= bytes) of K per stage: one 128-byte swizzle row
constexpr int MMA_K = 32;          // K of one tcgen05.mma.kind::i8
constexpr int NUM_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;   // 2 s

enum Where { W_PRODUCER_EMPTY = 1, W_MMA_FULL = 2, W_MMA_TMEM_EMPTY = 3, W_EPI_TMEM_FULL = 4, W_DRAIN = 5 };

template <int BN, int STAGES>
struct SmemLayout {
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGING_BYTES_PER_WARP = 32 * 128;        // 32 rows x 64 bf16
    static constexpr int OFF_STAGING = STAGES * STAGE_BYTES;
    static constexpr int OFF_SCH = OFF_STAGING + 4 * STAGING_BYTES_PER_WARP;
    static constexpr int OFF_BIAS = OFF_SCH + BN * 4;
    static constexpr int OFF_BARS = OFF_BIAS + BN * 4;             // full[STAGES], empty[STAGES], tfull[2], tempty[2]
    static constexpr int NUM_BARS = 2 * STAGES + 4;
    static constexpr int OFF_TMEM = OFF_BARS + NUM_BARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int TOTAL = OFF_ABORT + 4;
    static constexpr int DYN_BYTES = TOTAL + 1024;                 // slack to align the base to 1024
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int BN, int STAGES, bool RAW_I32>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_out,
               const float* __restrict__ s_tok, const float* __restrict__ s_ch, const float* __restrict__ bias,
               int32_t* __restrict__ raw_out, int M, int N, int K, int* status, int after_quantizer) {
    using L = SmemLayout<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bars = base + L::OFF_BARS;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(base_ptr + L::OFF_TMEM);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::OFF_ABORT);
    const WaitCtl ctl{abort_flag, status, WAIT_LIMIT_NS};

    constexpr uint32_t TMEM_COLS = 2 * BN;      // 512 or 256: a power of two >= 32

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_a);
        prefetch_tensormap(&tm_b);
        if (!RAW_I32) prefetch_tensormap(&tm_out);
    }
    if (warp == 1) {
        tmem_alloc(base + L::OFF_TMEM, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    const int num_m = (M + BM - 1) / BM, num_n = (N + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_kb = (K + BK - 1) / BK;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            if (after_quantizer) grid_dep_wait();      // qa / s_tok come from the kernel before this one
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                const int m0 = (t % num_m) * BM, n0 = (t / num_m) * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctl, W_PRODUCER_EMPTY, kStatusTimeout)) { ok = false; break; }
                    mbar_arrive_expect_tx(full_bar(stage), L::STAGE_BYTES);
                    const uint32_t sa = base + stage * L::STAGE_BYTES;
                    tma_load_2d(sa, &tm_a, full_bar(stage), kb * BK, m0);
                    tma_load_2d(sa + L::A_BYTES, &tm_b, full_bar(stage), kb * BK, n0);
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // let copies that are still in flight land before the CTA goes away
                int s = stage;
                uint32_t ph = phase;
                for (int i = 0; i < STAGES && i < issued; ++i) {
                    if (s == 0) { s = STAGES; ph ^= 1u; }
                    --s;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(s), ph) && globaltimer_ns() - t0 < 10000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_i8_idesc(BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                if (!mbar_wait(tempty_bar(buf), ((it >> 1) & 1) ^ 1u, ctl, W_MMA_TMEM_EMPTY, kStatusTimeout)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, ctl, W_MMA_FULL, kStatusTimeout)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * L::STAGE_BYTES;
                    const uint64_t da = make_kmajor_sw128_desc(sa);
                    const uint64_t db = make_kmajor_sw128_desc(sa + L::A_BYTES);
                    const int ksteps = min(BK, K - kb * BK + MMA_K - 1) / MMA_K;   // skip all-zero tail steps
#pragma unroll
                    for (int k = 0; k < BK / MMA_K; ++k) {
                        if (k < ksteps)   // advancing K by 32 bytes inside the swizzled row: +2 in 16-byte units
                            mma_i8_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    tc_commit(empty_bar(stage));          // stage is free once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(tfull_bar(buf));        // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int lg = warp & 3;                       // TMEM lane group this warp may read: 32*lg .. 32*lg+31
        const int ep_tid = threadIdx.x - 64;
        float* sm_sch = reinterpret_cast<float*>(base_ptr + L::OFF_SCH);
        float* sm_bias = reinterpret_cast<float*>(base_ptr + L::OFF_BIAS);
        const uint32_t staging = base + L::OFF_STAGING + (warp - 2) * L::STAGING_BYTES_PER_WARP;
        uint8_t* staging_ptr = base_ptr + L::OFF_STAGING + (warp - 2) * L::STAGING_BYTES_PER_WARP;
        const bool has_bias = bias != nullptr;
        if (after_quantizer) grid_dep_wait();          // s_tok comes from the kernel before this one
        bool ok = true;
        int it = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
            const int buf = it & 1;
            const int m0 = (t % num_m) * BM, n0 = (t / num_m) * BN;
            if (!RAW_I32) {
                asm volatile("bar.sync 1, 128;" ::: "memory");     // previous tile's readers are done
                for (int j = ep_tid; j < BN; j += EPI_THREADS) {
                    const int n = n0 + j;
                    sm_sch[j] = n < N ? __ldg(s_ch + n) : 0.f;
                    sm_bias[j] = (has_bias && n < N) ? __ldg(bias + n) : 0.f;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            const int row = m0 + lg * 32 + lane;
            const float st = (!RAW_I32 && row < M) ? __ldg(s_tok + row) : 0.f;
            if (ok && !mbar_wait(tfull_bar(buf), (it >> 1) & 1, ctl, W_EPI_TMEM_FULL, kStatusTimeout)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) continue;                         // keep taking the named barriers, skip the work
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 64; ++c) {
                uint32_t v0[32], v1[32];
                tmem_ld_32x32b_x32(t_row + c * 64, v0);
                tmem_ld_32x32b_x32(t_row + c * 64 + 32, v1);
                tmem_wait_ld();
                if (c == BN / 64 - 1) {                // accumulator fully read: hand the buffer back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(buf));
                }
                if (RAW_I32) {
                    if (row < M) {
                        int32_t* dst = raw_out + static_cast<int64_t>(row) * N + n0 + c * 64;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (n0 + c * 64 + j < N) dst[j] = static_cast<int32_t>(v0[j]);
                            if (n0 + c * 64 + 32 + j < N) dst[32 + j] = static_cast<int32_t>(v1[j]);
                        }
                    }
                } else {
                    uint32_t packed[32];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        // columns c*64 + 2j, +1 (from v0) and c*64 + 32 + 2j, +1 (from v1)
                        const float2 sc0 = *reinterpret_cast<const float2*>(sm_sch + c * 64 + 2 * j);
                        const float2 sc1 = *reinterpret_cast<const float2*>(sm_sch + c * 64 + 32 + 2 * j);
                        float a0 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(v0[2 * j])), st), sc0.x);
                        float a1 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(v0[2 * j + 1])), st), sc0.y);
                        float b0 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(v1[2 * j])), st), sc1.x);
                        float b1 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int>(v1[2 * j + 1])), st), sc1.y);
                        if (has_bias) {
                            const float2 bi0 = *reinterpret_cast<const float2*>(sm_bias + c * 64 + 2 * j);
                            const float2 bi1 = *reinterpret_cast<const float2*>(sm_bias + c * 64 + 32 + 2 * j);
                            a0 = __fadd_rn(a0, bi0.x); a1 = __fadd_rn(a1, bi0.y);
                            b0 = __fadd_rn(b0, bi1.x); b1 = __fadd_rn(b1, bi1.y);
                        }
                        packed[j] = pack_bf16x2(a0, a1);
                        packed[16 + j] = pack_bf16x2(b0, b1);
                    }
                    // the previous TMA store must have finished reading the staging buffer
                    if (lane == 0) bulk_wait_group_read<0>();
                    __syncwarp();
                    // row `lane` of the 32 x 128-byte box; 16-byte chunk i lives at chunk (i ^ (row & 7))
                    uint8_t* srow = staging_ptr + lane * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        uint4 q = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
                        *reinterpret_cast<uint4*>(srow + ((i ^ (lane & 7)) << 4)) = q;
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tm_out, staging, n0 + c * 64, m0 + lg * 32);
                        bulk_commit_group();
                    }
                }
            }
        }
        if (!RAW_I32 && lane == 0) bulk_wait_group<0>();
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---------------------------------------------------------------------------- host side

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeFn>(p);
    }();
    return fn;
}

// 2-D row-major tensor [rows, cols] of `elem_bytes`-sized elements, row stride ld_bytes, box [box_rows, box_cols], 128-byte swizzle.
bool encode_2d(CUtensorMap* tm, CUtensorMapDataType dt, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld_bytes,
               uint32_t box_rows, uint32_t box_cols) {
    EncodeFn enc = get_encode();
    if (enc == nullptr) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcConfig {
    const char* name;
    int bn, stages;
};
constexpr TcConfig kConfigs[] = {
    {"tc 128x256 4 stages", 256, 4},
    {"tc 128x128 6 stages", 128, 6},
};
constexpr int kNumConfigs = sizeof(kConfigs) / sizeof(kConfigs[0]);

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

template <int BN, int STAGES, bool RAW>
int launch_cfg(const GemmArgs& a, cudaStream_t st) {
    using L = SmemLayout<BN, STAGES>;
    static_assert(L::DYN_BYTES <= 232448, "shared memory budget");
    auto kern = gemm_tc_kernel<BN, STAGES, RAW>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] { attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES); });
    if (attr_err != cudaSuccess) return 6;

    CUtensorMap tm_a, tm_b, tm_out;
    if (!encode_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.qa, a.M, a.K, a.lda_q, BM, BK)) return 6;
    if (!encode_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.qw, a.N, a.K, a.K, BN, BK)) return 6;
    if (RAW) {
        tm_out = tm_a;   // unused
    } else {
        if (!encode_2d(&tm_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.out, a.M, a.N, a.ldo * 2, 32, 64)) return 6;
    }
    const int num_tiles = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(num_tiles < sm_count() ? num_tiles : sm_count());
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = L::DYN_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.after_quantizer ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_out, a.s_tok, a.s_ch, a.bias,
                                       RAW ? static_cast<int32_t*>(a.out) : nullptr, a.M, a.N, a.K, a.status,
                                       a.after_quantizer ? 1 : 0);
    return e == cudaSuccess ? 0 : 6;
}

template <bool RAW>
int launch_by_id(int id, const GemmArgs& a, cudaStream_t st) {
    switch (id) {
        case 0: return launch_cfg<256, 4, RAW>(a, st);
        case 1: return launch_cfg<128, 6, RAW>(a, st);
        default: return 1;
    }
}

int pick_config(int M, int N, int K) {
    (void)K;
    // small problems: more, smaller tiles fill the SMs better
    const long tiles256 = static_cast<long>((M + BM - 1) / BM) * ((N + 255) / 256);
    if (tiles256 < sm_count()) return 1;
    return 0;
}

} // namespace

int tc_num_configs() { return kNumConfigs; }
const char* tc_config_name(int id) { return (id >= 0 && id < kNumConfigs) ? kConfigs[id].name : nullptr; }

int launch_gemm_tc(const GemmArgs& a, int forced, cudaStream_t st) {
    const int id = (forced >= 0 && forced < kNumConfigs) ? forced : pick_config(a.M, a.N, a.K);
    return a.raw_i32 ? launch_by_id<true>(id, a, st) : launch_by_id<false>(id, a, st);
}

} // namespace w8a8
