// Row-wise symmetric absmax int8 quantizer (per-token for activations,
// per-channel for weights): HBM-bound, every input byte is read from memory once.
//
//   s    = amax > 0 ? amax / 127 : 1          (IEEE division)
//   q[k] = clamp(rne(x[k] / s), -127, 127)    (IEEE quotient, round half to even)
//
// Two kernels:
//   * quant_rows_staged_kernel (bf16 activations, the hot one): persistent CTAs stream groups of rows
//     through a ring of shared-memory stages filled by bulk async copies (cp.async.bulk, one per row,
//     completing on an mbarrier), several stages ahead of the warps that consume them, so that about
//     190 KB per SM are in flight without costing registers. A row is shared by WPR warps; each warp
//     makes two passes over its part of the row in shared memory (absmax, then quantize) with 128-bit
//     shared-memory loads and 64-bit global stores.
//   * quant_rows_kernel (fp32 weights, set-up; also bf16 rows too long for a stage): rows held in
//     registers between the two passes, 128-bit global loads.
#include "internal.h"
#include "ptx.cuh"
#include "quant_math.cuh"

#include <cuda_bf16.h>

#include <mutex>
#include <type_traits>

namespace w8a8 {
namespace {

// ------------------------------------------------------------------------------------------- arithmetic

// SmoothQuant hook: x'[k] = RN(float(x[k]) * mult[k]) before everything else. 8 smoothed values of a unit.
__device__ __forceinline__ void smooth8(const uint4& v, const float* __restrict__ mult8, float (&f)[8]) {
    const float4 m0 = __ldg(reinterpret_cast<const float4*>(mult8));
    const float4 m1 = __ldg(reinterpret_cast<const float4*>(mult8) + 1);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const float m[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __fmul_rn(__uint_as_float(w[i] << 16), m[2 * i]);
        f[2 * i + 1] = __fmul_rn(__uint_as_float(w[i] & 0xffff0000u), m[2 * i + 1]);
    }
}
__device__ __forceinline__ float absmax8f(const float (&f)[8], float m) {
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(f[i]));
    return m;
}
__device__ __forceinline__ uint64_t quant2f(float lo, float hi, const RowScale2& r2) {
    const uint64_t x = pack2(lo, hi);
    const uint64_t q0 = mul2(x, r2.inv);
    const uint64_t r0 = fma2(r2.neg_s, q0, x);
    const uint64_t q1 = fma2(r0, r2.inv, q0);
    const uint64_t r1 = fma2(r2.neg_s, q1, x);
    const uint64_t q2 = fma2(r1, r2.inv, q1);
    return add2(q2, r2.magic);
}
__device__ __forceinline__ uint2 quant8f(const float (&f)[8], const RowScale& rs, const RowScale2& r2) {
    if (rs.fast)
        return make_uint2(gather4(quant2f(f[0], f[1], r2), quant2f(f[2], f[3], r2)),
                          gather4(quant2f(f[4], f[5], r2), quant2f(f[6], f[7], r2)));
    return make_uint2(quant4(f[0], f[1], f[2], f[3], rs), quant4(f[4], f[5], f[6], f[7], rs));
}

// ------------------------------------------------------------------------------------------- staged kernel

constexpr int SG_WARPS = 16;                         // consumer warps per CTA (one more warp produces)
constexpr int SG_THREADS = (SG_WARPS + 1) * 32;
constexpr int SG_SMEM_BUDGET = 200 * 1024;           // shared memory for the rings of one SM
constexpr int SG_SMEM_MAX = 226 * 1024;              // all a CTA can have: only for rows too long for the budget above

// Where time-outs go and how long a wait may last (every wait is bounded, as everywhere), plus the test hook.
struct QuantCtl {
    int* status;            // workspace status word this kernel resets, or nullptr (standalone quantizer)
    int* sticky;            // device-wide sticky status word, or nullptr
    uint64_t wait_limit_ns;
    int starve;             // test hook: the producer of every CTA withholds its first row group
    int feed_lanes;         // > 0: a barrier pair per row slot, fed by this many lanes of the producer warp (slot r by
                            // lane r % feed_lanes); 0: a barrier pair per stage, fed by lane 0
};

__device__ __forceinline__ void bulk_load_row(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(bar) : "memory");
}

// WPR consumer warps share a row (power of two <= SG_WARPS); a stage holds RPS = SG_WARPS / WPR rows.
// SMOOTH: multiply every element by mult[k] first (SmoothQuant hook).
// GIVEN: the absmax of every row is handed in (amax_in, written by the producer of the activations, possibly the
// kernel just ahead in the stream): the search pass and the exchange between the row's warps fall away.
template <int WPR, bool SMOOTH, bool GIVEN>
__global__ void __launch_bounds__(SG_THREADS, 2)
quant_rows_staged_kernel(const __nv_bfloat16* __restrict__ x, int64_t ld, int rows, int K,
                         int8_t* __restrict__ q, float* __restrict__ s_out, const QuantCtl qc, int num_stages,
                         const float* __restrict__ mult, const float* amax_in) {
    int* const status = qc.status;
    // a dependent kernel (the GEMM) may set itself up while this one runs; it waits for this grid before reading
    grid_dep_launch_dependents();

    constexpr int RPS = SG_WARPS / WPR;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t row_bytes = static_cast<uint32_t>(K) * 2u;
    const uint32_t stage_bytes = RPS * row_bytes;
    // after the ring: full[num_stages][BPS], empty[num_stages][BPS], partial maxima, abort flag. With ROW_BARS
    // every row slot of a stage has its own pair of barriers: a row is worked on as soon as it has landed and handed
    // back as soon as its warps are done with it, so neither the first row of a launch nor the last one waits for the
    // others of its stage. The launcher keeps one pair per stage where that measured faster (long rows in short rings).
    const bool ROW_BARS = qc.feed_lanes > 0;
    const int BPS = ROW_BARS ? RPS : 1;
    const uint32_t bars = base + num_stages * stage_bytes;
    const int num_slots = num_stages * BPS;
    auto full_bar = [&](int s, int slot) { return bars + 8u * (s * BPS + (ROW_BARS ? slot : 0)); };
    auto empty_bar = [&](int s, int slot) { return bars + 8u * (num_slots + s * BPS + (ROW_BARS ? slot : 0)); };
    float* s_red = reinterpret_cast<float*>(base_ptr + num_stages * stage_bytes + 16 * num_stages * RPS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_red + SG_WARPS);
    __shared__ int dummy_status;
    const WaitCtl ctl{abort_flag, status != nullptr ? status : &dummy_status, qc.sticky, qc.wait_limit_ns};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < num_slots; i += SG_THREADS) {
        mbar_init(bars + 8u * i, 1);                          // full: the producer's arrival with the row's byte count
        mbar_init(bars + 8u * (num_slots + i), ROW_BARS ? WPR : SG_WARPS);    // empty: the warps of the row / stage
    }
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        dummy_status = 0;
    }
    fence_mbar_init();
    __syncthreads();
    // This kernel may itself have been launched early, behind a kernel that allowed it (programmatic dependent
    // launch): everything above touched shared memory only; global memory is touched after that kernel is complete.
    grid_dep_wait();
    if (status != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *status = 0;

    // Every CTA takes a contiguous share of the rows, as even as the row count allows (not whole stages: with 2816 rows
    // on 148 CTAs that is 20 rows each instead of 16 or 24), and walks it in groups of up to RPS rows (one stage each).
    const int rows_per_cta = (rows + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const int r_begin = min(rows, static_cast<int>(blockIdx.x) * rows_per_cta);
    const int r_end = min(rows, r_begin + rows_per_cta);
    const int my_groups = (r_end - r_begin + RPS - 1) / RPS;

    if (warp == SG_WARPS) {
        // ---------------------------------------------------------------- producer
        // ROW_BARS: the row slots of every stage are dealt to feed_lanes lanes (short rows: one lane per slot, so
        // that the waits for the slots overlap instead of queueing behind one thread; longer rows: one lane, whose
        // copies leave one after another and keep the rows of a stage staggered); otherwise lane 0 feeds whole stages.
        const int feed_lanes = ROW_BARS ? qc.feed_lanes : 1;
        if (lane < feed_lanes) {
            int stage = 0;
            uint32_t phase = 0;
            bool withhold = qc.starve != 0;
            for (int g = 0; g < my_groups; ++g) {
                const int r0 = r_begin + g * RPS;
                const int nr = min(RPS, r_end - r0);
                if (ROW_BARS) {
                    bool go = true;
                    for (int r = lane; r < nr; r += feed_lanes) {
                        if (!mbar_wait(empty_bar(stage, r), phase ^ 1u, ctl, 1, kStatusTimeout)) { go = false; break; }
                        if (!withhold) {
                            mbar_arrive_expect_tx(full_bar(stage, r), row_bytes);
                            bulk_load_row(base + stage * stage_bytes + r * row_bytes,
                                          x + static_cast<int64_t>(r0 + r) * ld, row_bytes, full_bar(stage, r));
                        }
                    }
                    if (!go) break;
                } else {
                    if (!mbar_wait(empty_bar(stage, 0), phase ^ 1u, ctl, 1, kStatusTimeout)) break;
                    if (!withhold) {
                        mbar_arrive_expect_tx(full_bar(stage, 0), nr * row_bytes);
                        for (int r = 0; r < nr; ++r)
                            bulk_load_row(base + stage * stage_bytes + r * row_bytes,
                                          x + static_cast<int64_t>(r0 + r) * ld, row_bytes, full_bar(stage, 0));
                    }
                }
                // test hook (withhold): nothing is posted for the first group, so the consumers' bounded wait runs out
                withhold = false;
                if (++stage == num_stages) { stage = 0; phase ^= 1u; }
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        const int slot = warp / WPR, part = warp % WPR;       // row of the stage, share of that row
        const int units = K >> 3;                             // 8-element (16-byte) units per row
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int g = 0; g < my_groups; ++g) {
            const int row = r_begin + g * RPS + slot;
            // an absmax that is handed in is fetched while the row's bytes are still on their way (plain, coherent
            // load: the value may have been written by the kernel ahead while this one was already resident)
            float amax_given = 0.f;
            if (GIVEN && row < r_end) amax_given = __ldcg(amax_in + row);
            if (ok && (row < r_end || !ROW_BARS) && !mbar_wait(full_bar(stage, slot), phase, ctl, 2, kStatusTimeout)) ok = false;
            ok = __all_sync(0xffffffffu, ok) != 0;
            const bool live = ok && row < r_end;
            const uint4* srow = reinterpret_cast<const uint4*>(base_ptr + stage * stage_bytes + slot * row_bytes);
            float amax = 0.f;
            if (GIVEN) {
                amax = amax_given;
            } else if (SMOOTH) {
                if (live) {
#pragma unroll 2
                    for (int u = part * 32 + lane; u < units; u += WPR * 32) {
                        float f[8];
                        smooth8(srow[u], mult + u * 8, f);
                        amax = absmax8f(f, amax);
                    }
                }
            } else {
                __nv_bfloat162 m2 = __float2bfloat162_rn(0.f);
                if (live) {
#pragma unroll 3
                    for (int u = part * 32 + lane; u < units; u += WPR * 32) m2 = absmax8(srow[u], m2);
                }
                amax = unpack_max(m2);
            }
            if (!GIVEN) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            }
            if (WPR > 1 && !GIVEN) {
                // the WPR warps of a row exchange their partial maxima through shared memory
                if (lane == 0) s_red[warp] = amax;
                asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "n"(WPR * 32) : "memory");
#pragma unroll
                for (int w = 0; w < WPR; ++w) amax = fmaxf(amax, s_red[slot * WPR + w]);
                asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "n"(WPR * 32) : "memory");   // s_red may be rewritten
            }
            if (live) {
                const RowScale rs = make_row_scale(amax);
                const RowScale2 r2 = make_row_scale2(rs);
                if (part == 0 && lane == 0) s_out[row] = rs.s;
                uint2* qrow = reinterpret_cast<uint2*>(q + static_cast<int64_t>(row) * K);
                if (SMOOTH) {
#pragma unroll 2
                    for (int u = part * 32 + lane; u < units; u += WPR * 32) {
                        float f[8];
                        smooth8(srow[u], mult + u * 8, f);      // the same rounded products as in the first pass
                        qrow[u] = quant8f(f, rs, r2);
                    }
                } else {
#pragma unroll 3
                    for (int u = part * 32 + lane; u < units; u += WPR * 32) qrow[u] = quant8(srow[u], rs, r2);
                }
            }
            __syncwarp();
            if (lane == 0 && (row < r_end || !ROW_BARS)) mbar_arrive(empty_bar(stage, slot));    // done with its row / the stage
            if (++stage == num_stages) { stage = 0; phase ^= 1u; }
        }
    }
}

// ------------------------------------------------------------------------------------------- register kernel

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
    __device__ __forceinline__ float absmax() const {
        return unpack_max(absmax8(hi, absmax8(lo, __float2bfloat162_rn(0.f))));
    }
    __device__ __forceinline__ uint4 quantize(const RowScale& rs) const {
        const RowScale2 r2 = make_row_scale2(rs);
        const uint2 a = quant8(lo, rs, r2), b = quant8(hi, rs, r2);
        return make_uint4(a.x, a.y, b.x, b.y);
    }
};

template <> struct Chunk<float> {
    float4 v[4];
    __device__ __forceinline__ void load(const float* p) {
        const float4* q = reinterpret_cast<const float4*>(p);
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = __ldg(q + i);
    }
    // 16 bf16 values widened to fp32 (exact)
    __device__ __forceinline__ void load(const __nv_bfloat16* p) {
        const uint4* q = reinterpret_cast<const uint4*>(p);
        const uint4 lo = __ldg(q), hi = __ldg(q + 1);
        const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v[i] = make_float4(__uint_as_float(w[2 * i] << 16), __uint_as_float(w[2 * i] & 0xffff0000u),
                               __uint_as_float(w[2 * i + 1] << 16), __uint_as_float(w[2 * i + 1] & 0xffff0000u));
    }
    // SmoothQuant hook: one rounded multiply per element by its input channel's factor
    __device__ __forceinline__ void scale(const float* __restrict__ mult16) {
        const float4* m = reinterpret_cast<const float4*>(mult16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = __ldg(m + i);
            v[i] = make_float4(__fmul_rn(v[i].x, f.x), __fmul_rn(v[i].y, f.y), __fmul_rn(v[i].z, f.z), __fmul_rn(v[i].w, f.w));
        }
    }
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __device__ __forceinline__ float absmax() const {
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) m = fmaxf(fmaxf(m, fmaxf(fabsf(v[i].x), fabsf(v[i].y))), fmaxf(fabsf(v[i].z), fabsf(v[i].w)));
        return m;
    }
    __device__ __forceinline__ uint4 quantize(const RowScale& rs) const {
        return make_uint4(quant4(v[0].x, v[0].y, v[0].z, v[0].w, rs), quant4(v[1].x, v[1].y, v[1].z, v[1].w, rs),
                          quant4(v[2].x, v[2].y, v[2].z, v[2].w, rs), quant4(v[3].x, v[3].y, v[3].z, v[3].w, rs));
    }
};

// WPR warps per row (a power of two <= 16); a CTA works on RPC = 16 / WPR rows at a time. Rows with more
// than WPR*32*CPL chunks stream the surplus twice (absmax pass, then quantize pass) from memory / L2.
// SMOOTH (SmoothQuant hook): elements are widened to fp32 and multiplied by mult[k] as they are loaded.
template <typename T, int WPR, bool SMOOTH, bool GIVEN>
__global__ void __launch_bounds__(WARPS * 32, 1)
quant_rows_kernel(const T* __restrict__ x, int64_t ld, int rows, int K,
                  int8_t* __restrict__ q, float* __restrict__ s_out, int* status, const float* __restrict__ mult,
                  const float* amax_in) {
    using C = Chunk<typename std::conditional<SMOOTH, float, T>::type>;
    auto fetch = [&](C& c, const T* row, int chunk) {
        c.load(row + chunk * 16);
        if constexpr (SMOOTH) c.scale(mult + chunk * 16);
    };
    // Activations: a dependent kernel (the GEMM) may set itself up while this one runs; it waits for this grid before it
    // reads them. Weights (fp32 input) are different: the GEMM requests its first weight tiles before that wait, so the
    // kernel that writes them must not release its dependents before it is complete.
    if (!std::is_same<T, float>::value) grid_dep_launch_dependents();
    grid_dep_wait();                      // launched early behind a kernel that allowed it: wait for that kernel's results
    if (status != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *status = 0;

    constexpr int RPC = WARPS / WPR;
    constexpr int STRIDE = WPR * 32;
    __shared__ float s_red[WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot = warp / WPR, w_in_row = warp % WPR;
    const int nchunks = K >> 4;
    const int c0 = w_in_row * 32 + lane;

#pragma unroll 1
    for (int base = blockIdx.x * RPC; base < rows; base += gridDim.x * RPC) {
        const int row = base + slot;
        const bool live = row < rows;
        const T* xr = x + static_cast<int64_t>(live ? row : 0) * ld;
        C reg[CPL];
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
            const int c = c0 + i * STRIDE;
            if (live && c < nchunks) fetch(reg[i], xr, c); else reg[i].zero();
        }
        if (GIVEN) {
            if (live) amax = __ldcg(amax_in + row);
        } else {
#pragma unroll
            for (int i = 0; i < CPL; ++i) amax = fmaxf(amax, reg[i].absmax());
            if (live) {
                for (int c = c0 + CPL * STRIDE; c < nchunks; c += STRIDE) {   // surplus chunks (very long rows)
                    C t;
                    fetch(t, xr, c);
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
        }
        if (live) {
            const RowScale s = make_row_scale(amax);
            if (w_in_row == 0 && lane == 0) s_out[row] = s.s;
            int8_t* qr = q + static_cast<int64_t>(row) * K;
#pragma unroll
            for (int i = 0; i < CPL; ++i) {
                const int c = c0 + i * STRIDE;
                if (c < nchunks) *reinterpret_cast<uint4*>(qr + c * 16) = reg[i].quantize(s);
            }
            for (int c = c0 + CPL * STRIDE; c < nchunks; c += STRIDE) {
                C t;
                fetch(t, xr, c);
                *reinterpret_cast<uint4*>(qr + c * 16) = t.quantize(s);
            }
        }
        if (WPR > 1 && !GIVEN) __syncthreads();    // s_red may be rewritten by the next sweep
    }
}

// ------------------------------------------------------------------------------------------- host side

// Launch that may start while the kernel ahead of it in the stream is still finishing (if that kernel allows it);
// the kernels above wait for it with griddepcontrol.wait before they touch global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// amax: the rows' absmax handed in (one pass), or nullptr (the kernel searches for it). Not combined with mult.
template <typename T, int WPR>
cudaError_t launch_reg(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status, const float* mult,
                       const float* amax, cudaStream_t st) {
    constexpr int RPC = WARPS / WPR;
    const int units = (rows + RPC - 1) / RPC;
    const int cap = sm_count() * 2;
    const int grid = units < cap ? units : cap;
    const float* none = nullptr;
    if (amax != nullptr)
        return launch_pdl(quant_rows_kernel<T, WPR, false, true>, grid, WARPS * 32, 0, st, x, ld, rows, K, q, s, status, none, amax);
    if (mult != nullptr)
        return launch_pdl(quant_rows_kernel<T, WPR, true, false>, grid, WARPS * 32, 0, st, x, ld, rows, K, q, s, status, mult, none);
    return launch_pdl(quant_rows_kernel<T, WPR, false, false>, grid, WARPS * 32, 0, st, x, ld, rows, K, q, s, status, none, none);
}

template <typename T>
cudaError_t dispatch_reg(const T* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status, const float* mult,
                         const float* amax, cudaStream_t st) {
    const int nchunks = K / 16;
    // fewest warps per row that keep the whole row in registers (<= CPL chunks per lane)
    if (nchunks <= 32 * CPL)  return launch_reg<T, 1>(x, ld, rows, K, q, s, status, mult, amax, st);
    if (nchunks <= 64 * CPL)  return launch_reg<T, 2>(x, ld, rows, K, q, s, status, mult, amax, st);
    if (nchunks <= 128 * CPL) return launch_reg<T, 4>(x, ld, rows, K, q, s, status, mult, amax, st);
    if (nchunks <= 256 * CPL) return launch_reg<T, 8>(x, ld, rows, K, q, s, status, mult, amax, st);
    return launch_reg<T, 16>(x, ld, rows, K, q, s, status, mult, amax, st);
}

template <int WPR>
cudaError_t launch_staged(const __nv_bfloat16* x, int64_t ld, int rows, int K, int8_t* q, float* s, int* status,
                          const float* mult, const float* amax, cudaStream_t st) {
    constexpr int RPS = SG_WARPS / WPR;
    const int stage_bytes = RPS * K * 2;
    const int groups = (rows + RPS - 1) / RPS;
    // With plenty of row groups two CTAs per SM (half the ring each) hide latencies better; with few, one
    // CTA per SM with the whole ring gets more stages ahead.
    const int ctas_per_sm = (groups >= 8 * sm_count() && SG_SMEM_BUDGET / 2 >= 2 * stage_bytes) ? 2 : 1;
    int num_stages = SG_SMEM_BUDGET / ctas_per_sm / stage_bytes;
    if (num_stages > 8) num_stages = 8;
    // very long rows (one row per stage, 64-113 KB): two stages out of everything a CTA can have
    if (num_stages < 2 && 2 * stage_bytes + 1024 <= SG_SMEM_MAX) num_stages = 2;
    // the ring indices of the kernel wrap at num_stages: a ring of fewer than two stages must never be launched
    if (num_stages < 2) return cudaErrorInvalidConfiguration;
    const int smem = num_stages * stage_bytes + 16 * num_stages * RPS + SG_WARPS * 4 + 16 + 128;
    static PerDeviceOnce smem_opt_in;
    const cudaError_t attr_err = smem_opt_in.run([] {
        cudaError_t e = cudaFuncSetAttribute(quant_rows_staged_kernel<WPR, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             SG_SMEM_MAX);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(quant_rows_staged_kernel<WPR, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     SG_SMEM_MAX);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(quant_rows_staged_kernel<WPR, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     SG_SMEM_MAX);
        return e;
    });
    if (attr_err != cudaSuccess) return attr_err;
    const int cap = ctas_per_sm * sm_count();
    // few rows: CTAs of as little as a quarter of a stage's rows each, so that more SMs share the work (M = 512,
    // K = 12288: 14.8 -> 5.5 us; M = 256, K = 3072: 6.8 -> 5.2 us, which is the host's launch rate)
    const int rmin = RPS >= 4 ? RPS / 4 : 1;
    const int want = (rows + rmin - 1) / rmin;
    const int grid = want < cap ? want : cap;
    const float* none = nullptr;
    // Barrier granularity and the lanes that feed the ring, from timings of back-to-back launches on B200: a pair of
    // barriers per row wherever the ring is long (one CTA per SM) or the rows are short; per stage for rows above
    // 4 KB in the half-size rings of two CTAs per SM. Short rows want a feeding lane per row slot (one thread's
    // wait-and-issue per row is what limits them), rows of 6 KB and more one or two.
    const int row_bytes = K * 2;
    int feed_lanes;
    if (row_bytes <= 2048)      feed_lanes = RPS;
    else if (row_bytes <= 4096) feed_lanes = 4;
    else if (ctas_per_sm == 2)  feed_lanes = 0;
    else                        feed_lanes = WPR <= 4 ? 2 : 1;
    if (feed_lanes > RPS) feed_lanes = RPS;
    const QuantCtl qc{status, sticky_status_word(), wait_limit_ns(), starve_mode() == kStarveQuant ? 1 : 0, feed_lanes};
    if (amax != nullptr)
        return launch_pdl(quant_rows_staged_kernel<WPR, false, true>, grid, SG_THREADS, smem, st, x, ld, rows, K, q, s, qc, num_stages, none, amax);
    if (mult != nullptr)
        return launch_pdl(quant_rows_staged_kernel<WPR, true, false>, grid, SG_THREADS, smem, st, x, ld, rows, K, q, s, qc, num_stages, mult, none);
    return launch_pdl(quant_rows_staged_kernel<WPR, false, false>, grid, SG_THREADS, smem, st, x, ld, rows, K, q, s, qc, num_stages, none, none);
}

} // namespace

cudaError_t launch_quantize_bf16(const void* A, int64_t lda, int M, int K, const float* mult, const float* amax, int8_t* qa,
                                 float* s_tok, int* status_to_clear, cudaStream_t st) {
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(A);
    // a warp handles up to 4 KB of a row (measured best among 1-16 KB); rows of up to 64 KB (K <= 32768) go
    // through the staged kernel with several stages, rows of up to 113 KB with two stages of one row each (a warp
    // then walks up to 7 KB), longer ones through the register kernel
    const int row_bytes = K * 2;
    if (row_bytes <= 2048)  return launch_staged<1>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);   // 16 rows per stage
    if (row_bytes <= 8192)  return launch_staged<2>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);   // 8 rows per stage
    if (row_bytes <= 16384) return launch_staged<4>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);
    if (row_bytes <= 32768) return launch_staged<8>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);
    if (2 * row_bytes + 1024 <= SG_SMEM_MAX) return launch_staged<16>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);
    return dispatch_reg<__nv_bfloat16>(x, lda, M, K, qa, s_tok, status_to_clear, mult, amax, st);
}

cudaError_t launch_quantize_f32(const float* W, int64_t ldw, int N, int K, const float* mult, int8_t* qw, float* s_ch,
                                cudaStream_t st) {
    return dispatch_reg<float>(W, ldw, N, K, qw, s_ch, nullptr, mult, nullptr, st);
}

} // namespace w8a8
