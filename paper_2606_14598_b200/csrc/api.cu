// C ABI of the library: argument validation, workspace layout, dispatch.
// No device memory is allocated here and nothing falls back to the CPU.
#include "../../include/w8a8_linear.h"
#include "internal.h"

#include <nvtx3/nvToolsExt.h>

#include <atomic>
#include <cstdint>
#include <mutex>

namespace {

using namespace w8a8;

constexpr size_t kStatusBlock = 256;
// kSkinnyM (internal.h): at or below this many tokens the weight-streaming path runs (measured: it wins up to 4-8
// tokens, the tensor-core path from 16 on)

std::atomic<int> g_forced_config{-1};
std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};     // 2 s
std::atomic<int> g_starve{0};
std::atomic<int> g_small_mode{-1};

// The one-kernel path takes bf16 activations without SmoothQuant factors; chosen by shape unless a test says otherwise.
bool use_small_path(int a_dtype, const float* a_mult, int forced, int64_t M, int64_t N, int64_t K) {
    if (a_dtype != W8A8_ACT_BF16 || a_mult != nullptr) return false;
    const int mode = g_small_mode.load();
    if (mode == 0) return false;
    if (mode == 1) return small_fused_eligible(M, N, K);
    return forced < 0 && small_fused_preferred(M, N, K);
}

// First time-out recorded by any kernel of this library on the device, kept until the host clears it. (The status
// word of a workspace is reset by every call on that workspace; this one is not.) Zero when the module is loaded.
__device__ int g_sticky_status;
std::mutex g_sticky_mutex;
int* g_sticky_ptr[64] = {};

// A named range around the enqueueing of a call, for timelines of profilers that read NVTX (header-only: it costs a
// few nanoseconds when no tool is attached).
struct Range {
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The kernels are built for sm_100a only: tcgen05.mma.kind::i8 exists on compute capability 10.0 and not, for
// instance, on 10.3.
int check_arch() {
    static thread_local int cached_dev = -1;
    static thread_local int cached_ok = 0;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return W8A8_ERR_CUDA;
    if (dev != cached_dev) {
        int major = 0, minor = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
            return W8A8_ERR_CUDA;
        cached_dev = dev;
        cached_ok = (major == 10 && minor == 0);
    }
    return cached_ok ? W8A8_OK : W8A8_ERR_ARCH;
}

int check_dims(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return W8A8_ERR_INVALID_ARG;
    if (M > INT32_MAX || N > INT32_MAX) return W8A8_ERR_INVALID_ARG;
    if (K > W8A8_K_MAX) return W8A8_ERR_K_OVERFLOW;
    if (K % 16 != 0) return W8A8_ERR_ALIGNMENT;
    return W8A8_OK;
}

// workspace for bf16 activations: [status 256 B][s_tok, padded to 256 B][qa]
void offsets(int64_t M, size_t* s_tok_off, size_t* qa_off) {
    *s_tok_off = kStatusBlock;
    *qa_off = *s_tok_off + round_up(static_cast<size_t>(M) * sizeof(float), 256);
}

} // namespace

namespace w8a8 {

uint64_t wait_limit_ns() { return g_wait_limit_ns.load(); }
int starve_mode() { return g_starve.load(); }
int small_path_mode() { return g_small_mode.load(); }

int* sticky_status_word() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_sticky_mutex);
    if (g_sticky_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_sticky_status) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
        g_sticky_ptr[dev] = static_cast<int*>(p);
    }
    return g_sticky_ptr[dev];
}

} // namespace w8a8

extern "C" {

uint64_t int8_debug_set_wait_limit_ns(uint64_t limit_ns) {
    if (limit_ns == 0) limit_ns = 2000000000ull;
    return g_wait_limit_ns.exchange(limit_ns);
}

int int8_debug_set_small_path(int mode) {
    if (mode < -1 || mode > 1) return -2;
    return g_small_mode.exchange(mode);
}

int int8_debug_set_starve(int mode) {
    if (mode != 0 && mode != kStarveGemm && mode != kStarveQuant) return -1;
    return g_starve.exchange(mode);
}

int int8_sticky_status(int clear, void* stream) {
    if (int e = check_arch()) return e;
    int* word = sticky_status_word();
    if (word == nullptr) return W8A8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int v = 0;
    if (cudaMemcpyAsync(&v, word, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return W8A8_ERR_CUDA;
    if (clear && cudaMemsetAsync(word, 0, sizeof(int), st) != cudaSuccess) return W8A8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return W8A8_ERR_CUDA;
    return v & 0xff;
}

const char* int8_status_string(int status) {
    switch (status) {
        case W8A8_OK: return "ok";
        case W8A8_ERR_INVALID_ARG: return "invalid argument";
        case W8A8_ERR_ALIGNMENT: return "alignment: pointers must be 16-byte aligned, K % 16 == 0, N % 8 == 0, row strides multiples of 16 bytes";
        case W8A8_ERR_K_OVERFLOW: return "K too large: K * 127^2 must stay below 2^31";
        case W8A8_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case W8A8_ERR_ARCH: return "device is not sm_100 (B200)";
        case W8A8_ERR_CUDA: return "CUDA call failed";
        case W8A8_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown status";
    }
}

int int8_linear_force_config(int config_id) { return g_forced_config.exchange(config_id); }
int int8_linear_num_configs(void) { return tc_num_configs() + 1; }
const char* int8_linear_config_name(int config_id) {
    if (config_id == tc_num_configs()) return "simt dp4a (skinny M / cross-check)";
    if (config_id == tc_num_configs() + 1) return "one kernel: quantizer + tc 128x32 per CTA (small problems)";
    return tc_config_name(config_id);
}

static int quantize_weight_impl(const float* W, int64_t N, int64_t K, int64_t ldw, const float* mult,
                                int8_t* qw, float* s_ch, void* stream) {
    const Range range("w8a8 quantize weight per channel");
    if (W == nullptr || qw == nullptr || s_ch == nullptr) return W8A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0 || N > INT32_MAX || K > INT32_MAX || ldw < K) return W8A8_ERR_INVALID_ARG;
    if (K % 16 != 0 || ldw % 4 != 0 || !aligned16(W) || !aligned16(qw) || !aligned16(mult)) return W8A8_ERR_ALIGNMENT;
    if (int e = check_arch()) return e;
    cudaError_t ce = launch_quantize_f32(W, ldw, static_cast<int>(N), static_cast<int>(K), mult, qw, s_ch,
                                         static_cast<cudaStream_t>(stream));
    return ce == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
}

static int quantize_act_impl(const void* A_bf16, int64_t M, int64_t K, int64_t lda, const float* mult, const float* amax,
                             int8_t* qa, float* s_tok, void* stream) {
    const Range range("w8a8 quantize act per token");
    if (A_bf16 == nullptr || qa == nullptr || s_tok == nullptr) return W8A8_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || M > INT32_MAX || K > INT32_MAX || lda < K) return W8A8_ERR_INVALID_ARG;
    if (K % 16 != 0 || lda % 8 != 0 || !aligned16(A_bf16) || !aligned16(qa) || !aligned16(mult)) return W8A8_ERR_ALIGNMENT;
    if (int e = check_arch()) return e;
    cudaError_t ce = launch_quantize_bf16(A_bf16, lda, static_cast<int>(M), static_cast<int>(K), mult, amax, qa, s_tok, nullptr,
                                          static_cast<cudaStream_t>(stream));
    return ce == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
}

int int8_quantize_weight_per_channel(const float* W, int64_t N, int64_t K, int64_t ldw,
                                     int8_t* qw, float* s_ch, void* stream) {
    return quantize_weight_impl(W, N, K, ldw, nullptr, qw, s_ch, stream);
}

int int8_quantize_weight_per_channel_smooth(const float* W, int64_t N, int64_t K, int64_t ldw, const float* w_mult,
                                            int8_t* qw, float* s_ch, void* stream) {
    if (w_mult == nullptr) return W8A8_ERR_INVALID_ARG;
    return quantize_weight_impl(W, N, K, ldw, w_mult, qw, s_ch, stream);
}

int int8_quantize_act_per_token(const void* A_bf16, int64_t M, int64_t K, int64_t lda,
                                int8_t* qa, float* s_tok, void* stream) {
    return quantize_act_impl(A_bf16, M, K, lda, nullptr, nullptr, qa, s_tok, stream);
}

int int8_quantize_act_per_token_given_absmax(const void* A_bf16, int64_t M, int64_t K, int64_t lda, const float* rowmax,
                                             int8_t* qa, float* s_tok, void* stream) {
    if (rowmax == nullptr) return W8A8_ERR_INVALID_ARG;
    return quantize_act_impl(A_bf16, M, K, lda, nullptr, rowmax, qa, s_tok, stream);
}

int int8_quantize_act_per_token_smooth(const void* A_bf16, int64_t M, int64_t K, int64_t lda, const float* a_mult,
                                       int8_t* qa, float* s_tok, void* stream) {
    if (a_mult == nullptr) return W8A8_ERR_INVALID_ARG;
    return quantize_act_impl(A_bf16, M, K, lda, a_mult, nullptr, qa, s_tok, stream);
}

size_t int8_linear_workspace_min_bytes(int64_t M, int64_t N, int64_t K, int a_dtype) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    if (a_dtype == W8A8_ACT_INT8) return kStatusBlock;
    if (a_dtype != W8A8_ACT_BF16) return 0;
    size_t s_off, q_off;
    offsets(M, &s_off, &q_off);
    return q_off + round_up(static_cast<size_t>(M) * static_cast<size_t>(K), 256);
}

size_t int8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dtype) {
    const size_t base = int8_linear_workspace_min_bytes(M, N, K, a_dtype);
    if (base == 0 || M <= kSkinnyM || M > INT32_MAX || N > INT32_MAX || K > W8A8_K_MAX) return base;
    // room for the partial accumulators of the K-split, where the automatic choice would use one
    return base + round_up(tc_max_scratch_bytes(static_cast<int>(M), static_cast<int>(N), static_cast<int>(K)), 256);
}

int int8_linear_plan(int64_t M, int64_t N, int64_t K, int a_dtype, size_t workspace_bytes,
                     int* config_id, int* cta_groups, int* split_tiles, int* split_parts) {
    if (int e = check_dims(M, N, K)) return e;
    const size_t base = int8_linear_workspace_min_bytes(M, N, K, a_dtype);
    if (base == 0) return W8A8_ERR_INVALID_ARG;
    if (workspace_bytes < base) return W8A8_ERR_WORKSPACE;
    // no device needed: the plan depends on the SM count only (148 is assumed when no device can be queried)
    const int forced = g_forced_config.load();
    TcPlan plan{};
    if (use_small_path(a_dtype, nullptr, forced, M, N, K)) {
        plan.config = tc_num_configs() + 1;
        plan.groups = static_cast<int>((N + 31) / 32);
    } else if ((forced < 0 && M <= kSkinnyM) || (forced >= 0 && (forced & 0xff) == tc_num_configs())) {
        plan.config = tc_num_configs();
    } else {
        plan = tc_plan(static_cast<int>(M), static_cast<int>(N), static_cast<int>(K), forced, workspace_bytes - base);
    }
    if (config_id) *config_id = plan.config;
    if (cta_groups) *cta_groups = plan.groups;
    if (split_tiles) *split_tiles = plan.split_tiles;
    if (split_parts) *split_parts = plan.split_parts;
    return W8A8_OK;
}

void int8_linear_workspace_offsets(int64_t M, int64_t K, size_t* s_tok_offset, size_t* qa_offset) {
    (void)K;
    size_t s_off, q_off;
    offsets(M, &s_off, &q_off);
    if (s_tok_offset) *s_tok_offset = s_off;
    if (qa_offset) *qa_offset = q_off;
}

// a_mult: SmoothQuant factors for bf16 activations, or nullptr. amax_in: the absmax of every row of bf16 activations,
// handed in (one-pass quantizer), or nullptr. rowmax_out: receives the absmax of every output row, or nullptr.
static int fused_impl(const void* A, int a_dtype, int64_t lda, const float* s_tok_in, const float* a_mult, const float* amax_in,
                      const int8_t* qw, const float* s_ch, const float* bias,
                      void* out_bf16, int64_t ldo, float* rowmax_out, int64_t M, int64_t N, int64_t K,
                      void* workspace, size_t workspace_bytes, void* stream) {
    const Range range("w8a8 linear fused");
    if (A == nullptr || qw == nullptr || s_ch == nullptr || out_bf16 == nullptr) return W8A8_ERR_INVALID_ARG;
    if (!aligned16(a_mult)) return W8A8_ERR_ALIGNMENT;
    if (a_dtype != W8A8_ACT_BF16 && a_dtype != W8A8_ACT_INT8) return W8A8_ERR_INVALID_ARG;
    if ((a_dtype == W8A8_ACT_INT8) != (s_tok_in != nullptr)) return W8A8_ERR_INVALID_ARG;
    if (int e = check_dims(M, N, K)) return e;
    if (lda < K || ldo < N) return W8A8_ERR_INVALID_ARG;
    const int64_t lda_bytes = lda * (a_dtype == W8A8_ACT_BF16 ? 2 : 1);
    if (N % 8 != 0 || ldo % 8 != 0 || lda_bytes % 16 != 0) return W8A8_ERR_ALIGNMENT;
    if (!aligned16(A) || !aligned16(qw) || !aligned16(out_bf16)) return W8A8_ERR_ALIGNMENT;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 ||
        workspace_bytes < int8_linear_workspace_min_bytes(M, N, K, a_dtype))
        return W8A8_ERR_WORKSPACE;
    if (int e = check_arch()) return e;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    const int forced = g_forced_config.load();
    if (use_small_path(a_dtype, a_mult, forced, M, N, K)) {
        if (rowmax_out != nullptr && cudaMemsetAsync(rowmax_out, 0, static_cast<size_t>(M) * sizeof(float), st) != cudaSuccess)
            return W8A8_ERR_CUDA;
        GemmArgs g{};
        g.rowmax = rowmax_out;
        g.qw = qw; g.s_ch = s_ch; g.bias = bias; g.out = out_bf16; g.ldo = ldo;
        g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
        g.status = status;
        size_t s_off, q_off;
        offsets(M, &s_off, &q_off);
        return launch_small_fused(A, lda, amax_in, g, reinterpret_cast<int8_t*>(ws + q_off),
                                  reinterpret_cast<float*>(ws + s_off), st) == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
    }
    const bool simt = (forced < 0 && M <= kSkinnyM) || (forced >= 0 && (forced & 0xff) == tc_num_configs());
    // whatever the workspace holds beyond the required part is scratch for the K-split of the partial wave
    const size_t scratch_off = int8_linear_workspace_min_bytes(M, N, K, a_dtype);
    TcPlan plan{};
    if (!simt) {
        plan = tc_plan(static_cast<int>(M), static_cast<int>(N), static_cast<int>(K), forced, workspace_bytes - scratch_off);
        // arrival counters and partial sums start at zero (ahead of the quantizer, so the GEMM still launches right behind it)
        if (plan.split_parts >= 2 && cudaMemsetAsync(ws + scratch_off, 0, plan.scratch_bytes, st) != cudaSuccess)
            return W8A8_ERR_CUDA;
    }
    // the row maxima are merged with atomic maxima by every tile of a row block: they start at zero
    if (rowmax_out != nullptr && cudaMemsetAsync(rowmax_out, 0, static_cast<size_t>(M) * sizeof(float), st) != cudaSuccess)
        return W8A8_ERR_CUDA;

    GemmArgs g{};
    g.rowmax = rowmax_out;
    g.qw = qw; g.s_ch = s_ch; g.bias = bias; g.out = out_bf16; g.ldo = ldo;
    g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
    g.raw_i32 = false; g.status = status; g.split_ws = plan.split_parts >= 2 ? ws + scratch_off : nullptr;
    if (a_dtype == W8A8_ACT_BF16) {
        size_t s_off, q_off;
        offsets(M, &s_off, &q_off);
        float* s_tok = reinterpret_cast<float*>(ws + s_off);
        int8_t* qa = reinterpret_cast<int8_t*>(ws + q_off);
        // the quantizer clears the status word; the GEMM behind it (programmatic dependent launch) sets
        // itself up while the quantizer runs and waits for it before its first read
        if (launch_quantize_bf16(A, lda, g.M, g.K, a_mult, amax_in, qa, s_tok, status, st) != cudaSuccess) return W8A8_ERR_CUDA;
        g.qa = qa; g.lda_q = K; g.s_tok = s_tok; g.after_quantizer = true;
    } else {
        g.qa = static_cast<const int8_t*>(A); g.lda_q = lda; g.s_tok = s_tok_in; g.after_quantizer = false;
    }
    if (simt) return launch_gemm_simt(g, st) == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
    return launch_gemm_tc(g, plan, st);
}

int int8_linear_fused(const void* A, int a_dtype, int64_t lda, const float* s_tok_in,
                      const int8_t* qw, const float* s_ch, const float* bias,
                      void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                      void* workspace, size_t workspace_bytes, void* stream) {
    return fused_impl(A, a_dtype, lda, s_tok_in, nullptr, nullptr, qw, s_ch, bias, out_bf16, ldo, nullptr, M, N, K,
                      workspace, workspace_bytes, stream);
}

int int8_linear_fused_rowmax(const void* A, int a_dtype, int64_t lda, const float* s_tok_in,
                             const int8_t* qw, const float* s_ch, const float* bias,
                             void* out_bf16, int64_t ldo, float* rowmax_out, int64_t M, int64_t N, int64_t K,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (rowmax_out == nullptr) return W8A8_ERR_INVALID_ARG;
    return fused_impl(A, a_dtype, lda, s_tok_in, nullptr, nullptr, qw, s_ch, bias, out_bf16, ldo, rowmax_out, M, N, K,
                      workspace, workspace_bytes, stream);
}

int int8_linear_fused_given_absmax(const void* A_bf16, int64_t lda, const float* rowmax_in,
                                   const int8_t* qw, const float* s_ch, const float* bias,
                                   void* out_bf16, int64_t ldo, float* rowmax_out, int64_t M, int64_t N, int64_t K,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    if (rowmax_in == nullptr) return W8A8_ERR_INVALID_ARG;
    if (rowmax_out != nullptr && M > 0) {
        // the output maxima are zeroed before the quantizer reads the input maxima: the two must not share memory
        const uintptr_t a = reinterpret_cast<uintptr_t>(rowmax_in), b = reinterpret_cast<uintptr_t>(rowmax_out);
        const uintptr_t bytes = static_cast<uintptr_t>(M) * sizeof(float);
        if (a < b + bytes && b < a + bytes) return W8A8_ERR_INVALID_ARG;
    }
    return fused_impl(A_bf16, W8A8_ACT_BF16, lda, nullptr, nullptr, rowmax_in, qw, s_ch, bias, out_bf16, ldo, rowmax_out, M, N, K,
                      workspace, workspace_bytes, stream);
}

int int8_linear_fused_smooth(const void* A_bf16, int64_t lda, const float* a_mult,
                             const int8_t* qw, const float* s_ch, const float* bias,
                             void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (a_mult == nullptr) return W8A8_ERR_INVALID_ARG;
    return fused_impl(A_bf16, W8A8_ACT_BF16, lda, nullptr, a_mult, nullptr, qw, s_ch, bias, out_bf16, ldo, nullptr, M, N, K,
                      workspace, workspace_bytes, stream);
}

int int8_linear_fused_host(const void* A_host, void* d_A,
                           const int8_t* qw, const float* s_ch, const float* bias,
                           void* d_out, void* out_host, int64_t M, int64_t N, int64_t K,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (A_host == nullptr || d_A == nullptr || d_out == nullptr || out_host == nullptr) return W8A8_ERR_INVALID_ARG;
    if (int e = check_dims(M, N, K)) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(d_A, A_host, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return W8A8_ERR_CUDA;
    int e = int8_linear_fused(d_A, W8A8_ACT_BF16, K, nullptr, qw, s_ch, bias, d_out, N, M, N, K,
                              workspace, workspace_bytes, stream);
    if (e != W8A8_OK) return e;
    if (cudaMemcpyAsync(out_host, d_out, static_cast<size_t>(M) * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return W8A8_ERR_CUDA;
    return W8A8_OK;
}

int int8_gemm_i32_debug(const int8_t* qa, const int8_t* qw, int32_t* acc,
                        int64_t M, int64_t N, int64_t K,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (qa == nullptr || qw == nullptr || acc == nullptr) return W8A8_ERR_INVALID_ARG;
    if (int e = check_dims(M, N, K)) return e;
    if (N % 4 != 0 || !aligned16(qa) || !aligned16(qw) || !aligned16(acc)) return W8A8_ERR_ALIGNMENT;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || workspace_bytes < kStatusBlock)
        return W8A8_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status = static_cast<int*>(workspace);
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return W8A8_ERR_CUDA;
    GemmArgs g{};
    g.qa = qa; g.lda_q = K; g.s_tok = nullptr; g.qw = qw; g.s_ch = nullptr; g.bias = nullptr;
    g.out = acc; g.ldo = N; g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
    g.raw_i32 = true; g.status = status; g.after_quantizer = false; g.split_ws = nullptr;
    const int forced = g_forced_config.load();
    if ((forced < 0 && M <= kSkinnyM) || (forced >= 0 && (forced & 0xff) == tc_num_configs()))
        return launch_gemm_simt(g, st) == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const TcPlan plan = tc_plan(g.M, g.N, g.K, forced, workspace_bytes - kStatusBlock);
    if (plan.split_parts >= 2) {
        if (cudaMemsetAsync(ws + kStatusBlock, 0, plan.scratch_bytes, st) != cudaSuccess) return W8A8_ERR_CUDA;
        g.split_ws = ws + kStatusBlock;
    }
    return launch_gemm_tc(g, plan, st);
}

int int8_check_status(void* workspace, void* stream) {
    if (workspace == nullptr) return W8A8_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return W8A8_ERR_CUDA;
    if (cudaMemsetAsync(workspace, 0, sizeof(int), st) != cudaSuccess) return W8A8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return W8A8_ERR_CUDA;
    return word & 0xff;
}

} // extern "C"
