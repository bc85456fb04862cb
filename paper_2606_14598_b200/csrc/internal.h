// Host-side launch functions shared by the translation units of the library.
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include <mutex>

namespace w8a8 {

// Function attributes (the opt-in to large dynamic shared memory) belong to a device: `set` runs once for every
// device a launch is made on, under a lock, and its result is remembered.
class PerDeviceOnce {
public:
    template <typename F>
    cudaError_t run(F&& set) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mutex_);
        if (!done_[dev]) {
            err_[dev] = set();
            done_[dev] = true;
        }
        return err_[dev];
    }

private:
    static constexpr int kMaxDevices = 64;
    std::mutex mutex_;
    bool done_[kMaxDevices] = {};
    cudaError_t err_[kMaxDevices] = {};
};

// SM count of the current device (148 if no device can be queried, so that host-only planning still works).
inline int sm_count() {
    static std::mutex mutex;
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mutex);
    if (cached[dev] == 0) {
        int v = 0;
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        cached[dev] = v > 0 ? v : 148;
    }
    return cached[dev];
}

// Device-side status codes written into the workspace status word (low byte
// is a w8a8_status value, the next byte says which wait gave up).
constexpr int kStatusTimeout = 7;

// ---- api.cu : controls shared by the launchers
// Bound of every device-side wait in nanoseconds (2 s unless a test lowered it).
uint64_t wait_limit_ns();
// Test-only starvation hook: 0 = none; kStarveGemm = the GEMM's producer withholds the first k-stage of its first
// tile; kStarveQuant = the staged quantizer's producer withholds its first row group. Nothing invalid is touched:
// the consumers' bounded waits run out, the kernel unwinds and returns, and the status word says which wait gave up.
constexpr int kStarveGemm = 1, kStarveQuant = 2;
int starve_mode();
// Device address, on the current device, of the word that keeps the first time-out of any call until the host
// reads and clears it (int8_sticky_status); nullptr if it cannot be resolved.
int* sticky_status_word();

// ---- quantize.cu
// status_to_clear: workspace status word the kernel resets (or nullptr).
// mult: per-input-channel factors fp32 [K] multiplied into the operand first (SmoothQuant hook), or nullptr.
// amax: the absmax of every row fp32 [M] handed in by the producer of A (one-pass quantizer), or nullptr; not with mult.
cudaError_t launch_quantize_bf16(const void* A, int64_t lda, int M, int K, const float* mult, const float* amax, int8_t* qa,
                                 float* s_tok, int* status_to_clear, cudaStream_t st);
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
    void* split_ws;        // scratch of the K-split (counters, then partial accumulators), or nullptr
    float* rowmax;         // fp32 [M], zero at launch: receives max_n |out[m,n]| of the bf16 values written; or nullptr
};
cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t st);

// ---- small_fused.cu : quantizer, GEMM and epilogue in one kernel, for problems of at most 128 tokens and K <= 1024
constexpr int kSkinnyM = 8;           // at or below this many tokens the weight-streaming path runs
constexpr int64_t kSmallFusedMaxCtas = 32;                 // 32-channel CTAs the one-kernel path is chosen for (N <= 1024)
constexpr int64_t kSmallFusedMaxTokens = 64;               // tokens up to which it is chosen
constexpr int64_t kSmallFusedMaxElemsPerCta = 8 << 10;     // elements of A one of its CTAs may have to quantize
bool small_fused_eligible(int64_t M, int64_t N, int64_t K);     // what the kernel can run
bool small_fused_preferred(int64_t M, int64_t N, int64_t K);    // where it is chosen when nothing is forced
// Writes the codes and scales to qa_out / s_tok_out as the two-kernel path does, the output to g.out.
cudaError_t launch_small_fused(const void* A_bf16, int64_t lda, const float* amax_in, const GemmArgs& g, int8_t* qa_out,
                               float* s_tok_out, cudaStream_t st);
// Test-only: -1 = chosen by small_fused_preferred (default), 0 = never, 1 = wherever small_fused_eligible.
int small_path_mode();

// ---- gemm_tc.cu : tcgen05 path
int tc_num_configs();
const char* tc_config_name(int id);
// How a shape is run: configuration, grid, and the K-split of the partial wave of tiles (0 parts = none).
struct TcPlan {
    int config;
    int groups;            // CTAs (or CTA pairs) launched
    int split_tiles;       // tiles of the partial wave that are cut along K
    int split_parts;       // parts per such tile
    size_t scratch_bytes;  // scratch the split needs (counters, then one int32 slab per tile); all zero at launch
    int wide_per_row;      // configurations of two sub-tiles: wide items (two column blocks) per block of rows
    int band;              // other configurations: row blocks per band of the tile order (1 = along N first)
};
// Picks a configuration for the shape (or `forced` if >= 0; forced + 0x100 = that configuration without K-split;
// bits 12-19 of `forced`, if not zero, are 1 + the number of wide items per block of rows; bits 20-27, if not zero,
// the band height of the tile order).
// A split is planned only if its scratch fits in scratch_bytes.
TcPlan tc_plan(int M, int N, int K, int forced, size_t scratch_bytes);
// Scratch the automatic choice uses when it is given enough.
size_t tc_max_scratch_bytes(int M, int N, int K);
// Launches the plan. Returns a w8a8_status.
int launch_gemm_tc(const GemmArgs& a, const TcPlan& plan, cudaStream_t st);

} // namespace w8a8
