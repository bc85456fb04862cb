/*
 * w8a8_linear.h -- C ABI of the B200 (sm_100a) fused W8A8 linear layer.
 *
 * The layer follows the paper's Method section: "The quantization recipe
 * (reused)" (per-channel symmetric int8 weights, per-token dynamic int8
 * activations) and "The fused kernel" (int8 x int8 -> int32 accumulation on
 * the tensor cores; per-token scale, per-channel scale and bias applied off the
 * int32 accumulator in the GEMM epilogue; one pass, dequantized output).
 *
 * Arithmetic, fixed for every entry point (IEEE binary32, round to nearest
 * even, no fused multiply-add, no flush to zero):
 *     s      = amax > 0 ? amax / 127 : 1           one division per row
 *     q[k]   = clamp(rne(x[k] / s), -127, 127)     one division per element
 *     acc    = sum_k qa[m,k] * qw[n,k]             exact, int32
 *     out    = bf16(((float(acc) * s_tok[m]) * s_ch[n]) + bias[n])
 * Inputs must be finite; NaN/Inf give unspecified values (never a hang or an
 * out-of-bounds access).
 *
 * Conventions for all calls:
 *   - Matrices are row-major. A is [M,K], W and qw are [N,K], out is [M,N];
 *     ld* are row strides in ELEMENTS.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer that the
 *     caller owns (allocated by the caller, e.g. through PyTorch). The library
 *     allocates no device memory and keeps no reference after the call's work
 *     has run.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work on it and return; they do not synchronize unless
 *     stated.
 *   - Calls are chained on the stream with programmatic dependent launch: a kernel may be set up, and the GEMM may
 *     already request its first WEIGHT tiles, while the kernel ahead of it on the stream is still finishing; it
 *     waits for that kernel before it reads activations, their scales, per-channel scales or bias, and before it
 *     writes anything. Weights (qw) must therefore be complete before the call is enqueued, or be written by
 *     int8_quantize_weight_per_channel (which does not release its dependents early), by a copy, or by a kernel
 *     that does not use cudaTriggerProgrammaticLaunchCompletion / griddepcontrol.launch_dependents.
 *   - The first call of a compute entry point on a device does one-time set-up for that device (function
 *     attributes, the address of the library's sticky status word); make it outside any stream capture. Later
 *     calls only enqueue kernel launches and at most two memsets and can be captured in a CUDA graph.
 *   - The return value is a w8a8_status. Argument errors are detected before
 *     anything is enqueued. There is no CPU fallback and no other backend: on a
 *     device that is not sm_100 (compute capability 10.0) the compute calls return W8A8_ERR_ARCH.
 */
#ifndef W8A8_LINEAR_H_
#define W8A8_LINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum w8a8_status {
    W8A8_OK = 0,
    W8A8_ERR_INVALID_ARG = 1, /* NULL pointer, M/N/K <= 0, ld smaller than the row, unknown dtype */
    W8A8_ERR_ALIGNMENT = 2,   /* pointer not 16-byte aligned, or K/N/ld break the 16-byte rules below */
    W8A8_ERR_K_OVERFLOW = 3,  /* K > 133144: K * 127^2 would not fit in int32 */
    W8A8_ERR_WORKSPACE = 4,   /* workspace NULL, misaligned or smaller than int8_linear_workspace_min_bytes() */
    W8A8_ERR_ARCH = 5,        /* current device is not compute capability 10.0 (sm_100: B200) */
    W8A8_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed (launch, descriptor encode) */
    W8A8_ERR_TIMEOUT = 7      /* a bounded device-side wait expired (reported by int8_check_status) */
} w8a8_status;

/* activation dtype selector of int8_linear_fused */
enum { W8A8_ACT_BF16 = 0, W8A8_ACT_INT8 = 1 };

/* Largest K the integer path accepts (K * 127^2 < 2^31). */
#define W8A8_K_MAX 133144

/*
 * Per-output-channel weight quantization (Method, "The quantization recipe":
 * per-channel int8 weights). Offline set-up step.
 *   W     in   fp32 [N,K], row stride ldw (elements, >= K, multiple of 4), 16-byte aligned
 *   qw    out  int8 [N,K] dense (row stride K), 16-byte aligned
 *   s_ch  out  fp32 [N]
 * Requires K % 16 == 0.
 */
int int8_quantize_weight_per_channel(const float* W, int64_t N, int64_t K, int64_t ldw,
                                     int8_t* qw, float* s_ch, void* stream);

/*
 * Per-token activation quantization (Method, "The fused kernel": per-token
 * scales are dynamic, computed online from the activations).
 *   A_bf16 in   bf16 [M,K], row stride lda (elements, >= K, multiple of 8), 16-byte aligned
 *   qa     out  int8 [M,K] dense, 16-byte aligned
 *   s_tok  out  fp32 [M]
 * Requires K % 16 == 0.
 */
int int8_quantize_act_per_token(const void* A_bf16, int64_t M, int64_t K, int64_t lda,
                                int8_t* qa, float* s_tok, void* stream);

/*
 * Bytes of caller-provided device workspace to give int8_linear_fused for this
 * problem (0 on invalid sizes). Layout, from the workspace base (which must be
 * 256-byte aligned): a 256-byte status block; then, for bf16 activations only,
 * s_tok as fp32 [M] (padded to 256 bytes) and qa as int8 [M,K] dense; then, for
 * shapes whose last wave of output tiles is mostly empty, room for int32 partial
 * accumulators (the tiles of that wave are cut along K over the idle SMs and
 * summed exactly; at most about 10 MB). The workspace needs no initialisation.
 * After a bf16 call the caller may read qa and s_tok back from there
 * (int8_linear_workspace_offsets gives the offsets).
 */
size_t int8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dtype);

/*
 * The smallest workspace int8_linear_fused accepts: the layout above without the
 * partial accumulators. With less than int8_linear_workspace_bytes() the results
 * are the same bit for bit; shapes with a mostly empty last wave run slower.
 */
size_t int8_linear_workspace_min_bytes(int64_t M, int64_t N, int64_t K, int a_dtype);

/* Byte offsets of s_tok and qa inside the workspace for bf16 activations. */
void int8_linear_workspace_offsets(int64_t M, int64_t K, size_t* s_tok_offset, size_t* qa_offset);

/*
 * The fused W8A8 linear (Method, "The fused kernel"):
 *     out[m,n] = bf16(acc[m,n] * s_tok[m] * s_ch[n] + bias[n]),
 *     acc = qa . qw^T in int32 on the tensor cores.
 *   A         in   a_dtype == W8A8_ACT_BF16: bf16 [M,K], quantized per token inside the call;
 *                  a_dtype == W8A8_ACT_INT8: int8 [M,K] codes in [-127,127] (-128 is tolerated
 *                  and exact while K <= 131071). Row stride lda elements; 16-byte aligned;
 *                  lda bytes a multiple of 16.
 *   s_tok_in  in   fp32 [M]; required iff a_dtype == W8A8_ACT_INT8, else must be NULL
 *   qw        in   int8 [N,K] dense, 16-byte aligned
 *   s_ch      in   fp32 [N]
 *   bias      in   fp32 [N] or NULL (no bias term)
 *   out_bf16  out  bf16 [M,N], row stride ldo elements (multiple of 8), 16-byte aligned
 *   workspace      device scratch, int8_linear_workspace_bytes() for full speed and at least
 *                  int8_linear_workspace_min_bytes(); two calls that may overlap on the device
 *                  need distinct workspaces
 * Requires K % 16 == 0, N % 8 == 0, K <= W8A8_K_MAX. The kernel configuration
 * (tile shape, pipeline depth, skinny-M path, one kernel instead of two for
 * bf16 problems of about one tile) is chosen from (M,N,K); the
 * paper's per-shape autotuning ("Why autotuning is load-bearing") is replaced
 * by a static per-shape table. Whatever is chosen, outputs and the codes and
 * scales left in the workspace are the same bit for bit.
 */
int int8_linear_fused(const void* A, int a_dtype, int64_t lda, const float* s_tok_in,
                      const int8_t* qw, const float* s_ch, const float* bias,
                      void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * SmoothQuant hook (Method, "The quantization recipe (reused)": the recipe is W8A8 with SmoothQuant,
 * alpha = 0.5). A per-input-channel factor is multiplied into the operand before it is quantized:
 *     x'[m,k] = float(A[m,k]) * a_mult[k]      W'[n,k] = W[n,k] * w_mult[k]      (one rounded fp32 multiply)
 * and everything else is as in the plain entry points applied to x' / W'. With a_mult = 1/s and w_mult = s the
 * product is unchanged and outlier channels of the activations are tamed; how s is calibrated (the paper uses
 * s_k = max|X_k|^0.5 / max|W_k|^0.5 over a calibration set) is the caller's business: the factors are inputs.
 *   a_mult / w_mult  in  fp32 [K], device, 16-byte aligned, required (use the plain entry points for none)
 * All other arguments, requirements and errors as for the entry point without the suffix.
 */
int int8_quantize_weight_per_channel_smooth(const float* W, int64_t N, int64_t K, int64_t ldw, const float* w_mult,
                                            int8_t* qw, float* s_ch, void* stream);
int int8_quantize_act_per_token_smooth(const void* A_bf16, int64_t M, int64_t K, int64_t lda, const float* a_mult,
                                       int8_t* qa, float* s_tok, void* stream);
int int8_linear_fused_smooth(const void* A_bf16, int64_t lda, const float* a_mult,
                             const int8_t* qw, const float* s_ch, const float* bias,
                             void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * The activation quantizer fused into the producer of the activations, as far as it can be stated exactly
 * (Method, "The fused kernel": the per-token scales are dynamic, computed online from the activations; the paper
 * does not say in how many passes). The quantizer's first pass only finds the largest magnitude of every token.
 * A producer that writes the activations can report that number on the way, and the quantizer then needs one pass:
 *
 * int8_linear_fused_rowmax
 *     int8_linear_fused that additionally writes rowmax_out[m] = max_n |out[m,n]|, the largest magnitude among the
 *     bf16 values it stored for token m (fp32 [M], device; exact: the maximum does not depend on the order).
 *     rowmax_out is zeroed by a memset on `stream` ahead of the kernels and merged with atomic maxima.
 * int8_quantize_act_per_token_given_absmax
 *     int8_quantize_act_per_token with the absmax of every row handed in: s = rowmax[m] > 0 ? rowmax[m] / 127 : 1,
 *     q = rne(x / s). PRECONDITION: rowmax[m] >= max_k |A[m,k]| and finite. Handed the row's own absmax the results
 *     equal int8_quantize_act_per_token's bit for bit; a larger value uses less of the int8 range; with a smaller
 *     one the codes of the elements above it are unspecified (the search pass is what would have caught them).
 * int8_linear_fused_given_absmax
 *     int8_linear_fused on bf16 activations whose quantizer takes rowmax_in [M] as above; rowmax_out may be NULL or,
 *     to chain linears, a buffer that does not overlap rowmax_in (W8A8_ERR_INVALID_ARG otherwise).
 * A chain y = L2(L1(x)) then runs L1 with _rowmax and L2 with _given_absmax on the same vector. An activation
 * function between the two (the MLP's GELU) stays with the caller: the kernel that applies it reports the row
 * maxima of what it writes. All other arguments, requirements and errors as for the plain entry points.
 */
int int8_linear_fused_rowmax(const void* A, int a_dtype, int64_t lda, const float* s_tok_in,
                             const int8_t* qw, const float* s_ch, const float* bias,
                             void* out_bf16, int64_t ldo, float* rowmax_out, int64_t M, int64_t N, int64_t K,
                             void* workspace, size_t workspace_bytes, void* stream);
int int8_quantize_act_per_token_given_absmax(const void* A_bf16, int64_t M, int64_t K, int64_t lda, const float* rowmax,
                                             int8_t* qa, float* s_tok, void* stream);
int int8_linear_fused_given_absmax(const void* A_bf16, int64_t lda, const float* rowmax_in,
                                   const int8_t* qw, const float* s_ch, const float* bias,
                                   void* out_bf16, int64_t ldo, float* rowmax_out, int64_t M, int64_t N, int64_t K,
                                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * Same computation with the activations and the result in HOST memory
 * (pinned memory makes the copies asynchronous): copies A to d_A, runs
 * int8_linear_fused on bf16 activations, copies the result to out_host, all on
 * `stream`, and returns without synchronizing.
 *   A_host   in   host bf16 [M,K] dense        d_A    device bf16 [M,K] staging (caller-owned)
 *   out_host out  host bf16 [M,N] dense        d_out  device bf16 [M,N] staging (caller-owned)
 * Weights, scales, bias and workspace are device pointers as above.
 */
int int8_linear_fused_host(const void* A_host, void* d_A,
                           const int8_t* qw, const float* s_ch, const float* bias,
                           void* d_out, void* out_host, int64_t M, int64_t N, int64_t K,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Allocation-free variant of the fused linear on bf16 activations. (The paper has no counterpart: it is
 * an interface convenience of this library.)
 *
 * For callers that cannot provide a workspace because they cannot allocate one: a server whose own arena
 * already owns all device memory, a latency-critical loop where cudaMalloc's implicit synchronisation is
 * not acceptable, a plug-in that only ever receives its input and output buffers. The scratch that
 * int8_linear_fused takes from the caller (status word, s_tok, qa, and, for shapes whose last wave of tiles is
 * cut along K, the arrival counters and int32 partial sums) is a fixed array of W8A8_STATIC_WORKSPACE_BYTES
 * inside the library's device image; every GPU on which the array's module has been loaded holds that much
 * memory until the process exits. The call itself makes no allocation call (no cudaMalloc, cudaFree or
 * allocating library routine). One caveat on when the memory is taken: with CUDA's default lazy module loading
 * the image that holds the array is loaded, and its 16 MiB reserved, by the first call on a device (the address
 * look-up below), not when the shared library is loaded. A caller whose arena is about to take all of the
 * device's memory makes one call at start-up, before the arena does, or runs with CUDA_MODULE_LOADING=EAGER.
 *
 *   Arguments as for int8_linear_fused with a_dtype == W8A8_ACT_BF16 (device pointers, caller-owned).
 *   sync_and_check  0: enqueue and return. Non-zero: additionally synchronize `stream` and return
 *                   W8A8_ERR_TIMEOUT if a bounded device-side wait gave up (as int8_check_status does).
 *
 * Limits and rules:
 *   - Problems whose scratch, int8_linear_workspace_min_bytes(M, N, K, W8A8_ACT_BF16), exceeds
 *     W8A8_STATIC_WORKSPACE_BYTES are refused with W8A8_ERR_WORKSPACE before anything is enqueued
 *     (roughly M * (K + 4) <= 16 MiB: e.g. M = 4608 tokens at K = 3072, not at K = 12288).
 *   - The first call on each device looks up the array's device address (a one-time set-up step under a
 *     mutex). Make that first call outside any stream capture.
 *   - All calls on a device share the one array. Calls on the same stream run one after the other and are
 *     safe; calls that may overlap on the GPU (different streams, different host threads) race on it and
 *     must be serialized by the caller, or use int8_linear_fused with separate workspaces.
 *   - The array keeps whatever the last call left in it. The caller clears nothing: each call resets the
 *     status word, rewrites the scales and codes it reads, and zeroes the counters and partial sums of a K-split
 *     with a memset on `stream` ahead of its kernels.
 */
#define W8A8_STATIC_WORKSPACE_BYTES (16u * 1024u * 1024u)
int int8_linear_fused_static(const void* A_bf16, int64_t lda,
                             const int8_t* qw, const float* s_ch, const float* bias,
                             void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                             int sync_and_check, void* stream);

/*
 * Test-only export of the raw accumulators of the tensor-core path (the int32
 * values the fused epilogue consumes): acc[m,n] = sum_k qa[m,k] * qw[n,k].
 *   qa in int8 [M,K] dense; qw in int8 [N,K] dense; acc out int32 [M,N] dense (N % 4 == 0);
 *   workspace as for int8_linear_fused with W8A8_ACT_INT8 (256 bytes at least; given
 *   int8_linear_workspace_bytes() it also takes the K-split path of the fused call).
 */
int int8_gemm_i32_debug(const int8_t* qa, const int8_t* qw, int32_t* acc,
                        int64_t M, int64_t N, int64_t K,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronizes `stream` and returns the device-side status word of `workspace`:
 * W8A8_OK, or W8A8_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the
 * kernel then released its resources and returned; outputs are undefined).
 * Clears the word. Returns W8A8_ERR_CUDA if the synchronize failed.
 * The word belongs to the LAST call enqueued on that workspace: every call resets it when it starts (which is
 * why a workspace needs no initialisation), so a time-out of an earlier call on the same workspace is no longer
 * there. Check after each call, or use int8_sticky_status() after many.
 * Diagnostics in the same 256-byte status block: at byte offset 64 the first CTA of the last tensor-core GEMM
 * on this workspace leaves four uint64 stamps: SM cycle counter and nanosecond timer when its work started, and
 * both again when it ended. (cycles_end - cycles_start) / (ns_end - ns_start) is the SM clock in GHz that the
 * launch really ran at, which under a dense tensor load is lower than the clock NVML reports.
 */
int int8_check_status(void* workspace, void* stream);

/*
 * Device-wide sticky status: the first time-out recorded by ANY call of this library on the current device
 * (whatever its workspace; the standalone quantizers, which have none, included) since the word was last
 * cleared. Synchronizes `stream` and returns W8A8_OK or W8A8_ERR_TIMEOUT; clear != 0 also resets the word.
 * Work still running on other streams is not waited for. The word lives in the library's device image and is
 * zero when the library is loaded.
 */
int int8_sticky_status(int clear, void* stream);

/*
 * Test-only controls of the bounded waits (Method, "The fused kernel" has no counterpart; they exist so that the
 * give-up path of the kernels can be executed without faulting or hanging a GPU).
 *   int8_debug_set_wait_limit_ns  bound of every device-side wait for the launches that follow, in nanoseconds
 *                                 (default 2 s; 0 restores the default). Returns the previous value.
 *   int8_debug_set_starve         0: off. 1: the GEMM's producer warp withholds the first pipeline stage of its
 *                                 first tile. 2: the staged activation quantizer's producer withholds its first
 *                                 group of rows. No invalid address is touched and nothing traps: the consumers'
 *                                 waits run out, the kernel frees what it holds and returns, and the status word
 *                                 reports W8A8_ERR_TIMEOUT. Outputs of such a launch are undefined.
 *                                 Returns the previous mode, -1 for an unknown one.
 * Both are process-wide and not meant to be changed while calls are being enqueued from other threads.
 */
uint64_t int8_debug_set_wait_limit_ns(uint64_t limit_ns);
int int8_debug_set_starve(int mode);

/*
 * Test-only choice of the one-kernel path (Method, "The fused kernel": the paper's kernel leaves the per-token
 * quantizer to a launch of its own; for bf16 problems of at most 128 tokens and K <= 1024 this library can run
 * quantizer, GEMM and epilogue in one launch, the CTAs of a cluster sharing the quantizer's work; results, workspace contents
 * and status behaviour are those of the two-kernel path, bit for bit).
 *   -1  chosen from the shape (default: more than 8 and at most 64 tokens, K <= 1024, N <= 1024, at most 8 Ki
 *       elements of A per CTA of a cluster of up to four; never while a configuration is forced or with SmoothQuant
 *       factors)
 *    0  never
 *    1  wherever the kernel can run (1 <= M <= 128, K <= 1024), forced configurations notwithstanding
 * Returns the previous mode, -2 for an unknown one. With mode 1 and int8_debug_set_starve(1) the kernel's only wait
 * (for its MMAs) runs out. Process-wide, like the other test controls.
 */
int int8_debug_set_small_path(int mode);

/*
 * Force a kernel configuration for sweeps and tests. -1 = choose from the shape; -2 = choose from the shape
 * but never cut tiles along K; id = that configuration; id + 0x100 = that configuration, never cut along K.
 * For the configuration whose tiles are two sub-tiles side by side, bits 12-19, if not zero, are 1 + the number of
 * such wide tiles per block of 256 rows (the remaining column blocks run as single sub-tiles); too large a
 * number falls back to the library's choice. For the other tensor-core configurations bits 20-27, if not zero,
 * are the height, in row blocks, of the bands the tiles are walked in (1 = along N first; by default the library
 * bands the order only when the two int8 operands together exceed what stays in L2). Returns the previous value.
 */
int int8_linear_force_config(int config_id);

/*
 * Reports how int8_linear_fused would run this problem on the current device with a workspace of
 * workspace_bytes (under the forced configuration, if one is set): the kernel configuration, the number
 * of CTAs or CTA pairs launched, and the K-split of the last wave (split_tiles tiles cut into split_parts
 * parts each; both 0 when nothing is cut). Any output pointer may be NULL. Launches nothing and needs no
 * device (the SM count of the current device is used, 148 if none can be queried).
 */
int int8_linear_plan(int64_t M, int64_t N, int64_t K, int a_dtype, size_t workspace_bytes,
                     int* config_id, int* cta_groups, int* split_tiles, int* split_parts);

/* Number of kernel configurations that can be forced, and a short description of one (NULL if out of range). The id
 * int8_linear_num_configs() itself names the one-kernel path for small problems, which int8_linear_plan reports where
 * the shape selects it and which cannot be forced through int8_linear_force_config. */
int int8_linear_num_configs(void);
const char* int8_linear_config_name(int config_id);

/* Static string for a status code. */
const char* int8_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* W8A8_LINEAR_H_ */
