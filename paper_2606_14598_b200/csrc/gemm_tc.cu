// Tensor-core W8A8 GEMM with the dequantizing epilogue, for sm_100a.
//
//   acc[m,n] = sum_k qa[m,k] * qw[n,k]        tcgen05.mma.kind::i8, int32 in TMEM
//   out[m,n] = bf16(((float(acc) * s_tok[m]) * s_ch[n]) + bias[n])
//
// One persistent CTA per SM. With CG = 1 every CTA walks output tiles of 128 x BN on its own. With
// CG = 2 the two CTAs of a cluster form a pair (tcgen05 cta_group::2) that walks tiles of 256 x BN:
// each CTA loads its own 128 rows of A and its own half of the W tile, the leader CTA
// issues one MMA for both, and each CTA ends up with its 128 x BN half of the accumulator in its own
// TMEM. A pair moves half as many W bytes per SM through shared memory as two independent CTAs, which
// is what the shared-memory bandwidth needs at the int8 rate. Every load is a plain per-CTA TMA load: the
// leader signals the peer's barriers with a second, plain tcgen05.commit / mbarrier.arrive.
//
// A tile is NSUB sub-tiles of BNS columns side by side (BN = NSUB * BNS). TMEM holds two accumulator slots
// of up to 256 columns, and consecutive sub-tiles alternate between them:
//   NSUB = 1  consecutive tiles alternate slots, so the epilogue of one tile overlaps the k-loop of the next;
//   NSUB = 2  the two sub-tiles of a tile share every A stage (each k-block is multiplied into both slots), which
//             cuts the operand bytes a CTA pulls out of L2 per MMA by a quarter (BNS = 256) or a sixth (BNS = 192):
//             the L2 -> SM feed, not the tensor pipe, is what holds the 256 x 256 tile down. The price is that both
//             slots complete together; the next tile therefore starts staggered: as soon as slot 0 is drained its
//             sub-tile runs ahead over the k-blocks the ring already holds while the epilogue drains slot 1, then
//             sub-tile 1 catches up on the same stages and releases them. To the epilogue a tile simply looks like
//             NSUB consecutive tiles.
// Warp roles:
//   warp 0    TMA producer: loads the 128 x 128-byte A tile and the W tile(s) of each k-block into a ring of
//             shared-memory stages (128-byte swizzle, K-major: both operands are row-major over K)
//   warp 1    allocates TMEM and issues the MMAs (one thread), 4 per k-block and sub-tile
//             (K = 32 each); tcgen05.commit releases the stage / publishes the sub-tile
//   warps 2-5 epilogue: tcgen05.ld the accumulator (lane = row, so s_tok is one
//             scalar per thread; s_ch and bias are per-column broadcasts from
//             shared memory), dequantize, pack to bf16, stage in swizzled shared
//             memory, TMA-store 32 x 64 boxes (TMA clips ragged M and N)
//   warps 6-9 helpers: idle until the CTA's last tile, whose epilogue no k-loop hides;
//             there they take part of the boxes (a warp reads only the TMEM lanes of
//             its index modulo 4, so they pair up with warps 2-5 lane group by lane group)
// (Eight epilogue warps on every tile, two per TMEM lane group, with the per-column scales read straight from
// global memory, were measured slower on the double-buffered 256 x 256 tile: 121.5 against 117.2 us on the MLP
// up-projection.)
//
// K-split of the partial wave (NSUB = 1 only): when the number of tiles is not a multiple of the number of CTA
// groups, the last num_tiles % groups tiles would keep only a few SMs busy for a whole tile time. The host may ask
// for them to be cut along K into split_s parts, one part per group. Every part adds its int32 partial
// accumulator into the tile's slab of the workspace (integer sums: the result does not depend on the
// order); a per-tile counter tells the part that finishes last to read the sums back and run the epilogue.
// No CTA ever waits for another one.
//
// Every mbarrier wait is bounded: on expiry the CTA records W8A8_ERR_TIMEOUT in
// the workspace status word, all roles unwind, TMEM is freed and the kernel
// returns.
#include "../../include/w8a8_linear.h"
#include "internal.h"
#include "ptx.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

namespace w8a8 {
namespace {

constexpr int BM = 128;            // rows of A per tile (= TMEM lanes)
constexpr int BK = 128;            // int8 elements (= bytes) of K per k-block: one 128-byte swizzle row
constexpr int MMA_K = 32;          // K of one tcgen05.mma.kind::i8
constexpr int EPI_THREADS = 128;    // warps 2..5: the epilogue of every tile
constexpr int HELPER_WARP0 = 6;     // warps 6..9: take part of the columns of a CTA's last tile, whose epilogue nothing hides
constexpr int NUM_THREADS = 64 + 2 * EPI_THREADS;
constexpr int SMEM_MAX = 232448;   // dynamic shared memory a CTA can opt in to

enum Where { W_PRODUCER_EMPTY = 1, W_MMA_FULL = 2, W_MMA_TMEM_EMPTY = 3, W_EPI_TMEM_FULL = 4 };

template <int CG, int BNS, int NSUB, int STAGES, int KBS>
struct SmemLayout {
    static constexpr int BN = BNS * NSUB;                           // columns of a tile
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_ROWS = BNS / CG;                         // W rows of one sub-tile this CTA loads
    static constexpr int B_BYTES = B_ROWS * BK;
    static constexpr int KB_BYTES = A_BYTES + NSUB * B_BYTES;       // one k-block: A tile + W tile(s) of 128 bytes of K
    static constexpr int STAGE_BYTES = KBS * KB_BYTES;              // a pipeline stage holds KBS k-blocks
    static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
    static constexpr int STAGING_BOX_BYTES = 32 * 128;             // one 32-row x 64-column bf16 box
    // two boxes alternate per epilogue warp where shared memory allows, else one
    static constexpr int STAGING_BUFS = (RING_BYTES + 8 * STAGING_BOX_BYTES + 16 * BNS + 1280 <= SMEM_MAX) ? 2 : 1;
    static constexpr int STAGING_BYTES_PER_WARP = STAGING_BUFS * STAGING_BOX_BYTES;
    static constexpr int OFF_STAGING = RING_BYTES;
    // per-column scales and bias of a sub-tile, double-buffered by accumulator slot
    static constexpr int OFF_SCH = OFF_STAGING + 4 * STAGING_BYTES_PER_WARP;
    static constexpr int OFF_BIAS = OFF_SCH + 2 * BNS * 4;
    // full[STAGES * KBS] (one per k-block), empty[STAGES] (one per stage), tfull[2], tempty[2]
    static constexpr int OFF_BARS = OFF_BIAS + 2 * BNS * 4;
    static constexpr int NUM_FULL = STAGES * KBS;
    static constexpr int NUM_BARS = NUM_FULL + STAGES + 4;
    static constexpr int OFF_TMEM = OFF_BARS + NUM_BARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 4;
    static constexpr int OFF_LAST = OFF_ABORT + 4;                 // "this CTA finishes the split tile" (epilogue warps)
    static constexpr int TOTAL = OFF_LAST + 4;
    static constexpr int DYN_BYTES = TOTAL + 1024;                 // slack to align the base to 1024
    static_assert(B_BYTES % 1024 == 0, "operand tiles start on a swizzle-atom boundary");
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// What a kernel needs beyond its operands: the bound of its waits, where time-outs are recorded, test hooks.
struct RunCtl {
    int* status;            // workspace status word
    int* sticky;            // device-wide sticky status word (or nullptr)
    uint64_t wait_limit_ns;
    int after_quantizer;    // the quantizer ahead of this kernel has reset the status word
    int starve;             // test hook: the producer withholds the first k-stage of its first tile
};

template <int CG, int BNS, int NSUB, int STAGES, int KBS, bool RAW_I32>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_out,
               const float* s_tok, const float* __restrict__ s_ch, const float* __restrict__ bias,
               int32_t* __restrict__ raw_out, int M, int N, int K, const RunCtl rc,
               int split_tiles, int split_s, int32_t* split_slabs, int* split_counters, int wide_per_row, int band,
               float* rowmax) {
    using L = SmemLayout<CG, BNS, NSUB, STAGES, KBS>;
    constexpr int BN = L::BN;
    // the next kernel in the stream, if it was launched to allow it (the next call's quantizer is), may be scheduled
    // as this grid's CTAs retire and set itself up; it waits for this whole grid before it touches global memory
    grid_dep_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;     // position in the CTA pair; 0 leads
    const bool leader = rank == 0;
    const uint32_t bars = base + L::OFF_BARS;
    // Operands arrive per k-block (the MMAs of a k-block start as soon as its 128 bytes of K have landed);
    // shared memory is handed back per stage of KBS k-blocks (one tcgen05.commit per stage).
    auto full_bar = [&](int s, int sub) { return bars + 8u * (s * KBS + sub); };          // used in the leader
    auto empty_bar = [&](int s) { return bars + 8u * (L::NUM_FULL + s); };                // one per CTA
    auto tfull_bar = [&](int b) { return bars + 8u * (L::NUM_FULL + STAGES + b); };       // one per CTA
    auto tempty_bar = [&](int b) { return bars + 8u * (L::NUM_FULL + STAGES + 2 + b); };  // used in the leader
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(base_ptr + L::OFF_TMEM);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::OFF_ABORT);
    const WaitCtl ctl{abort_flag, rc.status, rc.sticky, rc.wait_limit_ns};

    // two accumulator slots, each at a power-of-two column offset (the allocation must be a power of two >= 32)
    constexpr uint32_t TMEM_BUF = BNS <= 128 ? 128u : 256u;
    constexpr uint32_t TMEM_COLS = 2 * TMEM_BUF;
    static_assert(BNS % 64 == 0 && BNS <= 256, "BNS: whole 64-column output boxes, at most 256 TMEM columns per slot");
    static_assert(NSUB == 1 || NSUB == 2, "a tile is one or two sub-tiles");

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            for (int sub = 0; sub < KBS; ++sub) mbar_init(full_bar(s, sub), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4 * CG); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_a);
        prefetch_tensormap(&tm_b);
        if (!RAW_I32) prefetch_tensormap(&tm_out);
    }
    if (warp == 1) {
        if (CG == 2) { tmem_alloc_pair(base + L::OFF_TMEM, TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(base + L::OFF_TMEM, TMEM_COLS); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();            // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    constexpr int TILE_M = BM * CG;
    const int num_m = (M + TILE_M - 1) / TILE_M;
    const int num_nb = (N + BNS - 1) / BNS;                     // column blocks of one sub-tile's width
    // Work items. NSUB = 1: one item per tile. With band = 1 they run along N first, then the next block of rows: a
    // wave of concurrent tiles then shares a few row blocks of A and all of W, which is fine while both operands stay
    // in L2. When they do not (the host decides), bands of `band` row blocks are walked column by column, so that a
    // wave covers about as many row blocks as column blocks and fetches the fewest operand bytes from DRAM (its CTAs
    // move along K in step, so within a wave every operand byte is fetched once). NSUB = 2: every block of rows is covered by
    // wide_per_row wide items (two column blocks side by side, sharing A) followed by narrow items (one column
    // block) for the rest; all wide items come first in the list, then all narrow ones, and item i belongs to CTA
    // group i mod groups. The host picks wide_per_row so that the groups end up with equal work (e.g. 18 x 12 column
    // blocks on 74 pairs: 4 wide + 4 narrow per row block give 72 pairs one wide and one narrow item each).
    const int wide = NSUB == 2 ? wide_per_row : 0;
    const int narrow = NSUB == 2 ? num_nb - 2 * wide : num_nb;
    const int num_wide = num_m * wide;
    const int num_tiles = num_wide + num_m * narrow;
    const int wide_div = wide > 0 ? wide : 1, narrow_div = narrow > 0 ? narrow : 1;   // (a kind that is absent is never decoded)
    const int num_kb = (K + BK - 1) / BK;
    const int first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;
    // Work list of this CTA group: whole items first_tile, first_tile + tile_step, ... below tiles_whole, then
    // (K-split) part unit_part of tile unit_tile: stages [unit_sb, unit_se) of its k-loop.
    const int num_kstages = (num_kb + KBS - 1) / KBS;
    const int tiles_whole = num_tiles - split_tiles;
    const bool has_unit = NSUB == 1 && split_s >= 2 && first_tile < split_tiles * split_s;
    const int unit_slot = has_unit ? first_tile / split_s : 0, unit_part = has_unit ? first_tile % split_s : 0;
    const int unit_tile = tiles_whole + unit_slot;
    const int unit_sb = has_unit ? num_kstages * unit_part / split_s : 0;
    const int unit_se = has_unit ? num_kstages * (unit_part + 1) / split_s : 0;
    struct Item { int m0, n0, nsub; };                          // first row (of the pair), first column, sub-tiles
    const int band_tiles = band * num_nb;                       // tiles of a full band (NSUB = 1)
    auto item = [&](int t) -> Item {
        if (NSUB == 1) {
            const int b = t / band_tiles, r = t - b * band_tiles;
            const int rows_here = min(band, num_m - b * band);  // the last band may be lower
            return Item{(b * band + r % rows_here) * TILE_M, (r / rows_here) * BNS, 1};
        }
        if (t < num_wide) return Item{(t / wide_div) * TILE_M, (t % wide_div) * 2 * BNS, 2};
        const int u = t - num_wide;
        return Item{(u / narrow_div) * TILE_M, (2 * wide + u % narrow_div) * BNS, 1};
    };
    // items of this group below L
    auto count_below = [&](int L) { return L > first_tile ? (L - first_tile + tile_step - 1) / tile_step : 0; };
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs of a pair)
        // The kernel is always launched so that it may start while the kernel ahead of it in the stream is finishing
        // (the quantizer, or whatever the caller ran): everything up to here touched no global memory.
        int stage = 0;
        uint32_t phase = 0;
        int issued = 0;
        bool ok = true;
        bool withhold = rc.starve != 0;                     // test hook: this CTA's very first stage never arrives
        const uint64_t keep = l2_policy_evict_last();       // operands are re-read by other tiles: keep them in L2
        // the loads of pipeline stage `ks` of item `it` into ring slot `st`: the barrier's byte count (armed once per
        // k-block), the A tile and / or the W tile(s). A stage always receives all its k-blocks: those past the end of
        // K are zero-filled by TMA (and skipped by the MMA thread), which keeps the byte count of the barrier constant.
        auto load_stage = [&](const Item& it, int ks, int st, bool arm, bool load_a, bool load_b) {
            const int m0 = it.m0 + rank * BM;
            const int n0 = it.n0 + rank * L::B_ROWS;
            const uint32_t kb_bytes = L::A_BYTES + it.nsub * L::B_BYTES;
#pragma unroll
            for (int sub = 0; sub < KBS; ++sub) {
                const uint32_t sa = base + st * L::STAGE_BYTES + sub * L::KB_BYTES;
                const int kx = (ks * KBS + sub) * BK;
                if (CG == 2) {
                    // the leader's barrier counts the bytes of both CTAs
                    if (arm && leader) mbar_arrive_expect_tx(full_bar(st, sub), 2 * kb_bytes);
                    const uint32_t fb = mapa_shared(full_bar(st, sub), 0);
                    if (load_a) tma_load_2d_pair_hint(sa, &tm_a, fb, kx, m0, keep);
#pragma unroll
                    for (int h = 0; h < NSUB; ++h)
                        if (load_b && h < it.nsub) tma_load_2d_pair_hint(sa + L::A_BYTES + h * L::B_BYTES, &tm_b, fb, kx, n0 + h * BNS, keep);
                } else {
                    if (arm) mbar_arrive_expect_tx(full_bar(st, sub), kb_bytes);
                    if (load_a) tma_load_2d_hint(sa, &tm_a, full_bar(st, sub), kx, m0, keep);
#pragma unroll
                    for (int h = 0; h < NSUB; ++h)
                        if (load_b && h < it.nsub) tma_load_2d_hint(sa + L::A_BYTES + h * L::B_BYTES, &tm_b, full_bar(st, sub), kx, n0 + h * BNS, keep);
                }
            }
        };
        // The first piece of work of this CTA group (a whole item, or its part of a tile cut along K).
        const bool first_is_unit = !(first_tile < tiles_whole);
        const int first_t = first_is_unit ? unit_tile : first_tile;
        const int first_sb = first_is_unit ? unit_sb : 0, first_se = first_is_unit ? unit_se : num_kstages;
        const bool any_work = first_tile < tiles_whole || has_unit;
        int pre = 0;                                        // stages of that piece whose W tiles were requested early
        if (lane == 0) {
            // The weights do not depend on the kernel ahead of this one (the quantizer writes activations): the W tiles
            // of the first ring of stages are requested before the wait, the A tiles after it, so that the first MMA
            // waits for the short trip of the freshly written activations out of L2 rather than for cold weights out
            // of DRAM. (Weights, like every operand but the activations and their scales, must therefore be complete
            // before the call is enqueued, or be written by a kernel that does not release its dependents early.)
            if (any_work && !withhold) {
                const Item it = item(first_t);
                pre = min(STAGES, first_se - first_sb);
                for (int i = 0; i < pre; ++i) load_stage(it, first_sb + i, i, true, false, true);   // the ring starts empty
            }
            grid_dep_wait();
            // without a quantizer ahead of it (which clears the status word) the kernel clears it itself; a time-out
            // can only be recorded a whole wait limit later
            if (!rc.after_quantizer && blockIdx.x == 0) *rc.status = 0;
            // diagnostics: CTA 0 stamps the SM cycle counter and the nanosecond timer when its work starts and when it
            // ends (status block, byte 64): their ratio is the SM clock this launch really ran at
            if (blockIdx.x == 0) {
                unsigned long long* stamps = reinterpret_cast<unsigned long long*>(rc.status + 16);
                stamps[0] = static_cast<unsigned long long>(clock64());
                stamps[1] = globaltimer_ns();
            }
            if (pre > 0) {
                const Item it = item(first_t);
                for (int i = 0; i < pre; ++i) load_stage(it, first_sb + i, i, false, true, false);
                issued = pre;
                stage = pre == STAGES ? 0 : pre;
                phase = pre == STAGES ? 1u : 0u;
            }
        }
        __syncwarp();
        // stages [sb, se) of item t; the first `skip` of them have been issued already
        auto produce = [&](int t, int sb, int se, int skip) {
            const Item it = item(t);
            if (lane == 0) {
                for (int ks = sb + skip; ks < se; ++ks) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctl, W_PRODUCER_EMPTY, kStatusTimeout)) { ok = false; break; }
                    if (withhold) {
                        // neither the byte count nor a copy is posted for this stage: its barriers never complete, the
                        // MMA thread's bounded wait runs out, and every role unwinds
                        withhold = false;
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    load_stage(it, ks, stage, true, true, true);
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            ok = __all_sync(0xffffffffu, ok) != 0;
        };
        for (int t = first_tile; t < tiles_whole && ok; t += tile_step) produce(t, 0, num_kstages, t == first_t ? pre : 0);
        if (has_unit && ok) produce(unit_tile, unit_sb, unit_se, first_is_unit ? pre : 0);
        if (!ok && lane == 0 && (CG == 1 || leader)) {
            // let copies that are still in flight land before the CTA goes away
            int s = stage;
            uint32_t ph = phase;
            for (int i = 0; i < STAGES && i < issued; ++i) {
                if (s == 0) { s = STAGES; ph ^= 1u; }
                --s;
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(full_bar(s, KBS - 1), ph) && globaltimer_ns() - t0 < 10000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = make_i8_idesc(TILE_M, BNS);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int c = 0;                                     // sub-tiles begun so far: slot = c & 1, use of that slot = c >> 1
            auto slot_tmem = [&](int cc) { return tmem_base + static_cast<uint32_t>(cc & 1) * TMEM_BUF; };
            auto wait_slot = [&](int cc) {                 // the epilogue has drained the slot's previous sub-tile
                if (!mbar_wait(tempty_bar(cc & 1), ((cc >> 1) & 1) ^ 1u, ctl, W_MMA_TMEM_EMPTY, kStatusTimeout)) return false;
                tc_fence_after();
                return true;
            };
            // the MMAs of k-block (st, sub) into sub-tile h; `fresh`: this k-block is the first of the sub-tile
            auto issue = [&](int st, int sub, int kbi, int h, uint32_t d_tmem, bool fresh) {
                const uint32_t sa = base + st * L::STAGE_BYTES + sub * L::KB_BYTES;
                const uint64_t da = make_kmajor_sw128_desc(sa);
                const uint64_t db = make_kmajor_sw128_desc(sa + L::A_BYTES + h * L::B_BYTES);
                // K steps of this k-block that hold data (0 for a k-block past the end of K)
                const int left = K - kbi * BK;
                const int ksteps = left <= 0 ? 0 : min(BK, left + MMA_K - 1) / MMA_K;
#pragma unroll
                for (int k = 0; k < BK / MMA_K; ++k) {
                    if (k < ksteps) {   // advancing K by 32 bytes inside the swizzled row: +2 in 16-byte units
                        const uint32_t acc = (fresh && k == 0) ? 0u : 1u;   // the first MMA overwrites
                        if (CG == 2) mma_i8_ss_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, acc);
                        else mma_i8_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, acc);
                    }
                }
            };
            auto wait_full = [&](int st, int sub, uint32_t ph) {
                if (!mbar_wait(full_bar(st, sub), ph, ctl, W_MMA_FULL, kStatusTimeout)) return false;
                tc_fence_after();
                return true;
            };
            // the stage is free (in both CTAs) once the MMAs issued so far have read it. One commit per stage, not per
            // k-block: with 128-byte stages the commits and barrier round trips cost ~8% of the run time
            auto release_stage = [&](int st) {
                // (signalling only the leader and letting its producer pass the release on to the peer with a remote
                // arrive was measured: 147 against 110 us on the MLP down-projection. The release -> refill latency
                // is what this pipeline lives on. One commit with a CTA mask that arrives on both barriers at once
                // measured the same as these two: 111.0 / 115.0 us.)
                if (CG == 2) { tc_commit_pair(empty_bar(st)); tc_commit_pair(mapa_shared(empty_bar(st), 1)); }
                else tc_commit(empty_bar(st));
            };
            auto publish = [&](int cc) {                   // the sub-tile's accumulator is complete (in both CTAs)
                if (CG == 2) { tc_commit_pair(tfull_bar(cc & 1)); tc_commit_pair(mapa_shared(tfull_bar(cc & 1), 1)); }
                else tc_commit(tfull_bar(cc & 1));
            };
            auto mma_tile = [&](int nsub, int sb, int se) {
                int ks = sb;
                if (NSUB == 2 && nsub == 2) {
                    // Staggered start. Both slots were published together, but the epilogue drains slot 0 first:
                    // sub-tile 0 runs ahead over the stages the ring can hold while slot 1 is still being drained,
                    // then sub-tile 1 catches up on the same stages and hands them back.
                    const int lead = min(STAGES, se - sb);
                    if (!wait_slot(c)) { ok = false; return; }
                    int st = stage;
                    uint32_t ph = phase;
                    for (int i = 0; i < lead && ok; ++i) {
#pragma unroll
                        for (int sub = 0; sub < KBS; ++sub) {
                            if (!wait_full(st, sub, ph)) { ok = false; break; }
                            issue(st, sub, (sb + i) * KBS + sub, 0, slot_tmem(c), i == 0 && sub == 0);
                        }
                        if (++st == STAGES) { st = 0; ph ^= 1u; }
                    }
                    if (!ok) return;
                    if (!wait_slot(c + 1)) { ok = false; return; }
                    for (int i = 0; i < lead; ++i) {
#pragma unroll
                        for (int sub = 0; sub < KBS; ++sub)
                            issue(stage, sub, (sb + i) * KBS + sub, 1, slot_tmem(c + 1), i == 0 && sub == 0);
                        release_stage(stage);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                    ks = sb + lead;
                } else {
                    if (!wait_slot(c)) { ok = false; return; }
                }
                for (; ks < se; ++ks) {
#pragma unroll
                    for (int sub = 0; sub < KBS; ++sub) {
                        if (!wait_full(stage, sub, phase)) { ok = false; break; }
#pragma unroll
                        for (int h = 0; h < NSUB; ++h)
                            if (h < nsub) issue(stage, sub, ks * KBS + sub, h, slot_tmem(c + h), ks == sb && sub == 0);
                    }
                    if (!ok) return;
                    release_stage(stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
#pragma unroll
                for (int h = 0; h < NSUB; ++h)
                    if (h < nsub) publish(c + h);
                c += nsub;
            };
            for (int t = first_tile; t < tiles_whole && ok; t += tile_step) mma_tile((NSUB == 2 && t < num_wide) ? 2 : 1, 0, num_kstages);
            if (has_unit && ok) mma_tile(1, unit_sb, unit_se);
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5, helpers 6..9)
        const int lg = warp & 3;                       // TMEM lane group this warp may read: 32*lg .. 32*lg+31
        const int ep_tid = threadIdx.x - 64;
        const bool helper = warp >= HELPER_WARP0;
        float* sm_sch = reinterpret_cast<float*>(base_ptr + L::OFF_SCH);
        float* sm_bias = reinterpret_cast<float*>(base_ptr + L::OFF_BIAS);
        // staging boxes: the epilogue warps have their own; the helpers borrow the operand ring, which is idle by
        // the time the last tile's accumulators are complete
        const int stg_off = helper ? (warp - HELPER_WARP0) * L::STAGING_BYTES_PER_WARP
                                   : L::OFF_STAGING + (warp - 2) * L::STAGING_BYTES_PER_WARP;
        const uint32_t staging = base + stg_off;
        uint8_t* staging_ptr = base_ptr + stg_off;
        // The epilogue of a CTA's last tile overlaps with nothing: there the helpers take the upper part of the boxes.
        const int n_regular = count_below(tiles_whole);                              // whole items of this CTA group
        const int n_sub = n_regular + count_below(min(num_wide, tiles_whole));      // their sub-tiles (a wide item has two)
        const int t_last = first_tile + (n_regular - 1) * tile_step;                // the group's last whole item
        const int last_nsub = (NSUB == 2 && n_regular > 0 && t_last < num_wide) ? 2 : 1;
        constexpr int ALL_CHUNKS = BNS / 32;
        constexpr int C_SPLIT = 2 * (BNS / 64 - BNS / 128);          // 32-column chunks the epilogue warps keep on that tile
        const bool helpers_on = !RAW_I32 && n_regular > 0 && !has_unit && C_SPLIT < ALL_CHUNKS;
        const bool has_bias = bias != nullptr;
        const uint64_t stream_out = l2_policy_evict_first();        // the output is written once and not read here
        grid_dep_wait();                               // s_tok may come from the kernel before this one
        bool ok = true;
        int c = 0;                                     // sub-tile counter: slot = c & 1, use of the slot = c >> 1
        volatile int* last_flag = reinterpret_cast<volatile int*>(base_ptr + L::OFF_LAST);
        // chunks [c_lo, c_hi) of sub-tile h of tile t; `shared_tile`: the helpers work on this sub-tile too
        auto epi_tile = [&](int t, int h, bool unit, int c_lo, int c_hi, bool shared_tile) {
            const int buf = c & 1;
            const Item it = item(t);
            const int m0 = it.m0 + rank * BM, n0 = it.n0 + h * BNS;
            const float* sch_buf = sm_sch + buf * BNS;
            const float* bias_buf = sm_bias + buf * BNS;
            if (!RAW_I32 && !helper) {
                // the slot's buffer was last read two sub-tiles ago, which every warp has left behind
                for (int j = ep_tid; j < BNS; j += EPI_THREADS) {
                    const int n = n0 + j;
                    sm_sch[buf * BNS + j] = n < N ? __ldg(s_ch + n) : 0.f;
                    sm_bias[buf * BNS + j] = (has_bias && n < N) ? __ldg(bias + n) : 0.f;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            // the helpers have been parked here since the start of the kernel: the scales of this sub-tile are in place
            if (shared_tile) asm volatile("bar.sync 2, 256;" ::: "memory");
            const int row = m0 + lg * 32 + lane;
            // plain (coherent) load: the quantizer ahead of this kernel wrote s_tok while this kernel was already resident
            const float st = (!RAW_I32 && row < M) ? __ldcg(s_tok + row) : 0.f;
            if (ok && !mbar_wait(tfull_bar(buf), (c >> 1) & 1, ctl, W_EPI_TMEM_FULL, kStatusTimeout)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && !unit) return;                  // later tiles still take their named barriers, but skip the work
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + buf * TMEM_BUF;
            // One chunk = 32 accumulator columns of this thread's row. Two chunks make a 32 x 64 output box.
            // The TMEM load of the next chunk is in flight while the current one is converted.
            const uint64_t st2 = pack2(st, st);
            // optional side output: the largest magnitude this thread's row receives from this sub-tile (bf16 values as
            // stored; columns outside N come out as +0 and do not count), merged into rowmax[row] at the end
            __nv_bfloat162 rmax2 = __float2bfloat162_rn(0.f);
            auto flush_rowmax = [&]() {
                if (RAW_I32 || rowmax == nullptr || row >= M) return;
                const uint32_t mb = *reinterpret_cast<const uint32_t*>(&rmax2);
                const uint32_t bits = max(mb << 16, mb & 0xffff0000u);      // non-negative floats order like their bit patterns
                if (bits != 0u) atomicMax(reinterpret_cast<unsigned int*>(rowmax) + row, bits);
            };
            auto process = [&](int cc, const uint32_t (&v)[32]) {
                const int col = cc * 32, hh = cc & 1, cb = cc >> 1;
                const int sbuf = cb & (L::STAGING_BUFS - 1);  // staging boxes alternate: the store of one overlaps the next
                if (RAW_I32) {
                    if (row < M) {
                        int32_t* dst = raw_out + static_cast<int64_t>(row) * N + n0 + col;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + col + j < N) dst[j] = static_cast<int32_t>(v[j]);
                    }
                } else {
                uint32_t packed[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    // (float(acc) * s_tok) * s_ch + bias on two columns at a time; each half rounds like the scalar op
                    uint64_t tt = pack2(__int2float_rn(static_cast<int>(v[2 * j])), __int2float_rn(static_cast<int>(v[2 * j + 1])));
                    tt = mul2(tt, st2);
                    tt = mul2(tt, *reinterpret_cast<const uint64_t*>(sch_buf + col + 2 * j));
                    float a0, a1;
                    unpack2(tt, a0, a1);
                    if (has_bias) {
                        // scalar adds: a packed add right behind the packed multiply was seen to be contracted
                        // into a fused multiply-add by the assembler, which changes the rounding
                        const float2 bi = *reinterpret_cast<const float2*>(bias_buf + col + 2 * j);
                        a0 = __fadd_rn(a0, bi.x);
                        a1 = __fadd_rn(a1, bi.y);
                    }
                    packed[j] = pack_bf16x2(a0, a1);
                }
                if (rowmax != nullptr) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) rmax2 = __hmax2(rmax2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&packed[j])));
                }
                if (hh == 0) {
                    // the store issued STAGING_BUFS boxes ago (same staging box) must have finished reading it
                    if (lane == 0) bulk_wait_group_read<L::STAGING_BUFS - 1>();
                    __syncwarp();
                }
                // row `lane` of the 32 x 128-byte box; 16-byte chunk i lives at chunk (i ^ (row & 7))
                uint8_t* srow = staging_ptr + sbuf * L::STAGING_BOX_BYTES + lane * 128;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 q = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
                    *reinterpret_cast<uint4*>(srow + (((hh * 4 + i) ^ (lane & 7)) << 4)) = q;
                }
                if (hh == 1) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d_hint(&tm_out, staging + sbuf * L::STAGING_BOX_BYTES, n0 + cb * 64, m0 + lg * 32, stream_out);
                        bulk_commit_group();
                    }
                }
                }
            };
            auto release_accumulator = [&]() {         // every TMEM load of this sub-tile has completed
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && !helper) {            // (nothing follows a tile the helpers work on)
                    if (CG == 2) mbar_arrive_cluster(mapa_shared(tempty_bar(buf), 0));
                    else mbar_arrive(tempty_bar(buf));
                }
            };
            constexpr int CHUNKS = ALL_CHUNKS;
            uint32_t va[32], vb[32];
            if (!unit) {
                tmem_ld_32x32b_x32(t_row + c_lo * 32, va);
#pragma unroll 1
                for (int cc = c_lo; cc < c_hi; cc += 2) {
                    tmem_wait_ld();
                    tmem_ld_32x32b_x32(t_row + (cc + 1) * 32, vb);
                    process(cc, va);
                    tmem_wait_ld();
                    if (cc + 2 < c_hi) tmem_ld_32x32b_x32(t_row + (cc + 2) * 32, va);
                    else release_accumulator();
                    process(cc + 1, vb);
                }
                flush_rowmax();
                return;
            }
            // ---- one K part of a split tile. Every part adds its int32 accumulators into the tile's slab in
            // global memory (zeroed by the host before the launch) with reductions, which need no reply. Slab
            // layout: [CTA of the pair][column][128 rows], so that the 32 rows of a warp are 128 contiguous bytes.
            constexpr int SLAB = BN * BM;
            int32_t* slab = split_slabs + static_cast<size_t>(unit_slot * CG + rank) * SLAB;
            if (ok) {
                int32_t* mine = slab + lg * 32 + lane;
                auto put = [&](int cc, const uint32_t (&v)[32]) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) red_add_s32(mine + (cc * 32 + j) * BM, static_cast<int32_t>(v[j]));
                };
                tmem_ld_32x32b_x32(t_row, va);
#pragma unroll 1
                for (int cc = 0; cc < CHUNKS; cc += 2) {
                    tmem_wait_ld();
                    tmem_ld_32x32b_x32(t_row + (cc + 1) * 32, vb);
                    put(cc, va);
                    tmem_wait_ld();
                    if (cc + 2 < CHUNKS) tmem_ld_32x32b_x32(t_row + (cc + 2) * 32, va);
                    else release_accumulator();
                    put(cc + 1, vb);
                }
            }
            // The part that arrives last at the tile's counter finishes the tile (fence, then count: every
            // reduction counted before ours has been applied before we read the slab).
            __threadfence();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ep_tid == 0) *last_flag = atomicAdd(split_counters + unit_slot * CG + rank, 1) == split_s - 1 ? 1 : 0;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*last_flag == 0) return;               // uniform over the epilogue warps: the barriers below stay matched
            __threadfence();
            // This is the CTA's last piece of work and its MMAs have completed: the operand ring is free. Pull the
            // whole slab into it with asynchronous copies (all in flight at once), then run the usual epilogue.
            static_assert(NSUB == 2 || SLAB * 4 <= L::RING_BYTES, "the slab fits in the operand ring");
            for (int i = ep_tid; i < SLAB / 4; i += EPI_THREADS) cp_async_16(base + i * 16, slab + i * 4);
            cp_async_wait_all();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (!ok) return;                           // a wait of this warp gave up: no output from it
            const int32_t* sm_slab = reinterpret_cast<const int32_t*>(base_ptr) + lg * 32 + lane;
#pragma unroll 1
            for (int cc = 0; cc < CHUNKS; ++cc) {
#pragma unroll
                for (int j = 0; j < 32; ++j) va[j] = static_cast<uint32_t>(sm_slab[(cc * 32 + j) * BM]);
                process(cc, va);
            }
            flush_rowmax();
        };
        if (!helper) {
            for (int t = first_tile; t < tiles_whole; t += tile_step) {
                const int nsub = (NSUB == 2 && t < num_wide) ? 2 : 1;
                for (int h = 0; h < nsub; ++h, ++c) {
                    const bool shared_tile = helpers_on && c >= n_sub - last_nsub;
                    epi_tile(t, h, false, 0, shared_tile ? C_SPLIT : ALL_CHUNKS, shared_tile);
                }
            }
            if (has_unit) epi_tile(unit_tile, 0, true, 0, ALL_CHUNKS, false);
        } else if (helpers_on) {
            c = n_sub - last_nsub;
            for (int h = 0; h < last_nsub; ++h, ++c) epi_tile(t_last, h, false, C_SPLIT, ALL_CHUNKS, true);
        }
        if (!RAW_I32 && lane == 0) bulk_wait_group<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long* stamps = reinterpret_cast<unsigned long long*>(rc.status + 16);
        stamps[2] = static_cast<unsigned long long>(clock64());
        stamps[3] = globaltimer_ns();
    }
    if (CG == 2) cluster_sync_all();            // nobody leaves while the peer may still signal its barriers
    tc_fence_after();
    if (warp == 1) {
        if (CG == 2) tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else tmem_dealloc(tmem_base, TMEM_COLS);
    }
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
    int cg, bns, nsub, stages, kbs;
    float eff;      // measured throughput per SM relative to configuration 2 (large shapes, whole waves)
};
constexpr TcConfig kConfigs[] = {
    // measured on the c4 shapes (hot L2): pair 256x256 3 x 256 B: 115 / 111 us; one CTA 128x256 4 x 128 B: 129 / 121 us;
    // pair 256x192: 130 / 123 us; one CTA 128x128: 164 / 154 us; pair 256x128: 168 / 162 us. Stage shapes of the
    // 256x256 pair at the same 192 KB: 6 x 128 B of K 126 / 118 us (120 / 114 us with a single commit per stage),
    // 2 x 384 B 123 / 117 us (both directions lose).
    // Pair tiles of two sub-tiles: 2 x 256 wins cold bursts where K is deep and the wide items fill whole waves
    // (M = 9472, K = 12288 -> N = 3072: 208-225 against 216-237 us) and loses once the power cap bites (see tc_plan);
    // 2 x 192 lost everywhere (N = 192 MMAs) and is not built.
    {"tc 128x256 per CTA, 4 stages x 128 B of K", 1, 256, 1, 4, 1, 0.89f},
    {"tc 128x128 per CTA, 3 stages x 256 B of K", 1, 128, 1, 3, 2, 0.72f},
    {"tc 256x256 per CTA pair, 3 stages x 256 B of K", 2, 256, 1, 3, 2, 1.00f},
    {"tc 256x128 per CTA pair, 4 stages x 256 B of K", 2, 128, 1, 4, 2, 0.70f},
    {"tc 256x192 per CTA pair, 3 stages x 256 B of K", 2, 192, 1, 3, 2, 0.88f},
    {"tc 256x512 (2 x 256) per CTA pair, 4 stages x 128 B of K", 2, 256, 2, 4, 1, 1.08f},
};
constexpr int kNumConfigs = sizeof(kConfigs) / sizeof(kConfigs[0]);
constexpr int kNoSplitBit = 0x100;        // added to a forced configuration id: no K-split of the partial wave
constexpr size_t kCounterBytes = 1024;    // per-tile arrival counters at the head of the split scratch (<= 148 ints)
constexpr int kMaxSplit = 8;              // parts per tile
constexpr int kMinStagesPerPart = 4;

template <int CG, int BNS, int NSUB, int STAGES, int KBS, bool RAW>
int launch_cfg(const GemmArgs& a, const TcPlan& plan, cudaStream_t st) {
    using L = SmemLayout<CG, BNS, NSUB, STAGES, KBS>;
    static_assert(L::DYN_BYTES <= SMEM_MAX, "shared memory budget");
    auto kern = gemm_tc_kernel<CG, BNS, NSUB, STAGES, KBS, RAW>;
    static PerDeviceOnce smem_opt_in;
    if (smem_opt_in.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES); }) != cudaSuccess)
        return W8A8_ERR_CUDA;

    CUtensorMap tm_a, tm_b, tm_out;
    if (!encode_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.qa, a.M, a.K, a.lda_q, BM, BK)) return W8A8_ERR_CUDA;
    if (!encode_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.qw, a.N, a.K, a.K, L::B_ROWS, BK)) return W8A8_ERR_CUDA;
    if (RAW) {
        tm_out = tm_a;   // unused
    } else {
        if (!encode_2d(&tm_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.out, a.M, a.N, a.ldo * 2, 32, 64)) return W8A8_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CG * plan.groups);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = L::DYN_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (CG == 2) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    cfg.attrs = attr;
    cfg.numAttrs = na;
    RunCtl rc{};
    rc.status = a.status;
    rc.sticky = sticky_status_word();
    rc.wait_limit_ns = wait_limit_ns();
    rc.after_quantizer = a.after_quantizer ? 1 : 0;
    rc.starve = starve_mode() == kStarveGemm ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_out, a.s_tok, a.s_ch, a.bias,
                                       RAW ? static_cast<int32_t*>(a.out) : nullptr, a.M, a.N, a.K, rc,
                                       plan.split_tiles, plan.split_parts,
                                       reinterpret_cast<int32_t*>(static_cast<uint8_t*>(a.split_ws) + kCounterBytes),
                                       static_cast<int*>(a.split_ws), plan.wide_per_row, plan.band > 0 ? plan.band : 1,
                                       a.raw_i32 ? nullptr : a.rowmax);
    return e == cudaSuccess ? W8A8_OK : W8A8_ERR_CUDA;
}

template <bool RAW>
int launch_by_id(const GemmArgs& a, const TcPlan& plan, cudaStream_t st) {
    switch (plan.config) {
        case 0: return launch_cfg<1, 256, 1, 4, 1, RAW>(a, plan, st);
        case 1: return launch_cfg<1, 128, 1, 3, 2, RAW>(a, plan, st);
        case 2: return launch_cfg<2, 256, 1, 3, 2, RAW>(a, plan, st);
        case 3: return launch_cfg<2, 128, 1, 4, 2, RAW>(a, plan, st);
        case 4: return launch_cfg<2, 192, 1, 3, 2, RAW>(a, plan, st);
        case 5: return launch_cfg<2, 256, 2, 4, 1, RAW>(a, plan, st);
        default: return W8A8_ERR_INVALID_ARG;
    }
}

// Grid and K-split of one configuration on one shape, with its estimated run time in microseconds.
// Whole waves of tiles cost a tile time each; the partial wave (tiles % groups, or all tiles when there are
// fewer tiles than groups) is cut along K into as many parts as there are idle groups (at least
// kMinStagesPerPart pipeline stages per part, at most kMaxSplit parts, and only if the scratch has room),
// which shortens it to 1/parts of a tile time plus the cost of adding the partial sums up. With only_if_faster
// the cut is dropped when the estimate says it does not pay (it pays for deep K: K >= ~8192).
// Configurations of two sub-tiles are never cut; their degree of freedom is how many of a row block's column
// blocks are paired into wide items (see the kernel): the count that gives the busiest group the least work wins.
TcPlan plan_config(int id, int M, int N, int K, bool allow_split, bool only_if_faster, size_t scratch_bytes, int wide_forced,
                   int band_forced, double* est_us) {
    const TcConfig& c = kConfigs[id];
    TcPlan p{};
    p.config = id;
    p.band = 1;
    if (c.nsub == 1) {
        // Tile order: while both int8 operands stay in L2 (126 MB; 96 MB leaves room for the output on its way out)
        // the tiles run along N first. Beyond that a wave of G concurrent tiles should span as many row blocks as
        // column blocks: bands of about sqrt(G * BN / TILE_M) row blocks, walked column by column.
        const int groups_all = sm_count() / c.cg;
        const int rows_all = (M + BM * c.cg - 1) / (BM * c.cg);
        if (band_forced > 0) {
            p.band = band_forced;
        } else if ((static_cast<double>(M) + N) * K > 96e6) {
            int b = 1;
            while ((b + 1) * (b + 1) * BM * c.cg <= groups_all * c.bns) ++b;
            p.band = b;
        }
        if (p.band > rows_all) p.band = rows_all;
    }
    const int max_groups = sm_count() / c.cg;
    const int num_m = (M + BM * c.cg - 1) / (BM * c.cg);
    // launch, pipeline fill, last epilogue; a pair pays for its cluster launch and for filling stages of twice the
    // bytes (fitted on shapes of about one wave at K = 1536-3072: 3072 x 1536 x 1536 runs 8.9 us on single CTAs,
    // 10.7 us on pairs with the same per-CTA tile)
    const double fixed_us = c.cg == 1 ? 4.0 : 5.5;
    if (c.nsub == 2) {
        // ~20.3 int8 TOPS per SM for the 256 x 256 pair tile in whole waves; a unit = one column block of a row block
        const int num_nb = (N + c.bns - 1) / c.bns;
        const double unit_us = 2.0 * BM * c.bns * static_cast<double>(K) / 20.3e6;
        const double wide_unit_us = unit_us / c.eff, narrow_unit_us = unit_us / 0.88;   // narrow items run on four 128-byte stages
        const double wide_exposed_us = 2.5;            // the drain of a wide item's first accumulator overlaps nothing
        int best_w = 0;
        double best = 0.0;
        for (int w = (wide_forced >= 0 ? wide_forced : 0); w <= (wide_forced >= 0 ? wide_forced : num_nb / 2); ++w) {
            const long wide_items = static_cast<long>(num_m) * w, all_items = wide_items + static_cast<long>(num_m) * (num_nb - 2 * w);
            const long groups = all_items < max_groups ? all_items : max_groups;
            double worst = 0.0;
            for (long g = 0; g < groups; ++g) {
                const long nw = wide_items > g ? (wide_items - g + groups - 1) / groups : 0;
                const long na = all_items > g ? (all_items - g + groups - 1) / groups : 0;
                const double t = nw * (2.0 * wide_unit_us + wide_exposed_us) + (na - nw) * narrow_unit_us;
                if (t > worst) worst = t;
            }
            if (w == (wide_forced >= 0 ? wide_forced : 0) || worst < best) { best = worst; best_w = w; }
        }
        const long items = static_cast<long>(num_m) * (num_nb - best_w);
        p.wide_per_row = best_w;
        p.groups = static_cast<int>(items < max_groups ? items : max_groups);
        if (est_us) *est_us = fixed_us + best;
        return p;
    }
    const long tiles = static_cast<long>(num_m) * ((N + c.bns - 1) / c.bns);
    const int bn = c.bns;
    const int whole_waves = static_cast<int>(tiles / max_groups);
    const int rest = static_cast<int>(tiles % max_groups);
    const int kstages = ((K + BK - 1) / BK + c.kbs - 1) / c.kbs;
    int parts = 1;
    if (allow_split && rest > 0) {
        parts = max_groups / rest;
        if (parts > kstages / kMinStagesPerPart) parts = kstages / kMinStagesPerPart;
        if (parts > kMaxSplit) parts = kMaxSplit;
        const size_t need = kCounterBytes + static_cast<size_t>(rest) * c.cg * bn * BM * sizeof(int32_t);
        if (parts < 2 || need > scratch_bytes) parts = 1;
    }
    // A partial wave that is left whole runs its tiles faster than the full-wave rate, since the operand traffic of a
    // full wave is what holds the rate down: measured 0.68-0.80 of the tile time with a tenth to a third of the SMs
    // active for single CTAs, whose full-wave rate suffers most from that traffic, and 0.86-0.97 for CTA pairs. A wave
    // cut along K keeps every SM busy and pays for zeroing the slabs, the reductions, the pipeline refill and the
    // read-back: 7-9 us measured on single CTAs with 128-column slabs, 11-12 us with 256-column ones and on pairs
    // (M = 192-512, K = 8192, N = 264-2048).
    const double tile_us = 2.0 * BM * bn * static_cast<double>(K) / 20.3e6 / c.eff;
    const double few = c.cg == 1 ? 0.72 : 0.85;
    const double whole_rest_us = tile_us * (few + (1.0 - few) * rest / max_groups);
    const double split_rest_us = tile_us / parts + (c.cg == 1 ? 5.5 + 6.0 * bn / 256 : 12.0);
    if (parts > 1 && only_if_faster && split_rest_us >= whole_rest_us) parts = 1;
    double est = fixed_us + whole_waves * tile_us;
    if (rest > 0) est += parts > 1 ? split_rest_us : whole_rest_us;
    if (parts > 1) {
        p.split_tiles = rest;
        p.split_parts = parts;
        p.groups = whole_waves > 0 ? max_groups : rest * parts;
        p.scratch_bytes = kCounterBytes + static_cast<size_t>(rest) * c.cg * bn * BM * sizeof(int32_t);
    } else {
        p.split_tiles = 0;
        p.split_parts = 0;
        // From three waves on: the fewest groups that need no more waves than all of them would. Every group then gets
        // the same number of tiles (216 tiles are three waves on 74 pairs and exactly three tiles each on 72), and the
        // SMs left out leave their share of the power budget to the others (measured: 0.3-0.7% faster on the c3 / c4
        // shapes; with two waves, 132 tiles on 66 instead of 74 pairs, 1% slower, so short grids keep every group).
        const long waves = (tiles + max_groups - 1) / max_groups;
        p.groups = static_cast<int>(waves >= 3 ? (tiles + waves - 1) / waves : (tiles < max_groups ? tiles : max_groups));
        p.scratch_bytes = 0;
    }
    if (est_us) *est_us = est;
    return p;
}

} // namespace

int tc_num_configs() { return kNumConfigs; }
const char* tc_config_name(int id) { return (id >= 0 && id < kNumConfigs) ? kConfigs[id].name : nullptr; }

TcPlan tc_plan(int M, int N, int K, int forced, size_t scratch_bytes) {
    // forced: -1 automatic, -2 automatic without K-split, id, or id + 0x100 for that configuration without K-split;
    // bits 12-19, if not zero, are 1 + the number of wide items per row block (two-sub-tile configurations);
    // bits 20-27, if not zero, are the band height in row blocks of the tile order (single-sub-tile configurations)
    const bool allow_split = forced == -1 || (forced >= 0 && (forced & kNoSplitBit) == 0);
    const int id = forced < 0 ? -1 : (forced & (kNoSplitBit - 1));
    const int wide_forced = forced < 0 ? -1 : ((forced >> 12) & 0xff) - 1;
    const int band_forced = forced < 0 ? 0 : ((forced >> 20) & 0xff);          // 0 = from the sizes
    if (id >= 0 && id < kNumConfigs) {
        int wf = wide_forced;
        if (kConfigs[id].nsub == 2 && wf > ((N + kConfigs[id].bns - 1) / kConfigs[id].bns) / 2) wf = -1;   // not possible: choose
        return plan_config(id, M, N, K, allow_split, false, scratch_bytes, wf, band_forced, nullptr);   // forced: cut whenever possible
    }
    // lowest estimated time; on (near) ties the earlier entry of this preference order wins
    // The configuration of two sub-tiles per tile is not among the candidates: alternating with the 256 x 256 pair in
    // one process (M = 9216, K = 12288 -> N = 3072, 60 launches each) it won the first, cold round (208 against
    // 216 us) and lost every later one (235-260 against 223-237 us): it keeps the tensor pipe busier, draws more
    // power and is clocked down further (1.23-1.38 against 1.33-1.42 GHz measured inside the kernels). It stays
    // available as a forced configuration.
    constexpr int order[] = {2, 0, 4, 3, 1};
    TcPlan best{};
    double best_us = 0.0;
    for (int i = 0; i < static_cast<int>(sizeof(order) / sizeof(order[0])); ++i) {
        double us = 0.0;
        const TcPlan p = plan_config(order[i], M, N, K, allow_split, true, scratch_bytes, -1, 0, &us);
        if (i == 0 || us < best_us * 0.97) { best = p; best_us = us; }
    }
    return best;
}

size_t tc_max_scratch_bytes(int M, int N, int K) {
    // what the automatic choice would use with unlimited scratch
    return tc_plan(M, N, K, -1, static_cast<size_t>(-1)).scratch_bytes;
}

int launch_gemm_tc(const GemmArgs& a, const TcPlan& plan, cudaStream_t st) {
    if (plan.split_parts >= 2 && a.split_ws == nullptr) return W8A8_ERR_INVALID_ARG;
    return a.raw_i32 ? launch_by_id<true>(a, plan, st) : launch_by_id<false>(a, plan, st);
}

} // namespace w8a8
