// Fused sm_100a kernel for bf16 heads: Eq. 1 masks (Philox), Eq. 2 masking, Eq. 3 on tcgen05
// tensor cores with fp32 accumulators in TMEM, and the argmax of Sec. 3.2 in the epilogue.  W is
// streamed from HBM once per launch and no logit is written (except on request: the debug call
// the JS criterion and nucleus sampling ask for them).  On heads whose vocabulary slices are a
// single tile the masked hidden rows exist in shared memory only; on larger heads they are staged
// once per call through global memory.  W tiles are loaded with an L2 evict-first policy.
//
// Work split.  The vocabulary is cut into one contiguous slice per CTA (one CTA per SM) and
// each slice into equal tiles of `tile_rows` <= 128 vocabulary rows.  The MMA is "swapped": a
// W tile is the M = 128 operand, the masked hidden rows are the N operand (N = rows padded to
// a multiple of 16, at most 256), so accumulator lane m is vocabulary row m of the tile and
// column n is path n.  TMEM (512 columns) is a ring of 512/N accumulator slots, one per tile.
//
// Loop order.  Tiles are taken in groups of `group_tiles`; inside a group the hidden-size
// blocks (64 elements = one 128-byte swizzled row) are the outer loop and the tiles the inner
// one, all accumulators of the group being live at once, while W streams through a ring of
// TMA stages exactly once.  The masked operand of a block is needed once per group:
//   - one group (single-tile slices): builder warps generate the masks with Philox in
//     registers and write the masked rows of each block into a shared-memory ring, once per call;
//   - several groups ("staged"): the mask pass ahead in the stream has written the masked rows to a staging
//     buffer in global memory once per call.  W tiles and operand blocks share one ring of
//     "steps": a step is the group's W tiles of one hidden-size block with the operand block
//     behind them, one barrier for "all of it has landed" and one for "the MMAs are done with
//     it", so that the issuing warp waits once and commits once per step.  A group takes at most
//     half of the accumulator slots: the epilogue of one group overlaps the MMAs of the next.
//     Staged launches run as CTA pairs (see kPair below).
//
// Warp roles (14 warps):
//   warp 0      TMA producer: one thread issues cp.async.bulk.tensor loads of W
//   warp 1      MMA issuer: the whole warp runs the loop converged, one elected lane issues
//               tcgen05.mma and the commits (their operands then live in uniform registers)
//   warps 2-5   epilogue: tcgen05.ld the finished accumulators of a group, scale by 1/(1-p),
//               reduce each column over tiles and lanes to (max, first index), keep the best
//               per path; warp 2 also allocates and frees TMEM; the last CTA of a one-launch
//               call then runs the histogram and the acceptance
//   warps 6-13  one group: operand builders.  Staged: warps 6-9 are a second set of epilogue
//               warps, one thread of warp 10 streams the staged operand, the rest retire
// Rings are guarded by mbarriers; every wait has a time limit after which the CTA sets the
// error word, drains and frees TMEM instead of hanging.
#include <new>

#include "dm_finalize.cuh"
#include "dm_internal.h"
#include "dm_ptx.cuh"

namespace dm {

namespace {

constexpr int kThreads = 14 * 32;
constexpr int kExpWarps = 8;
constexpr int kFirstEpiWarp = 2, kFirstExpWarp = 6;
constexpr int kBlockK = 64;                 // hidden-size elements per stage (128 bytes of bf16)
constexpr int kTileM = 128;                 // UMMA M
constexpr int kMaxNPad = 256;               // UMMA N limit
constexpr int kWStageBytes = kTileM * kBlockK * 2;
constexpr int kTmemCols = 512;
constexpr int kMaxWStages = 12;
constexpr long long kWaitLimitCycles = 2000000000ll;   // default limit of every wait: about one second
constexpr int kPollNs = 32;                 // pause between polls of a barrier on the critical path
constexpr int kIdlePollNs = 500;            // ... and of one that completes once per tile group
constexpr int kSmemLimit = 227 * 1024;
constexpr int kBarBytes = 1024;             // mbarriers + TMEM address + abort flag
// Launch-shape thresholds, in operand rows after padding to 16 (measured on the Llama-3-8B and
// Qwen3-8B heads; see plan_smem).
#ifndef DM_PAIR_MIN_NPAD
#define DM_PAIR_MIN_NPAD 16     // staged launches at least this wide run as CTA pairs
#endif
#ifndef DM_STAGED_MIN_NPAD
#define DM_STAGED_MIN_NPAD 16   // slices of several tiles at least this wide are staged even if they would fit TMEM as one group
#endif
#ifndef DM_W_EVICT_FIRST_MIN_BYTES
#define DM_W_EVICT_FIRST_MIN_BYTES 0   // heads larger than this many bytes stream W with the L2 evict-first policy
#endif
#ifndef DM_PAIR_GRAN
#define DM_PAIR_GRAN 32        // operand rows of a pair launch are padded to a multiple of this (16 or 32)
#endif
#ifndef DM_PAIR_PAD_MIN
#define DM_PAIR_PAD_MIN 64      // narrower pair launches are padded to this many accumulator columns
#endif
constexpr int kPairMinNPad = DM_PAIR_MIN_NPAD;   // staged launches at least this wide run as CTA pairs

struct FusedParams {
    const __nv_bfloat16* H;
    int d, V;
    int v_offset;     // added to every token id (vocabulary-sharded heads)
    int rows;         // paths per row block of this launch (<= 256; the last block may hold fewer)
    int row0;         // first path of this launch within the call
    int rows_total;   // paths of the whole call (stride of the partials array)
    int n_pad;        // rows rounded up to a multiple of 16
    int kb_count;     // d / 64
    int tiles_per_cta, tile_rows, slice_rows;
    int group_tiles;  // tiles whose accumulators are live together
    int n_slots;      // accumulator slots in TMEM (512 / n_pad)
    int nsw, nsb;     // stages of the W ring and of the operand ring
    // staged: one ring of `nsw` steps.  A step holds the group's W tiles of one hidden-size block and,
    // behind them, the operand block; one barrier says that all of it has landed, one that the MMAs
    // are done with it, so that the issuing thread waits and commits once per step.
    uint32_t step_bytes;
    int staged;       // masked operand comes from the staging buffer through TMA (tmap_b)
    int pdl;          // launched with programmatic stream serialization: see the griddep_wait() calls
    int w_evict_first;   // W tiles are loaded with the L2 evict-first policy (heads larger than L2)
    long long wait_limit;   // clock cycles after which a wait on an mbarrier gives up (see dm_debug_set_wait_limit)
    int row_blocks;   // 1, or 2: two blocks of 256 paths share one pass over W (see fused_launch)
    RowMap map;
    uint32_t key0, key1, thr;
    float scale;
    int sample;       // the epilogue adds Gumbel noise to logit * inv_temp before the maximum (sampling decode)
    float inv_temp;
    unsigned long long* partials;   // [vocabulary slice][rows_total]
    float* dbg_logits;              // [rows_total][V] or null
    uint32_t* err;
    // fold != 0 (a call of one launch): the CTAs reduce their per-path best into `best` with atomic
    // maxima instead of writing per-slice partials.  fold == 1: the last CTA to finish also runs the
    // histogram and the acceptance and zeroes `best` again; `ticket` counts finished CTAs and is
    // left at 0.  fold == 2: `best` is the caller's array (zero before the launch), nothing more.
    int fold;
    unsigned int* ticket;
    unsigned long long* best;       // [rows_total], all zero between calls: CTAs reduce into it when folding
    FinalizeArgs fin;
    // byte offsets into the 1024-aligned dynamic shared memory
    uint32_t off_w, off_b, off_rowinfo, off_best, off_bar;
};

struct RowInfo { int q; uint32_t s, t, i; };

__device__ __forceinline__ uint32_t mask_pair(uint32_t bits2) {
    // bit 0 -> low bf16 kept, bit 1 -> high bf16 kept
    return ((bits2 & 1u) ? 0x0000FFFFu : 0u) | ((bits2 & 2u) ? 0xFFFF0000u : 0u);
}

// kPair: the kernel runs as clusters of two CTAs (staged mode only).  Each CTA keeps its own
// vocabulary slice, W ring, TMEM and epilogue, but loads only half of the operand rows; the
// leader (cluster rank 0) issues cta_group::2 MMAs that multiply both CTAs' W tiles by the
// operand rows of both, which halves the operand's shared-memory and L2 traffic per CTA.
// Barriers that the MMA issuer waits on live in the leader; those that it signals exist in both
// CTAs and are reached by multicast commits.
template <bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
fused_head_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_b,
                  const FusedParams P) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = ptx::smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    RowInfo* s_row = reinterpret_cast<RowInfo*>(smem + P.off_rowinfo);
    unsigned long long* s_best = reinterpret_cast<unsigned long long*>(smem + P.off_best);  // [4][n_pad]
    uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + P.off_bar);
    // barrier layout: w_full[nsw] w_empty[nsw] b_ready[nsb] b_empty[nsb] slot_full[S] slot_empty[S]
    const uint32_t bar0 = smem_base + P.off_bar;
    const uint32_t w_full = bar0, w_empty = w_full + 8 * P.nsw;
    const uint32_t b_ready = w_empty + 8 * P.nsw, b_empty = b_ready + 8 * P.nsb;
    const uint32_t slot_full = b_empty + 8 * P.nsb, slot_empty = slot_full + 8 * P.n_slots;
    const int n_bars = 2 * P.nsw + 2 * P.nsb + 2 * P.n_slots + 1;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + n_bars);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
    volatile unsigned int* s_ticket = reinterpret_cast<volatile unsigned int*>(s_tmem + 2);
    volatile int* s_never = reinterpret_cast<volatile int*>(s_tmem + 3);   // stays 0: for the one wait that an abort must not cut short

    const int wps = kExpWarps / P.nsb;   // operand-builder warps per ring stage
    const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;   // 0 = leader of the pair
    const uint32_t dealloc_bar = slot_empty + 8 * P.n_slots;      // pair only: the other CTA is done with TMEM
    // CTA -> (vocabulary slice, row block).  With two row blocks per launch the CTAs (or CTA pairs)
    // alternate between the blocks: the two that share a slice run side by side and the second
    // one's W loads hit L2, so that W crosses the HBM interface once for 512 paths.
    const int unit = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // CTA, or CTA pair
    const int rb = unit % P.row_blocks;
    const int slice = kPair ? (unit / P.row_blocks) * 2 + (int)(blockIdx.x & 1) : unit / P.row_blocks;
    const int row0 = P.row0 + rb * P.rows;       // first path of this CTA's row block within the call
    const int my_rows = min(P.rows, P.rows_total - row0);   // the second block of a launch may be shorter

    if (threadIdx.x == 0) {
        ptx::prefetch_tensormap(&tmap_w);
        if (P.staged) ptx::prefetch_tensormap(&tmap_b);
        for (int s = 0; s < P.nsw; ++s) { ptx::mbar_init(w_full + 8 * s, P.staged ? 2 : 1); ptx::mbar_init(w_empty + 8 * s, 1); }
        for (int s = 0; s < P.nsb; ++s) {
            ptx::mbar_init(b_ready + 8 * s, P.staged ? 1 : wps);
            ptx::mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < P.n_slots; ++s) { ptx::mbar_init(slot_full + 8 * s, 1); ptx::mbar_init(slot_empty + 8 * s, kPair ? 16 : P.staged ? 8 : 12); }
        ptx::mbar_init(dealloc_bar, 1);
        *s_abort = 0;
        *s_never = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == kFirstEpiWarp) {   // an epilogue warp owns TMEM: it is still whole at the end
        if (kPair) {
            ptx::tmem_alloc_pair(ptx::smem_u32(s_tmem), kTmemCols);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(ptx::smem_u32(s_tmem), kTmemCols);
            ptx::tmem_relinquish();
        }
    }
    for (int r = threadIdx.x; r < my_rows; r += kThreads) {
        RowKey k;
        bool ok = row_key(P.map, row0 + r, k);
        if (!ok) atomicExch(P.err, (uint32_t)ERR_BAD_ROW);
        s_row[r] = RowInfo{ok ? k.q : -1, k.s, k.t, k.i};
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (kPair) ptx::cluster_sync_all();   // the other CTA's barriers are initialised before anyone signals them
    ptx::tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    // The next call's kernel may be scheduled as soon as SMs free up: its prologue and its first W
    // loads then overlap this kernel's tail.  W is never written while calls are in flight, so the
    // W producer and the MMA issuer need not wait for the kernel ahead; whoever reads H or the
    // staged operand, or writes global memory, does (griddep_wait below).
    if (P.pdl) ptx::griddep_launch_dependents();

    const int v_cta0 = slice * P.slice_rows;
    int my_tiles = 0;
    if (v_cta0 < P.V) {
        my_tiles = (P.V - v_cta0 + P.tile_rows - 1) / P.tile_rows;
        if (my_tiles > P.tiles_per_cta) my_tiles = P.tiles_per_cta;
    }
    // A pair steps through the same number of tiles: rows past the end of W load as zeros and
    // are never taken by the epilogue.
    if (kPair) my_tiles = P.tiles_per_cta;
    const int G = P.group_tiles;
    const int n_groups = (my_tiles + G - 1) / G;

    // Polling an mbarrier is not free for the TMA unit that updates it, so each wait is made by
    // one lane only.  The producer and the MMA issuer are single threads; the other lanes of
    // their warps retire at once instead of idling at a barrier.
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane != 0) return;
        // Ring positions, phases and coordinates advance by increments: this lone thread must
        // issue one load every few hundred cycles, and an integer division costs about that.
        const uint32_t tx_bytes = (uint32_t)P.tile_rows * (kBlockK * 2);
        uint32_t bar_full = w_full, bar_empty = w_empty, dst = smem_base + P.off_w, empty_parity = 1;
        int stage = 0;
        // W is read once per launch: its lines go first when L2 needs room, so that the staged
        // operand, and the logits a call may write, stay there.  Not when two row blocks share the
        // stream: the second reader of a tile is meant to find it in L2.
        const uint64_t w_policy = (P.row_blocks == 1 && P.w_evict_first) ? ptx::l2_policy_evict_first() : ptx::l2_policy_evict_normal();
        if (P.staged) {
            // one step per (group, hidden-size block): the group's W tiles side by side
            for (int g = 0; g < n_groups; ++g) {
                const int t0 = g * G, t1 = min(my_tiles, t0 + G);
                const int v_first = v_cta0 + t0 * P.tile_rows;
                const uint32_t step_tx = (uint32_t)(t1 - t0) * tx_bytes;
                for (int kb = 0, x = 0; kb < P.kb_count; ++kb, x += kBlockK) {
                    if (!ptx::mbar_wait<kPollNs>(bar_empty, empty_parity, s_abort, P.wait_limit)) {
                        atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_EMPTY);
                        return;
                    }
                    if (!kPair) ptx::mbar_arrive_expect_tx(bar_full, step_tx);
                    else if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full, 2 * step_tx);   // both CTAs' tiles count here
                    int v_tile = v_first;
                    uint32_t d = dst;
                    for (int tile = t0; tile < t1; ++tile, v_tile += P.tile_rows, d += kWStageBytes) {
                        if (kPair) ptx::tma_load_2d_pair_hint(d, &tmap_w, x, v_tile, ptx::map_to_cta(bar_full, 0), w_policy);
                        else ptx::tma_load_2d_hint(d, &tmap_w, x, v_tile, bar_full, w_policy);
                    }
                    bar_full += 8; bar_empty += 8; dst += P.step_bytes;
                    if (++stage == P.nsw) {
                        stage = 0; empty_parity ^= 1;
                        bar_full = w_full; bar_empty = w_empty; dst = smem_base + P.off_w;
                    }
                }
            }
            return;
        }
        for (int g = 0; g < n_groups; ++g) {
            const int t0 = g * G, t1 = min(my_tiles, t0 + G);
            const int v_first = v_cta0 + t0 * P.tile_rows;
            for (int kb = 0, x = 0; kb < P.kb_count; ++kb, x += kBlockK) {
                int v_tile = v_first;
                for (int tile = t0; tile < t1; ++tile, v_tile += P.tile_rows) {
                    if (!ptx::mbar_wait<kPollNs>(bar_empty, empty_parity, s_abort, P.wait_limit)) {
                        atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_EMPTY);
                        return;
                    }
                    if (kPair) {   // both tiles of the pair are counted on the leader's barrier
                        if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full, 2 * tx_bytes);
                        ptx::tma_load_2d_pair_hint(dst, &tmap_w, x, v_tile, ptx::map_to_cta(bar_full, 0), w_policy);
                    } else {
                        ptx::mbar_arrive_expect_tx(bar_full, tx_bytes);
                        ptx::tma_load_2d_hint(dst, &tmap_w, x, v_tile, bar_full, w_policy);
                    }
                    bar_full += 8; bar_empty += 8; dst += kWStageBytes;
                    if (++stage == P.nsw) {
                        stage = 0; empty_parity ^= 1;
                        bar_full = w_full; bar_empty = w_empty; dst = smem_base + P.off_w;
                    }
                }
            }
        }
        return;
    }
    if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp runs the loops below converged and one elected lane issues the MMAs and the
        // commits: every value an MMA takes then lives in uniform registers (a lone surviving lane
        // would pay a register move per operand, and the issuing thread is the busiest of the CTA).
        if (rank != 0) return;
        const uint32_t idesc = ptx::idesc_bf16_f32(kPair ? 2 * kTileM : kTileM, P.n_pad);
        const uint32_t b_stage_bytes = (uint32_t)(kPair ? P.n_pad / 2 : P.n_pad) * (kBlockK * 2);
        const uint64_t a_desc0 = ptx::smem_desc_sw128(smem_base + P.off_w);
        const uint64_t b_desc0 = ptx::smem_desc_sw128(smem_base + P.off_b);
        // W ring, operand ring and accumulator-slot cursors, all advanced by increments
        int sw = 0, sb = 0, slot = 0;
        uint32_t w_parity = 0, b_parity = 0, slot_parity = 1;   // slot_parity: parity of the slot_empty wait
        uint64_t a_desc = a_desc0, b_desc = b_desc0;
        uint32_t bar_wf = w_full, bar_we = w_empty, bar_br = b_ready, bar_be = b_empty;
        if (P.staged) {
            // One wait and one commit per step: the step's barrier covers its W tiles and its operand
            // block.  The whole warp runs this loop converged and one elected lane issues: every
            // value an MMA takes then lives in uniform registers.
            const uint32_t step_units = P.step_bytes >> 4;
            b_desc = ptx::smem_desc_sw128(smem_base + P.off_w + (uint32_t)G * kWStageBytes);
            const uint64_t b_step0 = b_desc;
            for (int g = 0; g < n_groups; ++g) {
                const int t0 = g * G, t1 = min(my_tiles, t0 + G);
                const int slot0 = slot;
                for (int tile = t0; tile < t1; ++tile) {   // the group's accumulator slots must be drained
                    if (!ptx::mbar_wait_converged<kPollNs, true>(slot_empty + 8 * slot, slot_parity, s_abort, P.wait_limit)) {
                        if (lane == 0) atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_ACC_EMPTY);
                        return;
                    }
                    if (++slot == P.n_slots) { slot = 0; slot_parity ^= 1; }
                }
                ptx::tc_fence_after();
                for (int kb = 0; kb < P.kb_count; ++kb) {
                    if (!ptx::mbar_wait_converged<kPollNs, true>(bar_wf, w_parity, s_abort, P.wait_limit)) {
                        if (lane == 0) atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_FULL);
                        return;
                    }
                    ptx::tc_fence_after();
                    if (ptx::elect_one()) {
                        int sl = slot0;
                        uint32_t d_tmem = tmem_base + (uint32_t)(slot0 * P.n_pad);
                        uint64_t a_tile = a_desc;
                        for (int tile = t0; tile < t1; ++tile) {
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)   // 16 elements = 32 bytes = 2 descriptor units
                                if (kPair) ptx::mma_f16_pair(d_tmem, a_tile + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                                else ptx::mma_f16(d_tmem, a_tile + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                            a_tile += kWStageBytes >> 4;
                            d_tmem += (uint32_t)P.n_pad;
                            if (++sl == P.n_slots) { sl = 0; d_tmem = tmem_base; }
                        }
                        if (kPair) ptx::mma_commit_pair(bar_we, 3); else ptx::mma_commit(bar_we);
                    }
                    __syncwarp();
                    bar_wf += 8; bar_we += 8; a_desc += step_units; b_desc += step_units;
                    if (++sw == P.nsw) { sw = 0; w_parity ^= 1; bar_wf = w_full; bar_we = w_empty; a_desc = a_desc0; b_desc = b_step0; }
                }
                if (ptx::elect_one()) {
                    int sl = slot0;
                    for (int tile = t0; tile < t1; ++tile) {
                        if (kPair) ptx::mma_commit_pair(slot_full + 8 * sl, 3); else ptx::mma_commit(slot_full + 8 * sl);
                        if (++sl == P.n_slots) sl = 0;
                    }
                }
                __syncwarp();
            }
            return;
        }
        for (int g = 0; g < n_groups; ++g) {
            const int t0 = g * G, t1 = min(my_tiles, t0 + G);
            const int slot0 = slot;
            for (int tile = t0; tile < t1; ++tile) {   // the group's accumulator slots must be drained
                if (!ptx::mbar_wait_converged<kPollNs, false>(slot_empty + 8 * slot, slot_parity, s_abort, P.wait_limit)) {
                    if (lane == 0) atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_ACC_EMPTY);
                    return;
                }
                if (++slot == P.n_slots) { slot = 0; slot_parity ^= 1; }
            }
            ptx::tc_fence_after();
            for (int kb = 0; kb < P.kb_count; ++kb) {
                if (!ptx::mbar_wait_converged<kPollNs, false>(bar_br, b_parity, s_abort, P.wait_limit)) {
                    if (lane == 0) atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_OPERAND);
                    return;
                }
                int sl = slot0;
                uint32_t d_tmem = tmem_base + (uint32_t)(slot0 * P.n_pad);
                for (int tile = t0; tile < t1; ++tile) {
                    if (!ptx::mbar_wait_converged<kPollNs, false>(bar_wf, w_parity, s_abort, P.wait_limit)) {
                        if (lane == 0) atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_FULL);
                        return;
                    }
                    ptx::tc_fence_after();
                    if (ptx::elect_one()) {
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)   // 16 elements = 32 bytes = 2 descriptor units
                            ptx::mma_f16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                        ptx::mma_commit(bar_we);
                    }
                    __syncwarp();
                    bar_wf += 8; bar_we += 8; a_desc += kWStageBytes >> 4;
                    if (++sw == P.nsw) { sw = 0; w_parity ^= 1; bar_wf = w_full; bar_we = w_empty; a_desc = a_desc0; }
                    d_tmem += (uint32_t)P.n_pad;
                    if (++sl == P.n_slots) { sl = 0; d_tmem = tmem_base; }
                }
                if (ptx::elect_one()) ptx::mma_commit(bar_be);
                __syncwarp();
                bar_br += 8; bar_be += 8; b_desc += b_stage_bytes >> 4;
                if (++sb == P.nsb) { sb = 0; b_parity ^= 1; bar_br = b_ready; bar_be = b_empty; b_desc = b_desc0; }
            }
            if (ptx::elect_one()) {
                int sl = slot0;
                for (int tile = t0; tile < t1; ++tile) {
                    ptx::mma_commit(slot_full + 8 * sl);
                    if (++sl == P.n_slots) sl = 0;
                }
            }
            __syncwarp();
        }
        return;
    }
    if (warp >= kFirstExpWarp && P.staged) {
        if (warp < kFirstExpWarp + 4) {
            // warps 6-9 have no operand to build: they become a second set of epilogue warps
        } else {
            // -------------------------------------------------------------- operand producer
            // The masked rows were written to the staging buffer by mask_operand_kernel; one
            // thread streams the [n_pad x 64] block of every (group, block) step through TMA.
            if (threadIdx.x != (kFirstExpWarp + 4) * 32) return;
            if (P.pdl) ptx::griddep_wait();   // the staged operand is written by the kernel ahead
            const int b_rows = kPair ? P.n_pad / 2 : P.n_pad;      // a pair splits the operand rows
            const int b_row0 = row0 + (int)rank * b_rows;
            const uint32_t b_stage_bytes = (uint32_t)b_rows * (kBlockK * 2);
            // the operand block of a step lands behind the step's W tiles and counts on the same barrier
            const uint32_t dst0 = smem_base + P.off_w + (uint32_t)G * kWStageBytes;
            uint32_t bar_r = w_full, bar_e = w_empty, dst = dst0, parity = 1;
            int stage = 0;
            for (int g = 0; g < n_groups; ++g)
                for (int kb = 0, x = 0; kb < P.kb_count; ++kb, x += kBlockK) {
                    if (!ptx::mbar_wait<kPollNs>(bar_e, parity, s_abort, P.wait_limit)) {
                        atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_EMPTY);
                        return;
                    }
                    if (kPair) {
                        if (rank == 0) ptx::mbar_arrive_expect_tx(bar_r, 2 * b_stage_bytes);
                        ptx::tma_load_2d_pair(dst, &tmap_b, x, b_row0, ptx::map_to_cta(bar_r, 0));
                    } else {
                        ptx::mbar_arrive_expect_tx(bar_r, b_stage_bytes);
                        ptx::tma_load_2d(dst, &tmap_b, x, b_row0, bar_r);
                    }
                    bar_r += 8; bar_e += 8; dst += P.step_bytes;
                    if (++stage == P.nsw) { stage = 0; parity ^= 1; bar_r = w_full; bar_e = w_empty; dst = dst0; }
                }
            return;
        }
    } else if (warp >= kFirstExpWarp) {
        // ------------------------------------------------------------------ operand builders
        if (P.pdl) ptx::griddep_wait();       // H may be the output of the kernel ahead
        const int e = warp - kFirstExpWarp;
        const int grp = e % P.nsb, sub = e / P.nsb;
        const uint32_t b_stage_bytes = (uint32_t)P.n_pad * (kBlockK * 2);
        {   // rows [rows, n_pad) of every stage stay zero for the whole kernel
            const int tid = threadIdx.x - kFirstExpWarp * 32;
            uint4* bz = reinterpret_cast<uint4*>(smem + P.off_b);
            const int n16 = (int)(P.nsb * b_stage_bytes / 16);
            for (int x = tid; x < n16; x += kExpWarps * 32) bz[x] = make_uint4(0, 0, 0, 0);
            ptx::fence_proxy_async_smem();
            ptx::bar_sync(2, kExpWarps * 32);
        }
        unsigned char* my_stage = smem + P.off_b + grp * b_stage_bytes;
        const int n_items = my_rows * 8;           // (row, 16-byte chunk) pairs per block
        const int stride = wps * 32;               // threads working on this stage
        const int total_b = n_groups * P.kb_count;
        for (int m = grp; m < total_b; m += P.nsb) {
            const int kb = m % P.kb_count;
            const __nv_bfloat16* h_kb = P.H + kb * kBlockK;
            // the hidden-state loads do not depend on the stage being free: start them first
            uint4 hv[4];
            int it0 = sub * 32 + lane;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int it = it0 + u * stride;
                if (it < n_items) {
                    const int q = max(s_row[it >> 3].q, 0);
                    hv[u] = __ldg(reinterpret_cast<const uint4*>(h_kb + (size_t)q * P.d + (it & 7) * 8));
                }
            }
            if (!ptx::mbar_wait_warp<kPollNs>(b_empty + 8 * grp, ((m / P.nsb) & 1) ^ 1, s_abort,
                                              P.wait_limit)) {
                atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_EMPTY);
                break;
            }
            for (; it0 < n_items; it0 += 4 * stride) {
                // next batch of hidden-state chunks, in flight while this batch is masked
                uint4 hv_next[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int it = it0 + (4 + u) * stride;
                    if (it < n_items) {
                        const int q = max(s_row[it >> 3].q, 0);
                        hv_next[u] = __ldg(reinterpret_cast<const uint4*>(h_kb + (size_t)q * P.d + (it & 7) * 8));
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int it = it0 + u * stride;
                    if (it >= n_items) continue;
                    const int r = it >> 3, c = it & 7;
                    const RowInfo ri = s_row[r];
                    RowKey k{0, ri.s, ri.t, ri.i};
                    const uint32_t quad = (uint32_t)(kb * (kBlockK / 4) + c * 2);
                    const uint32_t mbits = keep4(quad, k, P.key0, P.key1, P.thr) |
                                           (keep4(quad + 1, k, P.key0, P.key1, P.thr) << 4);
                    uint4 o;
                    o.x = hv[u].x & mask_pair(mbits);
                    o.y = hv[u].y & mask_pair(mbits >> 2);
                    o.z = hv[u].z & mask_pair(mbits >> 4);
                    o.w = hv[u].w & mask_pair(mbits >> 6);
                    // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
                    const uint32_t off = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u +
                                         (uint32_t)((c ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(my_stage + off) = o;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) hv[u] = hv_next[u];
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(b_ready + 8 * grp);
        }
        // The operand is built (once per call): these warps now help with the epilogue as two more sets.
    }

    {
        // ------------------------------------------------------------------ epilogue
        // Warps 2-5, plus warps 6-9 in staged mode, where no operand is built.  Warp w reads TMEM
        // lanes 32*(w mod 4)..+31; the warps of a lane quarter share the column chunks.
        if (P.pdl) ptx::griddep_wait();       // global writes (and the shared per-row best) only after the kernel ahead
        const int ew = warp & 3;                      // lane quarter = row of s_best
        const int set = warp < kFirstExpWarp ? 0 : 1 + (warp - kFirstExpWarp) / 4;
        const int n_sets = P.staged ? 2 : 3;
        const int lane_base = ew * 32;                // TMEM lanes this warp may read
        // A group's accumulators finish together.  Columns are then taken 16 at a time and, for
        // each, the group's tiles are walked with a per-lane running maximum (a lane always sees
        // increasing vocabulary rows, so a strictly larger value replaces).  Only then are the
        // 32 lanes reduced, once per column and group, by a halving exchange: in each of four
        // rounds a lane hands half of its packed (key, inverted index) columns to its partner
        // and keeps the maxima of the other half, so that 16 columns cost 16 exchanges, not 80.
        unsigned long long* my_best = s_best + ew * P.n_pad;
        // accumulator columns past the launch's paths (padding of the MMA's N) are never read
        const int n_cols = min(P.n_pad, (my_rows + 15) & ~15);
        for (int n0 = 16 * set; n0 < n_cols; n0 += 16 * n_sets)
            if (lane < 16) my_best[n0 + lane] = 0ull;
        __syncwarp();
        const int m = lane_base + lane;
        const float neg_inf = __uint_as_float(0xFF800000u);
        bool alive = true;
        for (int g = 0; g < n_groups && alive; ++g) {
            const int t0 = g * G, t1 = min(my_tiles, t0 + G);
            for (int tile = t0; tile < t1; ++tile) {
                // the tcgen05.ld below needs the whole warp: the outcome of the wait is warp-uniform
                if (!ptx::mbar_wait_warp<kIdlePollNs>(slot_full + 8 * (tile % P.n_slots), (tile / P.n_slots) & 1,
                                                      s_abort, P.wait_limit)) {
                    atomicCAS(P.err, 0u, (uint32_t)ERR_WAIT_ACC_FULL);
                    alive = false;
                    break;
                }
            }
            if (!alive) break;
            ptx::tc_fence_after();
            const int slot0 = t0 % P.n_slots;
            const int v0 = v_cta0 + t0 * P.tile_rows + m;     // this lane's vocabulary row in tile t0
#pragma unroll 1
            for (int n0 = 16 * set; n0 < n_cols; n0 += 16 * n_sets) {
                float best[16];
                int bv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) { best[j] = neg_inf; bv[j] = 0; }
                int slot = slot0, v = v0;
                for (int tile = t0; tile < t1; ++tile, v += P.tile_rows) {
                    const bool valid = (m < P.tile_rows) && (v < P.V);
                    uint32_t acc[16];
                    ptx::tmem_ld16(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(slot * P.n_pad + n0), acc);
                    ptx::tmem_ld_wait();
                    if (++slot == P.n_slots) slot = 0;
                    if (P.sample) {
                        // sampling decode: one Philox call and two logarithms per logit
                        if (valid) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (n0 + j < my_rows) {
                                    const RowInfo ri = s_row[n0 + j];
                                    const RowKey k{0, ri.s, ri.t, ri.i};
                                    const float val = fmaf(__uint_as_float(acc[j]) * P.scale, P.inv_temp,
                                                           gumbel_noise((uint32_t)(v + P.v_offset), k, P.key0, P.key1));
                                    if (val > best[j]) { best[j] = val; bv[j] = v; }
                                }
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float val = __uint_as_float(acc[j]) * P.scale;
                            if (valid && val > best[j]) { best[j] = val; bv[j] = v; }
                        }
                    }
                    if (P.dbg_logits != nullptr && valid) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (n0 + j < my_rows)
                                P.dbg_logits[(size_t)(row0 + n0 + j) * P.V + v] =
                                    s_row[n0 + j].q >= 0 ? __uint_as_float(acc[j]) * P.scale
                                                         : __uint_as_float(0x7FC00000u);
                    }
                }
                unsigned long long p16[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    p16[j] = best[j] != neg_inf ? pack_best(float_key(best[j]), (uint32_t)(bv[j] + P.v_offset)) : 0ull;
                unsigned long long p8[8], p4[4], p2[2], p1;
                {
                    const bool up = (lane & 16) != 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const unsigned long long give = up ? p16[j] : p16[j + 8], keep = up ? p16[j + 8] : p16[j];
                        const unsigned long long got = __shfl_xor_sync(0xFFFFFFFFu, give, 16);
                        p8[j] = got > keep ? got : keep;
                    }
                }
                {
                    const bool up = (lane & 8) != 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned long long give = up ? p8[j] : p8[j + 4], keep = up ? p8[j + 4] : p8[j];
                        const unsigned long long got = __shfl_xor_sync(0xFFFFFFFFu, give, 8);
                        p4[j] = got > keep ? got : keep;
                    }
                }
                {
                    const bool up = (lane & 4) != 0;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const unsigned long long give = up ? p4[j] : p4[j + 2], keep = up ? p4[j + 2] : p4[j];
                        const unsigned long long got = __shfl_xor_sync(0xFFFFFFFFu, give, 4);
                        p2[j] = got > keep ? got : keep;
                    }
                }
                {
                    const bool up = (lane & 2) != 0;
                    const unsigned long long give = up ? p2[0] : p2[1], keep = up ? p2[1] : p2[0];
                    const unsigned long long got = __shfl_xor_sync(0xFFFFFFFFu, give, 2);
                    p1 = got > keep ? got : keep;
                }
                {
                    const unsigned long long got = __shfl_xor_sync(0xFFFFFFFFu, p1, 1);
                    p1 = got > p1 ? got : p1;
                }
                // lanes 2x and 2x+1 now hold column 8*bit4 + 4*bit3 + 2*bit2 + bit1 of the chunk
                if ((lane & 1) == 0) {
                    const int n = n0 + (lane >> 1);
                    if (p1 > my_best[n]) my_best[n] = p1;   // equal keys: the smaller index packs larger
                }
            }
            // this warp has read its share of the group's accumulators: hand the slots back
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                int sl = slot0;
                for (int tile = t0; tile < t1; ++tile) {   // the issuer's barrier is the leader's
                    if (kPair && rank != 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(slot_empty + 8 * sl, 0));
                    else ptx::mbar_arrive(slot_empty + 8 * sl);
                    if (++sl == P.n_slots) sl = 0;
                }
            }
        }
        ptx::tc_fence_before();
        ptx::bar_sync(3, 4 * n_sets * 32);
        if (warp >= kFirstExpWarp) return;      // the helpers are done; warps 2-5 finish the CTA
        for (int n = threadIdx.x - kFirstEpiWarp * 32; n < my_rows; n += 4 * 32) {
            unsigned long long b = s_best[n];
#pragma unroll
            for (int w = 1; w < 4; ++w) {
                unsigned long long c = s_best[w * P.n_pad + n];
                b = c > b ? c : b;
            }
            if (P.fold) atomicMax(P.best + row0 + n, b);
            else P.partials[(size_t)slice * P.rows_total + row0 + n] = b;
        }
        // ------------------------------------------------------------------ teardown
        // Every accumulator has been read, hence every MMA and every TMA load has completed.
        // After an abandoned wait: tell the other CTA of a pair to give up as well (its next poll
        // sees the flag), then give copies and MMAs that may still be in flight time to finish.
        if (*s_abort) {
            if (kPair && threadIdx.x == kFirstEpiWarp * 32)
                ptx::st_cluster_u32(ptx::map_to_cta(ptx::smem_u32(const_cast<int*>(s_abort)), rank ^ 1u), 1u);
            for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        }
        ptx::tc_fence_before();
        ptx::bar_sync(1, 4 * 32);
        if (warp == kFirstEpiWarp) {
            ptx::tc_fence_after();
            if (kPair) {
                // Neither CTA may free TMEM, or leave, while the other still reads accumulators or
                // sends signals here: tell the other CTA that this one is done, wait for its word.
                // This wait ignores the abort flag: after an abort the other CTA still has to notice
                // the flag, drain and send its word, which takes it at most one more wait limit.
                if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(dealloc_bar, rank ^ 1u));
                ptx::mbar_wait_warp<kPollNs>(dealloc_bar, 0, s_never, 2 * max(P.wait_limit, kWaitLimitCycles));
                ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
            } else {
                ptx::tmem_dealloc(tmem_base, kTmemCols);
            }
        }
        if (P.fold == 1) {
            // ---------------------------------------------------------------- folded finalize
            // Whoever draws the last ticket knows that every CTA's partials are in global memory.
            const int tid_e = threadIdx.x - kFirstEpiWarp * 32;
            __threadfence();
            ptx::bar_sync(1, 4 * 32);
            if (tid_e == 0) *s_ticket = atomicAdd(P.ticket, 1u);
            ptx::bar_sync(1, 4 * 32);
            if (*s_ticket == gridDim.x - 1) {
                __threadfence();
                int32_t* scratch = reinterpret_cast<int32_t*>(smem + P.off_w);   // the rings are idle by now
                if (P.fin.B == 1) {
                    finalize_sequence(P.best, 1, P.rows_total, P.fin, 0, scratch, tid_e, 4 * 32, NamedSync{1, 4 * 32});
                } else {
                    // several sequences: each warp takes its own (a sequence is a chain of dependent
                    // global accesses of about 10 us; four of them run side by side), with scratch
                    // of its own if the idle rings have room for it
                    const uint32_t need = ((uint32_t)finalize_smem_bytes_dev(P.fin.T, P.fin.K + P.fin.plain, P.fin.N) + 15u) & ~15u;
                    const int n_par = min(4, (int)(P.off_rowinfo / need));
                    const int w = warp - kFirstEpiWarp;
                    if (w < n_par)
                        for (int b = w; b < P.fin.B; b += n_par)
                            finalize_sequence(P.best, 1, P.rows_total, P.fin, b, scratch + (size_t)w * (need / 4), lane, 32,
                                              WarpSync{});
                    ptx::bar_sync(1, 4 * 32);
                }
                if (P.fin.done != nullptr) {   // a host-buffer call: every result is written, tell the waiting host
                    __threadfence_system();
                    ptx::bar_sync(1, 4 * 32);
                    if (tid_e == 0) *reinterpret_cast<volatile uint32_t*>(P.fin.done) = P.fin.done_value;
                }
                for (int n = tid_e; n < P.rows_total; n += 4 * 32) P.best[n] = 0ull;   // ready for the next call
                if (tid_e == 0) *P.ticket = 0u;
            }
        }
    }

}

// Eq. 1 and the numerator of Eq. 2 for every path of a call whose rows do not fit the
// in-kernel builders: row r of the staging buffer receives hidden row q(r) with the dropped
// elements zeroed.  One thread per 16-byte chunk (two Philox quads).
__global__ void __launch_bounds__(256)
mask_operand_kernel(const __nv_bfloat16* __restrict__ H, __nv_bfloat16* __restrict__ out, int rows, int d,
                    RowMap map, uint32_t key0, uint32_t key1, uint32_t thr, uint32_t* __restrict__ err) {
    // The head kernel behind this one may be scheduled at once: it streams W until its operand
    // producer needs these rows, and that thread waits for this kernel to finish.  This kernel may
    // itself have been scheduled early: the kernel ahead may still read the staging buffer or
    // write H, so nothing is touched before it has finished.
    ptx::griddep_launch_dependents();
    ptx::griddep_wait();
    const int chunks = d >> 3;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)rows * chunks) return;
    const int r = (int)(idx / chunks), c = (int)(idx - (long long)r * chunks);
    RowKey k;
    if (!row_key(map, r, k) && c == 0) atomicExch(err, (uint32_t)ERR_BAD_ROW);
    const uint32_t mbits = keep4((uint32_t)(2 * c), k, key0, key1, thr) |
                           (keep4((uint32_t)(2 * c + 1), k, key0, key1, thr) << 4);
    const uint4 hv = __ldg(reinterpret_cast<const uint4*>(H + (size_t)k.q * d + c * 8));
    uint4 o;
    o.x = hv.x & mask_pair(mbits);
    o.y = hv.y & mask_pair(mbits >> 2);
    o.z = hv.z & mask_pair(mbits >> 4);
    o.w = hv.w & mask_pair(mbits >> 6);
    *reinterpret_cast<uint4*>(out + (size_t)r * d + c * 8) = o;
}

// The same for the regular row order (paths of a position next to each other): a block takes 32
// chunks of one hidden row, fetches them once and writes them under the mask of every path of the
// row, eight paths at a time.  H may then be host memory that the device can read (the host-buffer
// call): each hidden element crosses the host link once; the draft tokens of such a call ride along.
__global__ void __launch_bounds__(256)
mask_operand_by_position_kernel(const __nv_bfloat16* __restrict__ H, __nv_bfloat16* __restrict__ out, int d,
                                RowMap map, uint32_t key0, uint32_t key1, uint32_t thr,
                                const int32_t* __restrict__ draft_src, int32_t* __restrict__ draft_dst, int n_draft) {
    ptx::griddep_launch_dependents();
    __shared__ uint4 s_h[32];
    const int chunks = d >> 3, tiles = (chunks + 31) >> 5;
    const int q = (int)(blockIdx.x / tiles), c = (int)(blockIdx.x % tiles) * 32 + (threadIdx.x & 31);
    const int pl = threadIdx.x >> 5;
    const int kp = map.K + map.plain_extra;
    // The mask of the thread's first path depends on indices only: it is drawn before the wait,
    // while the kernel ahead drains (and, for a host-buffer call, before H has crossed the link).
    uint32_t mbits0 = 0;
    if (c < chunks && pl < kp) {
        RowKey k0;
        row_key(map, q * kp + pl, k0);
        mbits0 = keep4((uint32_t)(2 * c), k0, key0, key1, thr) | (keep4((uint32_t)(2 * c + 1), k0, key0, key1, thr) << 4);
    }
    ptx::griddep_wait();   // (see mask_operand_kernel)
    if (draft_src != nullptr && blockIdx.x == 0)
        for (int x = threadIdx.x; x < n_draft; x += 256) draft_dst[x] = draft_src[x];
    if (pl == 0 && c < chunks) s_h[threadIdx.x] = __ldg(reinterpret_cast<const uint4*>(H + (size_t)q * d + c * 8));
    __syncthreads();
    if (c >= chunks) return;
    const uint4 hv = s_h[threadIdx.x & 31];
    for (int i = pl; i < kp; i += 8) {
        const int r = q * kp + i;
        uint32_t mbits = mbits0;
        if (i != pl) {
            RowKey k;
            row_key(map, r, k);   // always valid in the regular order
            mbits = keep4((uint32_t)(2 * c), k, key0, key1, thr) | (keep4((uint32_t)(2 * c + 1), k, key0, key1, thr) << 4);
        }
        uint4 o;
        o.x = hv.x & mask_pair(mbits);
        o.y = hv.y & mask_pair(mbits >> 2);
        o.z = hv.z & mask_pair(mbits >> 4);
        o.w = hv.w & mask_pair(mbits >> 6);
        *reinterpret_cast<uint4*>(out + (size_t)r * d + c * 8) = o;
    }
}

}  // namespace

// ------------------------------------------------------------------------------ host side

// How the vocabulary is cut for launches that cover `row_blocks` blocks of 256 paths at once:
// the SMs are shared out between the row blocks, so a slice is `row_blocks` times longer.
struct SliceGeometry {
    CUtensorMap tmap_w;     // box [64 x tile_rows]
    int n_ctas;             // CTAs per row block = vocabulary slices
    int tiles_per_cta, tile_rows, slice_rows;
};

struct FusedState {
    SliceGeometry geo[2];   // [0]: one row block per launch, [1]: two
    // staging buffer for the masked operand of calls with too many rows for the in-kernel
    // builders, and one tensor map per box height n_pad = 16, 32, ..., 256 over it
    __nv_bfloat16* staging;
    int staging_rows;
    CUtensorMap tmap_b[kMaxNPad / 8];   // boxes of 8, 16, ..., 256 rows
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up at run time so that the library has no link-time
// dependency on libcuda (it must load on machines without a driver).
EncodeTiledFn encode_tiled_fn() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(fn);
}

struct SmemPlan {
    int nsw, nsb, group_tiles, n_slots, staged;
    int pair;    // run as clusters of two CTAs that split the operand rows
    int n_pad;   // operand rows after padding: a multiple of 16, of 32 for pairs
    uint32_t step_bytes;   // staged: bytes of one step (the group's W tiles, then the operand block)
    uint32_t off_w, off_b, off_rowinfo, off_best, off_bar, total;
};

#ifndef DM_EXPOSE_SLOTS
#define DM_EXPOSE_SLOTS 0
#endif

// Choose the operand mode (builders, staged, staged as CTA pairs) and the tile grouping, then
// split the 227 KB of shared memory between the rings.
bool plan_smem(int rows, int tiles_per_cta, SmemPlan* out) {
    SmemPlan best{};
    int n_pad = (rows + 15) & ~15;
    // A slice of several tiles is staged even where it would fit TMEM as one group (single-tile
    // groups: all but the last tile's epilogue overlaps the MMAs that follow), and staged launches
    // run as CTA pairs: half the MMA issue work and half the operand bytes per SM.  Measured faster
    // than lone CTAs, and than the one-group mode with its in-kernel Philox builders, at every
    // path count (Llama-3-8B head, 8-32 paths: 157 against 163 us per call; Qwen3-8B: 188 against
    // 193 us), so the builders are left with the heads whose slices are a single tile.  Pair
    // launches narrower than 64 accumulator columns are padded to 64 (N = 32 MMAs were 6 us slower
    // on the Llama-3-8B head); the columns past the call's paths are computed and ignored.
    const bool force_staged = n_pad >= DM_STAGED_MIN_NPAD && tiles_per_cta > 1;
    best.pair = ((tiles_per_cta > kTmemCols / n_pad || force_staged) && n_pad >= kPairMinNPad) ? 1 : 0;
    if (best.pair) n_pad = (rows + DM_PAIR_GRAN - 1) & ~(DM_PAIR_GRAN - 1);
    if (best.pair && n_pad < DM_PAIR_PAD_MIN) n_pad = DM_PAIR_PAD_MIN;
    best.n_pad = n_pad;
    best.n_slots = kTmemCols / n_pad;
    const uint32_t b_stage = (uint32_t)(best.pair ? n_pad / 2 : n_pad) * (kBlockK * 2);
    const uint32_t fixed = 256u * sizeof(RowInfo) + 4u * n_pad * 8u + kBarBytes;
    const uint32_t avail = kSmemLimit - 1024 - fixed;
    if (tiles_per_cta <= best.n_slots && !force_staged) {
        // One group: the whole slice is live at once and the builders generate the masks in
        // registers, once per call.  Four small operand stages, the rest goes to the W ring.
        best.group_tiles = tiles_per_cta;
        best.staged = 0;
        best.nsb = 4;
        for (;;) {   // shrink the operand ring until the W ring has six stages (or the ring is at two)
            const uint32_t used = (uint32_t)best.nsb * b_stage;
            if (used + 2u * kWStageBytes <= avail) {
                best.nsw = (int)((avail - used) / kWStageBytes);
                if (best.nsw > kMaxWStages) best.nsw = kMaxWStages;
                if (best.nsw >= 6 || best.nsb == 2) break;
            }
            if (best.nsb == 2) return false;
            best.nsb = 2;   // the eight builder warps split evenly over 4 or 2 stages
        }
        best.off_w = 0;
        best.off_b = (uint32_t)best.nsw * kWStageBytes;
        best.off_rowinfo = best.off_b + (uint32_t)best.nsb * b_stage;
    } else {
        // Several groups: the operand would have to be rebuilt for every group, so it is staged
        // through global memory by mask_operand_kernel and streamed in by TMA (no builders).
        // A group takes at most half of the accumulator slots, so that the epilogue of one group
        // overlaps the MMAs of the next (with two or three slots: single tiles).  The operand is
        // then fetched once per group, from L2, which costs nothing measurable: halving or
        // quartering those loads left the kernel's time unchanged.  Group sizes are evened out.
        int g = best.n_slots / 2;
        if (g < 1) g = 1;
        if (best.n_slots <= DM_EXPOSE_SLOTS) g = best.n_slots;
        // Up to 64 operand rows the epilogue of a tile is short next to its MMAs: single-tile groups
        // leave one tile's epilogue exposed at the end instead of half the slice's (3 us of 170 on the
        // Llama-3-8B head at 40-64 paths; from 96 rows up pairs of tiles are the faster choice).
        if (n_pad <= 64) g = 1;
        if (g >= tiles_per_cta) g = (tiles_per_cta + 1) / 2;   // at least two groups: the first epilogue overlaps
        const int n_groups = (tiles_per_cta + g - 1) / g;
        best.group_tiles = (tiles_per_cta + n_groups - 1) / n_groups;
        best.staged = 1;
        // One ring of steps; a step = the group's W tiles of one hidden-size block + the operand block.
        best.step_bytes = (uint32_t)best.group_tiles * kWStageBytes + b_stage;
        best.nsw = (int)(avail / best.step_bytes);
        if (best.nsw > kMaxWStages) best.nsw = kMaxWStages;
        if (best.nsw < 2) return false;
        best.nsb = 1;   // no separate operand ring
        best.off_w = 0;
        best.off_b = 0;
        best.off_rowinfo = (uint32_t)best.nsw * best.step_bytes;
    }
    best.off_best = best.off_rowinfo + 256u * sizeof(RowInfo);
    best.off_bar = best.off_best + 4u * n_pad * 8u;
    best.total = best.off_bar + kBarBytes + 1024u;
    *out = best;
    return best.total <= (uint32_t)kSmemLimit;
}

}  // namespace

bool fused_supported(const HeadDesc& head, int rows) {
    return head.dtype == DM_BF16 && head.d >= kBlockK && head.d % kBlockK == 0 && head.V >= 1 && rows >= 1;
}

int fused_create(FusedState** out, const HeadDesc& head, int max_rows, int /*max_hidden_rows*/,
                 size_t* bytes) {
    *out = nullptr;
    *bytes = 0;
    if (!fused_supported(head, 1)) return DM_OK;   // this head runs on the CUDA-core kernel
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return DM_ECUDA;
    FusedState* fs = new (std::nothrow) FusedState();
    if (fs == nullptr) return DM_ECUDA;
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) { delete fs; return DM_ECUDA; }
    const cuuint64_t gdim[2] = {(cuuint64_t)head.d, (cuuint64_t)head.V};
    const cuuint64_t gstride[1] = {(cuuint64_t)head.d * 2};
    const cuuint32_t estride[2] = {1, 1};
    CUresult r = CUDA_SUCCESS;
    for (int g = 0; g < 2; ++g) {
        // g = 0: every SM gets a vocabulary slice; g = 1: two row blocks per launch, so half as
        // many slices (an even number of them: CTA pairs take two neighbouring slices)
        SliceGeometry& geo = fs->geo[g];
        int ctas = g == 0 ? sms : (sms / 2) & ~1;
        if (ctas < 1) ctas = 1;
        int per = (head.V + ctas - 1) / ctas;
        if (per < 64) per = 64;
        geo.tiles_per_cta = (per + kTileM - 1) / kTileM;
        geo.tile_rows = (per + geo.tiles_per_cta - 1) / geo.tiles_per_cta;
        geo.slice_rows = geo.tiles_per_cta * geo.tile_rows;
        geo.n_ctas = (head.V + geo.slice_rows - 1) / geo.slice_rows;
        const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)geo.tile_rows};
        r = encode(&geo.tmap_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(head.W), gdim, gstride, box,
                   estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { delete fs; return DM_ECUDA; }
    }
    if (cudaFuncSetAttribute(fused_head_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) !=
            cudaSuccess ||
        cudaFuncSetAttribute(fused_head_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) !=
            cudaSuccess) {
        cudaGetLastError();
        delete fs;
        return DM_ECUDA;
    }
    // Staging buffer, only if the largest launch this context may see needs it.
    fs->staging = nullptr;
    fs->staging_rows = 0;
    const int widest = max_rows < kMaxNPad ? max_rows : kMaxNPad;
    SmemPlan plan;
    if (!plan_smem(widest, fs->geo[0].tiles_per_cta, &plan)) { delete fs; return DM_EUNSUPPORTED; }
    SmemPlan plan_two{};   // launches over two row blocks cut the vocabulary into longer slices
    const bool two_staged = max_rows > kMaxNPad && plan_smem(kMaxNPad, fs->geo[1].tiles_per_cta, &plan_two) &&
                            plan_two.staged;
    if (plan.staged || two_staged) {
        // room for the widest box a launch may ask for: a padded pair launch reads 2 x 32 rows
        fs->staging_rows = (max_rows + 31) & ~31;
        if (fs->staging_rows < DM_PAIR_PAD_MIN) fs->staging_rows = DM_PAIR_PAD_MIN;
        const size_t n = (size_t)fs->staging_rows * head.d * sizeof(__nv_bfloat16);
        if (cudaMalloc(&fs->staging, n) != cudaSuccess) { cudaGetLastError(); delete fs; return DM_ECUDA; }
        if (cudaMemset(fs->staging, 0, n) != cudaSuccess) { cudaGetLastError(); cudaFree(fs->staging); delete fs; return DM_ECUDA; }
        const cuuint64_t sdim[2] = {(cuuint64_t)head.d, (cuuint64_t)fs->staging_rows};
        for (int n8 = 1; n8 <= kMaxNPad / 8; ++n8) {
            const cuuint32_t sbox[2] = {(cuuint32_t)kBlockK, (cuuint32_t)(8 * n8)};
            if (8 * n8 > fs->staging_rows) { fs->tmap_b[n8 - 1] = fs->tmap_b[0]; continue; }
            r = encode(&fs->tmap_b[n8 - 1], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, fs->staging, sdim, gstride, sbox,
                       estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { cudaFree(fs->staging); delete fs; return DM_ECUDA; }
        }
        *bytes = n;
    }
    *out = fs;
    return DM_OK;
}

namespace {

// The mask pass over all rows of a call: by position in the regular row order (H is then read once
// per element, and the drafts of a host-buffer call may ride along), by row for explicit row lists.
int launch_mask_operand(int d, const void* H, int rows, const RowMap& map, const MaskKey& mk, __nv_bfloat16* out,
                        uint32_t* err, cudaStream_t stream, bool pdl, const int32_t* draft_src = nullptr,
                        int32_t* draft_dst = nullptr, int n_draft = 0) {
    // With programmatic stream serialization the pass is scheduled while the kernel ahead (the head
    // kernel of the previous call, say) drains, and so is the head kernel behind it: its prologue
    // and the fill of its W ring then overlap that tail.  Not for explicit row lists, which could
    // themselves be the output of the kernel ahead.
    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = (pdl && map.sel == nullptr) ? 1 : 0;
    const __nv_bfloat16* Hb = static_cast<const __nv_bfloat16*>(H);
    cudaError_t e;
    if (map.sel == nullptr) {
        const int kp = map.K + map.plain_extra, tiles = (d / 8 + 31) / 32;
        if (rows % kp != 0) return DM_EINVAL;
        cfg.gridDim = dim3((unsigned)((rows / kp) * tiles));
        e = cudaLaunchKernelEx(&cfg, mask_operand_by_position_kernel, Hb, out, d, map, mk.key0, mk.key1, mk.thr,
                               draft_src, draft_dst, n_draft);
    } else {
        const long long n_threads = (long long)rows * (d / 8);
        cfg.gridDim = dim3((unsigned)((n_threads + 255) / 256));
        e = cudaLaunchKernelEx(&cfg, mask_operand_kernel, Hb, out, rows, d, map, mk.key0, mk.key1, mk.thr, err);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace

int fused_debug_operand(const HeadDesc& head, const void* H, int rows, const RowMap& map, const MaskKey& mk,
                        void* out, uint32_t* err, cudaStream_t stream) {
    if (head.dtype != DM_BF16 || head.d % 8 != 0) return DM_EUNSUPPORTED;
    return launch_mask_operand(head.d, H, rows, map, mk, static_cast<__nv_bfloat16*>(out), err, stream, false);
}

void fused_destroy(FusedState* fs) {
    if (fs == nullptr) return;
    cudaFree(fs->staging);
    delete fs;
}

int fused_launch(FusedState* fs, const HeadDesc& head, const void* H, int /*n_hidden*/, int rows,
                 const RowMap& map, const MaskKey& mk, int* n_slices_out, unsigned long long* partials,
                 float* dbg_logits, uint32_t* err, cudaStream_t stream, int* launches_out,
                 const FinalizeArgs* fin, unsigned int* ticket, unsigned long long* best, bool* folded_out,
                 unsigned long long* packed_out, long long wait_limit, bool allow_pdl, const HostInputs* host,
                 bool* best_reduced_out) {
    if (folded_out) *folded_out = false;
    if (best_reduced_out) *best_reduced_out = false;
    if (fs == nullptr || !fused_supported(head, rows) || fs->geo[0].n_ctas + 1 > kMaxSlices) return DM_EUNSUPPORTED;
    // Slices of one-block launches: an even count (pairs need one); a CTA whose slice lies past the
    // end of W contributes empty partials.
    const int slices1 = (fs->geo[0].n_ctas + 1) & ~1;
    const int slices2 = (fs->geo[1].n_ctas + 1) & ~1;
    // More than 256 paths left: two row blocks (of 256, or of half the rest) are taken in one
    // launch.  The two CTAs that share a vocabulary slice stream the same W tiles side by side, so
    // W comes from HBM once for both blocks (the second reader hits L2) and a CTA runs twice as
    // many tiles.  Needs the staged operand (the longer slices never fit TMEM as one group).
    SmemPlan plan2;
    const bool use_two = rows > kMaxNPad && dbg_logits == nullptr && fs->staging != nullptr &&
                         plan_smem(kMaxNPad, fs->geo[1].tiles_per_cta, &plan2) && plan2.staged;
    if (use_two && slices2 < slices1) {
        // the two kinds of launch fill different numbers of slice rows of the partials: clear them
        if (cudaMemsetAsync(partials, 0, (size_t)slices1 * rows * sizeof(unsigned long long), stream) != cudaSuccess)
            return DM_ECUDA;
    }
    int launches = 0;
    bool operand_staged = false;
    if (host != nullptr) {
        // Inputs of the host-buffer call.  If the call's masked rows are staged in the regular row
        // order, the mask pass reads H where it is and brings the drafts along; otherwise a small
        // kernel copies both into the device staging buffer first.
        SmemPlan first;
        const int first_rows = rows < kMaxNPad ? rows : kMaxNPad;
        const bool direct = map.sel == nullptr && fs->staging != nullptr && rows <= fs->staging_rows &&
                            plan_smem(first_rows, fs->geo[0].tiles_per_cta, &first) && first.staged;
        if (direct) {
            const int st = launch_mask_operand(head.d, host->h_src, rows, map, mk, fs->staging, err, stream, allow_pdl,
                                               host->draft_src, host->draft_dst, host->n_draft);
            if (st != DM_OK) return st;
            operand_staged = true;
        } else {
            const int st = launch_host_gather(host->h_src, host->h_bytes, host->draft_src, host->n_draft, host->h_dst,
                                              host->draft_dst, stream);
            if (st != DM_OK) return st;
        }
        H = host->h_dst;   // (never read when the operand is staged)
        ++launches;
    }
    for (int row0 = 0; row0 < rows;) {
        const int left = rows - row0;
        int row_blocks = 1, block_rows = left < kMaxNPad ? left : kMaxNPad;
        if (use_two && left > kMaxNPad) {
            row_blocks = 2;
            block_rows = left >= 2 * kMaxNPad ? kMaxNPad : (((left + 1) / 2 + 31) & ~31);   // two halves
            SmemPlan probe;   // blocks this narrow may fit TMEM as one group: then no sharing of W
            if (!plan_smem(block_rows, fs->geo[1].tiles_per_cta, &probe) || !probe.staged) {
                row_blocks = 1;
                block_rows = kMaxNPad;
            }
        }
        const SliceGeometry& geo = fs->geo[row_blocks - 1];
        const int grid = (row_blocks == 2 ? slices2 : slices1) * row_blocks;
        FusedParams P{};
        P.H = static_cast<const __nv_bfloat16*>(H);
        P.d = head.d; P.V = head.V; P.v_offset = head.v_offset;
        P.rows = block_rows;
        P.row0 = row0; P.rows_total = rows;
        P.row_blocks = row_blocks;
        SmemPlan plan;
        if (!plan_smem(P.rows, geo.tiles_per_cta, &plan)) return DM_EUNSUPPORTED;
        P.n_pad = plan.n_pad;
        P.kb_count = head.d / kBlockK;
        P.tiles_per_cta = geo.tiles_per_cta; P.tile_rows = geo.tile_rows; P.slice_rows = geo.slice_rows;
        P.group_tiles = plan.group_tiles; P.n_slots = plan.n_slots;
        P.nsw = plan.nsw; P.nsb = plan.nsb; P.staged = plan.staged; P.step_bytes = plan.step_bytes;
        if (plan.staged && !operand_staged) {
            // one pass over all rows of the call; the launches below read their own rows of it
            if (fs->staging == nullptr || rows > fs->staging_rows) return DM_EWORKSPACE;
            const int st = launch_mask_operand(head.d, H, rows, map, mk, fs->staging, err, stream, allow_pdl);
            if (st != DM_OK) return st;
            operand_staged = true;
            ++launches;
        }
        P.off_w = plan.off_w; P.off_b = plan.off_b;
        P.off_rowinfo = plan.off_rowinfo; P.off_best = plan.off_best; P.off_bar = plan.off_bar;
        P.map = map;
        P.key0 = mk.key0; P.key1 = mk.key1; P.thr = mk.thr; P.scale = mk.scale;
        P.sample = mk.sample; P.inv_temp = mk.inv_temp;
        P.partials = partials; P.dbg_logits = dbg_logits; P.err = err;
        // a call of one launch finishes itself; larger calls leave it to finalize_kernel
        P.fold = (fin != nullptr && ticket != nullptr && best != nullptr && rows <= kMaxNPad &&
                  finalize_smem_bytes(fin->T, fin->K + fin->plain, fin->N) <= 32 * 1024) ? 1 : 0;
        P.ticket = ticket;
        P.best = best;
        if (P.fold) { P.fin = *fin; if (folded_out) *folded_out = true; }
        if (packed_out != nullptr) {
            // the caller wants one packed word per path: reduce straight into the caller's array
            // (which the caller has zeroed on this stream); every launch of the call has rows of its own
            P.fold = 2;
            P.best = packed_out;
            if (folded_out) *folded_out = true;
        } else if (!P.fold && best != nullptr && best_reduced_out != nullptr) {
            // a call of several launches: each reduces its rows into the per-row array; one small
            // finalize kernel then reads one word per path (the caller zeroes the array afterwards)
            P.fold = 2;
            *best_reduced_out = true;
        }
        // Programmatic stream serialization, except when the row selection of the debug call could
        // itself be the output of the kernel ahead (it is read in the prologue).
        P.pdl = (map.sel == nullptr && allow_pdl) ? 1 : 0;
        P.w_evict_first = (size_t)head.V * head.d * sizeof(__nv_bfloat16) > (size_t)DM_W_EVICT_FIRST_MIN_BYTES ? 1 : 0;
        P.wait_limit = wait_limit > 0 ? wait_limit : kWaitLimitCycles;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = plan.total;
        cfg.stream = stream;
        cudaLaunchAttribute attrs[2]{};
        int n_attrs = 0;
        if (P.pdl) {
            attrs[n_attrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attrs[n_attrs].val.programmaticStreamSerializationAllowed = 1;
            ++n_attrs;
        }
        if (plan.pair) {   // clusters of two CTAs
            attrs[n_attrs].id = cudaLaunchAttributeClusterDimension;
            attrs[n_attrs].val.clusterDim.x = 2; attrs[n_attrs].val.clusterDim.y = 1; attrs[n_attrs].val.clusterDim.z = 1;
            ++n_attrs;
        }
        cfg.attrs = attrs;
        cfg.numAttrs = n_attrs;
        const cudaError_t launched =
            plan.pair ? cudaLaunchKernelEx(&cfg, fused_head_kernel<true>, geo.tmap_w, fs->tmap_b[P.n_pad / 16 - 1], P)
                      : cudaLaunchKernelEx(&cfg, fused_head_kernel<false>, geo.tmap_w,
                                           plan.staged ? fs->tmap_b[P.n_pad / 8 - 1] : geo.tmap_w, P);
        if (launched != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        if (cudaGetLastError() != cudaSuccess) return DM_ECUDA;
        ++launches;
        row0 += row_blocks * block_rows;
    }
    *n_slices_out = slices1;
    *launches_out = launches;
    return DM_OK;
}

}  // namespace dm
