// BCSR SpMM kernel for sm_100a (Sec. 3.1 - 3.3 of the paper, re-designed for Blackwell).
//
// Work unit ("tile"): one block-row I of A times BN_T = 128 * GROUPS columns of B
// ("tokens").  For every stored block p of the block-row the tile accumulates
//     D[n, r] += sum_c  B[J_p*b + c, n0 + n] * A_p[r, c]
// i.e. the tokens sit on the 128 TMEM lanes (MMA M side, operand read MN-major straight
// from row-major B) and the b rows of the block are the MMA N side (operand = the stored
// block, K-major).  One shape therefore serves b = 16, 32, 64 and 128, and an epilogue thread
// holds one token: a warp's registers are a [C row][32 tokens] tile, row-major like C.
//
// Roles (192 threads, one CTA per SM, persistent):
//   warp 0      TMA producer: per pipeline stage (1, 2 or 4 stored blocks) one request for
//               the A blocks and one 3-D request per block for its B tile (2*GROUPS boxes of
//               b x 64 tokens), issued by different lanes of one warp-instruction, into a
//               STAGES-deep shared-memory ring; full/empty mbarriers with phase bits.
//   warp 1      MMA issuer: one thread issues tcgen05.mma into one of two TMEM accumulator
//               buffers; tcgen05.commit frees the ring slot / publishes the accumulator.
//   warps 2-5   epilogue: tcgen05.ld -> registers -> one of the warp's staging tiles in shared
//               memory (16 fp32 or 32 16-bit C rows x 32 tokens = 2 KB; a ring of as many tiles
//               per warp as fit beside the stage ring, so that the warp fills the next tile
//               while earlier TMA stores are still reading theirs) -> one TMA store per tile,
//               which also clips at the edges of C (zeros for empty block-rows); overlaps the
//               next tile's MMAs thanks to the second TMEM buffer.
// Value types (FMT): fp16, bf16 (K = 16 per MMA), TF32 (fp32 storage, K = 8; the token tile then
// uses the 128-byte swizzle with 32-byte atoms, and blocks wider than 32 columns pass through the
// ring in 32-column slices), E4M3 (K = 32): a K step is 32 bytes of an operand row in all of them.
// A tile of one part of a K-split block-row (record x < 0) stores an fp32 partial tile through
// tmP instead of C; bcsr_merge_kernel adds the parts in order.
// Optional variants, all template parameters:
//   CT = 1   C is written in the input's 16-bit type instead of fp32.
//   CM = 1   "column-major" operands (the layout of the paper's BCSR kernel, Sec. 3.2, and of a
//            linear layer Y = X W^T, Sec. 4.4): B is given as X[N][k] (one row per token, k
//            contiguous) and C as Y[N][m].  The token tile is then a K-major MMA operand
//            (rows of min(b, 64) elements, swizzle = row bytes; b = 128 as two K halves), and
//            the staging tile is [32 tokens][16 or 32 columns of Y].
//   DYN = 1  dynamic tile scheduling with Cluster Launch Control (the direction Sec. 5 points
//            to after the paper's atomic-counter scheduler lost to the hardware block
//            scheduler, Sec. 3.6): the grid has one CTA per tile, in the schedule's global order
//            (slab by slab, longest block-row first); a CTA runs tile blockIdx.x and then
//            keeps cancelling the launch of not-yet-started CTAs and running their tiles.  A
//            seventh warp fetches the tile indices ahead of time into a four-deep ring that
//            the six working warps read.
// The host deals tiles to CTAs ahead of time: slab by slab (a slab = token tiles whose B rows
// fit in L2), longest block-row first, each tile to the least loaded CTA; CTA c walks its list.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"

namespace spmm {

namespace {

// ES = bytes per input element: 2 (fp16 / bf16), 4 (fp32 storage, TF32 arithmetic), or 1 (E4M3,
// column-major operands only).
// H = rows of one stored block = the MMA's N extent: B for the format's own b x b blocks, 128 for
// the stacked blocks of a row group (128 / b block-rows on top of one another, see format.h).
// CS = bytes per element of C, CM = column-major operands: they fix the epilogue's staging tile.
// A pipeline stage holds one "unit": kBps whole blocks (small b), or one of the kKS column
// slices a block is cut into where its rows are longer than 128 bytes of 4-byte elements
// (b = 64 / 128 with TF32: units of 32 columns, so that a stage stays a fraction of shared memory).
template <int B, int H, int GROUPS, int STAGES, int ES, int CS, int CM>
struct BcsrCfg {
    static constexpr int kKS = (H == B) ? bcsr_k_split(B, ES) : 1;     // stage units per block
    static constexpr int kKB = B / kKS;                      // columns of A (= rows of B) per unit
    static constexpr int kBB = kKB * ES;                     // bytes of one unit row (its K extent)
    static constexpr int kKSteps = kBB / 32;                 // MMAs per unit and token group (32 bytes of K each)
    static constexpr int kBnT = 128 * GROUPS;
    static constexpr int kTokBox = 128 / ES;                 // tokens per 128-byte box row (row-major B)
    static constexpr int kNBox = GROUPS * (128 / kTokBox);   // boxes per unit (row-major B)
    static constexpr int kBoxBytes = kKB * 128;              // kKB k-rows x 128 B (row-major B)
    static constexpr int kDenseBytes = kBnT * kBB;           // B tile of one unit
    static constexpr int kABytes = H * kBB;
    // Small blocks carry too little work for the fixed cost of a pipeline stage (barrier
    // round trip, request issue, MMA hand-off): a stage holds several consecutive stored
    // blocks of the block-row, their B tiles first, then their A blocks (one request).
    static constexpr int kBps = bcsr_blocks_per_stage(B);
    static constexpr int kStageBytes = ((kBps * (kDenseBytes + kABytes) + 1023) / 1024) * 1024;
    static constexpr int kAOff = kBps * kDenseBytes;         // A blocks inside the stage
    static constexpr int kARowBytes = kBB < 128 ? kBB : 128;
    static constexpr uint32_t kASwizzle = kARowBytes == 128 ? SWZ_128B : (kARowBytes == 64 ? SWZ_64B : SWZ_32B);
    // column-major operands: a token group's tile is 128 rows x kXRowBytes, K-major
    static constexpr int kXRowBytes = kARowBytes;
    static constexpr int kXGroupBytes = 128 * kXRowBytes;    // one K half of one token group
    static constexpr int kAccCols = GROUPS * H;
    static constexpr int kTmemCols = (2 * kAccCols <= 32) ? 32 : (2 * kAccCols <= 64 ? 64 : (2 * kAccCols <= 128 ? 128 : (2 * kAccCols <= 256 ? 256 : 512)));
    static constexpr int kBarrierBytes = 512;                // mbarriers, TMEM slot, flags, tile-index ring
    // Epilogue staging: a tile is kEpiCols accumulator columns (rows of C) x 32 tokens.  Every
    // epilogue warp owns a ring of kEpiBufs tiles: as many as fit beside the stage ring (the
    // operand stream comes first: a deeper stage ring gains more than more staging), at most
    // eight.  With more than one tile a warp fills the next tile while earlier TMA stores are
    // still reading theirs.
    static constexpr int kEpiCols = bcsr_epi_cols(B, CS == 2, CM != 0);
    static constexpr int kEpiTileBytes = kEpiCols * 32 * CS;
    static constexpr int kEpiRoom = (227 * 1024 - 1024 /*align*/ - kBarrierBytes - STAGES * kStageBytes) / (4 * kEpiTileBytes);
    static constexpr int kEpiBufs = kEpiRoom < 8 ? kEpiRoom : 8;
    static constexpr int kStagingBytes = 4 * kEpiBufs * kEpiTileBytes;
    static constexpr int kSmemBytes = STAGES * kStageBytes + kStagingBytes + 1024 /*align*/ + kBarrierBytes;
    static_assert(kEpiBufs >= 1 && kEpiBufs <= 8, "no room for the epilogue's staging tiles");
    static_assert(kEpiCols <= B && H % kEpiCols == 0, "a staging tile never straddles two block-rows");
    static_assert(2 * kAccCols <= 512, "accumulators exceed TMEM");
    static_assert(kSmemBytes <= 227 * 1024, "stage ring exceeds shared memory");
    static_assert((2 * STAGES + 7 + 8) * 8 + 64 <= kBarrierBytes, "barrier area");
    static_assert(kBps == 1 || (B <= 32 && kKS == 1), "multi-block stages are for the small block sizes");
    static_assert(kKS == 1 || kBB <= 128, "a column slice is at most one 128-byte row piece");
    static_assert(kBB % 32 == 0, "a block row must hold whole K steps");
    static_assert(H == B || (H == 128 && B < 128), "stacked blocks are 128 rows high");
};

// Ring depth for a shape: CAP stages, fewer where they would leave no room for one staging tile
// per epilogue warp.
template <int B, int H, int GROUPS, int CAP, int ES, int CS, int CM>
constexpr int bcsr_fit_stages() {
    using C1 = BcsrCfg<B, H, GROUPS, 1, ES, CS, CM>;
    const int s = (227 * 1024 - 1024 - C1::kBarrierBytes - 4 * C1::kEpiTileBytes) / C1::kStageBytes;
    return s > CAP ? CAP : (s < 2 ? 2 : s);
}

constexpr int kSchedDepth = 4;      // tile indices fetched ahead by the dynamic scheduler

template <int B, int H, int GROUPS, int STAGES, int FMT, int CT, int CM, int DYN>
__global__ void __launch_bounds__(DYN ? 224 : 192, 1)
bcsr_spmm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmB3, const __grid_constant__ CUtensorMap tmC,
                 const __grid_constant__ CUtensorMap tmP, const BcsrParams p) {
    constexpr int ES = FMT == 3 ? 1 : (FMT == 2 ? 4 : 2);
    static_assert(FMT != 2 || (!CT && !DYN && H == B), "TF32: fp32 C, static schedule, no row groups");
    static_assert(H == B || !DYN, "stacked blocks: static schedule only");
    using CElem = typename CType<FMT, CT>::type;
    using Cfg = BcsrCfg<B, H, GROUPS, STAGES, ES, static_cast<int>(sizeof(CElem)), CM>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    // stage ring | staging tiles of the epilogue warps | barriers
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::kStageBytes + Cfg::kStagingBytes);
    // barrier slots: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 5);
    const uint32_t drain_bar = bar0 + 8u * (2 * STAGES + 6);   // abort path: MMAs still in flight
    // dynamic scheduling: ring of fetched tile indices (16-byte answers) with full / empty barriers
    auto schf_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 7 + s); };
    auto sche_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 7 + kSchedDepth + s); };
    const uint32_t sched_resp = (bar0 + 8u * (2 * STAGES + 7 + 2 * kSchedDepth) + 15u) & ~15u;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WaitCtl ctl{abort_flag, p.status, p.wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
        mbar_init(drain_bar, 1);
        if constexpr (DYN) {
            for (int s = 0; s < kSchedDepth; ++s) { mbar_init(schf_bar(s), 1); mbar_init(sche_bar(s), 6); }
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmB3);
        prefetch_tmap(&tmC);
        prefetch_tmap(&tmP);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // the row groups' launch: the launch of the remaining block-rows may begin on the SMs this
    // grid leaves idle (the two write disjoint rows of C)
    if (p.overlap == 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int64_t N = p.N;
    // Static schedule: this CTA's range of the tile list.  Dynamic: tile blockIdx.x, then the
    // indices the scheduler warp obtains; every working warp walks the same sequence.
    int tile_begin = 0, tile_end = 0;
    if constexpr (!DYN) {
        tile_begin = __ldg(p.cta_ptr + blockIdx.x);
        tile_end = __ldg(p.cta_ptr + blockIdx.x + 1);
    }
    // Next tile of this warp's walk; nth = number of tiles it has taken so far.  A tile's record
    // {block-row, token tile, first stored block, end block} is all a role needs to know about
    // it; with the static schedule the following tile's record is requested one tile ahead
    // (*rec_next), so that its latency is not paid between tiles.
    auto next_tile = [&](uint32_t nth, int4* rec, int4* rec_next, bool* ok) -> bool {
        if constexpr (!DYN) {
            const int ti = tile_begin + static_cast<int>(nth);
            if (ti >= tile_end) return false;
            *rec = nth == 0 ? __ldg(p.tiles + ti) : *rec_next;
            if (ti + 1 < tile_end) *rec_next = __ldg(p.tiles + ti + 1);
            return true;
        } else {
            int ti_dyn;
            int* ti = &ti_dyn;
            if (nth == 0) { *rec = __ldg(p.tiles + blockIdx.x); return true; }
            // fetched tile nth is entry nth - 1 of the ring
            const int slot = (nth - 1u) % kSchedDepth;
            const uint32_t use = (nth - 1u) / kSchedDepth;
            if (!__all_sync(0xffffffffu, mbar_wait(schf_bar(slot), use & 1u, ctl, 5))) { *ok = false; return false; }
            uint32_t x;
            const bool valid = clc_query(sched_resp + 16u * slot, &x);
            fence_proxy_async_smem();           // the slot is rewritten by the asynchronous proxy later
            __syncwarp();
            if (lane == 0) mbar_arrive(sche_bar(slot));
            if (valid && x >= gridDim.x) {
                // cannot happen with a well-formed answer; recorded instead of trusted
                if (lane == 0 && atomicCAS(p.status, 0, 2) == 0) { p.status[1] = 8; p.status[2] = static_cast<int>(x); }
                *ok = false;
                return false;
            }
            *ti = static_cast<int>(x);
            if (valid) *rec = __ldg(p.tiles + *ti);
            return valid;
        }
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // A warp serialises the TMA requests of its lanes (~60 cycles each) but needs far
        // longer for requests issued one after the other by a single thread, so the loads of
        // a stage are spread over the lanes: lane x < nbox fetches B box x, lanes 8 / 9 the
        // A block (two halves when b = 128).  Lane 0 posts the stage's byte count first.
        {
            uint32_t it = 0;
            bool ok = true;
            // A blocks and the B slab are re-read by other CTAs while the slab lasts: ask L2 to
            // keep them in preference to the C lines streaming through
            const uint64_t keep = l2_policy_evict_last();
            int4 tcd, tcd_next;
            int Jl_next = 0;                 // block columns of the next tile's first 32 blocks, fetched a tile ahead
            bool have_next = false;
            for (uint32_t nth = 0; ok && next_tile(nth, &tcd, &tcd_next, &ok); ++nth) {
                const int n0 = tcd.y * Cfg::kBnT;
                const int nvalid = static_cast<int>(min_i64(Cfg::kBnT, N - n0));
                const int nbox = (nvalid + Cfg::kTokBox - 1) / Cfg::kTokBox;
                const bool whole_tile = p.use_3d && nvalid == Cfg::kBnT;
                const int pb = tcd.z, pe = tcd.w;
                const int Jl_first = have_next ? Jl_next : ((pb + lane < pe) ? __ldg(p.block_col_idx + pb + lane) : 0);
                if constexpr (!DYN) {
                    // the record of the following tile was requested when this one was taken
                    have_next = tile_begin + static_cast<int>(nth) + 1 < tile_end;
                    if (have_next) Jl_next = (tcd_next.z + lane < tcd_next.w) ? __ldg(p.block_col_idx + tcd_next.z + lane) : 0;
                }
                for (int q0 = pb; q0 < pe && ok; q0 += 32) {
                    // block columns of up to 32 stored blocks with one coalesced load
                    const int Jl = q0 == pb ? Jl_first : ((q0 + lane < pe) ? __ldg(p.block_col_idx + q0 + lane) : 0);
                    const int nq = min(32, pe - q0);
                    for (int jq = 0; jq < nq && ok; jq += Cfg::kBps)
#pragma unroll 1
                    for (int kp = 0; kp < Cfg::kKS; ++kp, ++it) {       // column slices of the block (1 unless TF32, b >= 64)
                        const int q = q0 + jq;
                        const int kx = kp * Cfg::kKB;                    // first column of A / first row of B of this unit
                        const int nb = min(Cfg::kBps, nq - jq);          // stored blocks in this stage
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1u;
                        if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(s), ph ^ 1u, ctl, 1))) { ok = false; break; }
                        const uint32_t sb = smem_base + s * Cfg::kStageBytes;
                        // the A request always brings kBps blocks (the box of the tensor map)
                        const uint32_t dense_tx = CM ? (whole_tile ? Cfg::kDenseBytes : ((nvalid + 127) >> 7) * (128 * Cfg::kBB))
                                                     : nbox * Cfg::kBoxBytes;
                        // (stacked blocks: one request per block, a box holds at most 256 rows)
                        if (lane == 0) mbar_arrive_expect_tx(full_bar(s), (H == B ? Cfg::kBps : nb) * Cfg::kABytes + nb * dense_tx);
                        __syncwarp();
                        if constexpr (CM) {
                            // X as [N / 128][128][k]: box = GROUPS x 128 tokens x min(b, 64) elements
                            // of block column J (b = 128: lanes nb.. fetch the second K half)
                            constexpr int kHalves = Cfg::kBB > 128 ? 2 : 1;
                            const int blk = lane % Cfg::kBps, hf = lane / Cfg::kBps;
                            const int J = __shfl_sync(0xffffffffu, Jl, jq + (blk < nb ? blk : 0));
                            if (whole_tile) {
                                if (blk < nb && hf < kHalves)
                                    tma_load_3d_hint(sb + blk * Cfg::kDenseBytes + hf * (GROUPS * Cfg::kXGroupBytes), &tmB3,
                                                     full_bar(s), J * B + kx + hf * (128 / ES), 0, n0 >> 7, keep);
                            } else {
                                // ragged tile: one request per 128-token group, rows >= N are zero filled
                                const int ngrp = (nvalid + 127) >> 7;
                                for (int g = 0; g < ngrp; ++g)
                                    if (blk < nb && hf < kHalves)
                                        tma_load_2d_hint(sb + blk * Cfg::kDenseBytes + hf * (GROUPS * Cfg::kXGroupBytes) + g * Cfg::kXGroupBytes,
                                                         &tmB, full_bar(s), J * B + kx + hf * (128 / ES), n0 + g * 128, keep);
                            }
                        } else
                        if (whole_tile) {
                            // all boxes of a unit with one request: B seen as [token box][k][128 bytes of
                            // tokens], box = kNBox x kKB x 128 bytes; lane i takes block i
                            const int J = __shfl_sync(0xffffffffu, Jl, jq + (lane < nb ? lane : 0));
                            if (lane < nb) tma_load_3d_hint(sb + lane * Cfg::kDenseBytes, &tmB3, full_bar(s), 0, J * B + kx, n0 / Cfg::kTokBox, keep);
                        } else {
                            for (int i = 0; i < nb; ++i) {
                                const int J = __shfl_sync(0xffffffffu, Jl, jq + i);
                                if (lane < nbox)
                                    tma_load_2d_hint(sb + i * Cfg::kDenseBytes + lane * Cfg::kBoxBytes, &tmB, full_bar(s),
                                                     n0 + lane * Cfg::kTokBox, J * B + kx, keep);
                            }
                        }
                        if constexpr (H == B) {
                            if (lane == 8) {
                                tma_load_2d_hint(sb + Cfg::kAOff, &tmA, full_bar(s), kx, q * B, keep);
                            } else if (Cfg::kBB > 128 && lane == 9) {
                                tma_load_2d_hint(sb + Cfg::kAOff + B * 128, &tmA, full_bar(s), 128 / ES, q * B, keep);
                            }
                        } else {
                            if (lane >= 8 && lane < 8 + nb)
                                tma_load_2d_hint(sb + Cfg::kAOff + (lane - 8) * Cfg::kABytes, &tmA, full_bar(s), 0, (q + lane - 8) * H, keep);
                        }
                    }
                }
            }
            if (!ok && lane == 0) {
                // leave no bulk copy in flight: wait (bounded) for the fills already issued
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j)
                    if (!mbar_drain_wait(full_bar(j % STAGES), (j / STAGES) & 1u, ctl, 21)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Warp-uniform control flow (all lanes wait and compute the uniform descriptors); one
        // elected lane issues the tcgen05 instructions.
        {
            // 8-bit floats: format code 0 = E4M3 in both operand fields
            constexpr uint32_t idesc = make_idesc(FMT == 3 ? 0 : FMT, 128, H, CM ? 0 : 1, 0);
            // row-major B: the token tile is MN-major; 4-byte elements need the 128-byte swizzle with
            // 32-byte atoms (a pattern of 4 k-rows), 2-byte elements the plain one (8 k-rows)
            const uint64_t adesc0 = CM ? make_smem_desc(0, 16, 8 * Cfg::kXRowBytes, Cfg::kASwizzle)
                                       : make_smem_desc(0, Cfg::kBoxBytes, ES == 4 ? 512 : 1024, ES == 4 ? SWZ_128B_BASE32B : SWZ_128B);
            constexpr int kStepBytes = (32 / ES) * 128;     // k-rows of one MMA x 128 bytes (row-major token tile)
            const uint64_t bdesc0 = make_smem_desc(0, 16, 8 * Cfg::kARowBytes, Cfg::kASwizzle);
            const bool leader = elect_one();
            uint32_t it = 0, tile_i = 0;
            bool ok = true;
            int4 tcd, tcd_next;
            for (; ok && next_tile(tile_i, &tcd, &tcd_next, &ok); ++tile_i) {
                const int n0 = tcd.y * Cfg::kBnT;
                const int nvalid = static_cast<int>(min_i64(Cfg::kBnT, N - n0));
                const int ngrp = (nvalid + 127) >> 7;
                const int acc = tile_i & 1;
                const uint32_t aph = (tile_i >> 1) & 1u;
                if (!__all_sync(0xffffffffu, mbar_wait(acce_bar(acc), aph ^ 1u, ctl, 2))) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d0 = tmem_base + acc * Cfg::kAccCols;
                const int pb = tcd.z, pe = tcd.w;
                for (int q = pb; q < pe && ok; q += Cfg::kBps)
#pragma unroll 1
                for (int kp = 0; kp < Cfg::kKS; ++kp, ++it) {
                    // stages never straddle the producer's 32-block windows (kBps divides 32)
                    const int nb = min(Cfg::kBps, min(pe - q, 32 - ((q - pb) & 31)));
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!__all_sync(0xffffffffu, mbar_wait(full_bar(s), ph, ctl, 3))) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sb = smem_base + s * Cfg::kStageBytes;
#pragma unroll
                    for (int i = 0; i < Cfg::kBps; ++i) {
                        if (i < nb) {
                            // descriptors differ only in their start-address field (bytes >> 4)
                            const uint64_t a0 = adesc0 + ((sb + i * Cfg::kDenseBytes) >> 4);
                            const uint64_t b0 = bdesc0 + ((sb + Cfg::kAOff + i * Cfg::kABytes) >> 4);
                            const uint32_t accum0 = (q > pb || i > 0 || kp > 0) ? 1u : 0u;
#pragma unroll
                            for (int ks = 0; ks < Cfg::kKSteps; ++ks) {
                                const uint32_t boff = Cfg::kBB <= 128 ? ks * 32 : (ks >> 2) * (B * 128) + (ks & 3) * 32;
#pragma unroll
                                for (int g = 0; g < GROUPS; ++g)
                                    if (leader && g < ngrp)
                                        umma_kind<FMT == 3 ? 2 : (FMT == 2 ? 1 : 0)>(d0 + g * H,
                                                       a0 + ((CM ? (Cfg::kBB <= 128 ? g * Cfg::kXGroupBytes + ks * 32
                                                                            : (ks >> 2) * (GROUPS * Cfg::kXGroupBytes) + g * Cfg::kXGroupBytes + (ks & 3) * 32)
                                                                 : g * (Cfg::kNBox / GROUPS) * Cfg::kBoxBytes + ks * kStepBytes) >> 4),
                                                       b0 + (boff >> 4), idesc, ks > 0 ? 1u : accum0);
                            }
                        }
                    }
                    if (leader) tc_commit(empty_bar(s));
                }
                if (!ok) break;
                if (leader) {
                    if (pe > pb) tc_commit(accf_bar(acc));
                    else mbar_arrive(accf_bar(acc));
                }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue warps
        const int qd = warp & 3;                    // TMEM lane quarter this warp may read
        uint32_t tile_i = 0;
        uint32_t chunk = 0;                         // staging tiles this warp has filled so far
        const uint32_t stg0 = smem_base + STAGES * Cfg::kStageBytes + (warp - 2) * (Cfg::kEpiBufs * Cfg::kEpiTileBytes);
        bool ok = true;
        int4 tcd, tcd_next;
        for (; ok && next_tile(tile_i, &tcd, &tcd_next, &ok); ++tile_i) {
            const int tI = tcd.x;
            const int n0 = tcd.y * Cfg::kBnT;
            const int nvalid = static_cast<int>(min_i64(Cfg::kBnT, N - n0));
            const int ngrp = (nvalid + 127) >> 7;
            const int acc = tile_i & 1;
            const uint32_t aph = (tile_i >> 1) & 1u;
            const bool has_blocks = tcd.w > tcd.z;
            // stacked blocks: the block-rows the group's 128 accumulator columns belong to
            int member = 0;
            if constexpr (H != B) member = lane < H / B ? __ldg(p.stack_rows + tI * (H / B) + lane) : 0;
            if (!__all_sync(0xffffffffu, mbar_wait(accf_bar(acc), aph, ctl, 4))) { ok = false; break; }
            tc_fence_after_sync();
            // K-split: a tile of one part of a long block-row (record x = -1 - slot) writes its fp32
            // partial tile, rows slot * b .. of the partial array, instead of C (fp32 row-major C only)
            const bool part = tI < 0;
            const int64_t row0 = static_cast<int64_t>(part ? -1 - tI : tI) * B;
            const CUtensorMap* tm_out = part ? &tmP : &tmC;
            constexpr int W = Cfg::kEpiCols;                // accumulator columns per staging tile
            for (int g = 0; g < ngrp; ++g) {
                const int nw = n0 + g * 128 + qd * 32;          // first token of this warp
                if (nw >= N) break;                             // the whole warp is beyond the last token
#pragma unroll 1
                for (int c0 = 0; c0 < H; c0 += W) {
                    uint32_t v[W];
                    if (has_blocks) {
                        const uint32_t ta = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) +
                                            acc * Cfg::kAccCols + g * H + c0;
                        tmem_ld_cols<W>(ta, v);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int j = 0; j < W; ++j) v[j] = 0u;
                    }
                    // registers -> the next tile of this warp's staging ring -> one TMA store.  The
                    // store that used this tile kEpiBufs chunks ago must have read it first.
                    const uint32_t stg = stg0 + (chunk % Cfg::kEpiBufs) * Cfg::kEpiTileBytes;
                    ++chunk;
                    if (lane == 0) bulk_wait_read<Cfg::kEpiBufs - 1>();
                    __syncwarp();
                    if constexpr (!CM) {
                        // tile [W rows][32 tokens], no swizzle: 128-byte rows of fp32 (64-byte rows
                        // of 2-byte elements); a warp's store covers one row, so no bank is hit twice
#pragma unroll
                        for (int j = 0; j < W; ++j) {
                            if constexpr (sizeof(CElem) == 4) {
                                st_shared_u32(stg + j * 128 + lane * 4, v[j]);
                            } else {
                                const CElem h = from_f32<CElem>(__uint_as_float(v[j]));
                                st_shared_u16(stg + j * 64 + lane * 2, *reinterpret_cast<const unsigned short*>(&h));
                            }
                        }
                    } else {
                        // tile [32 tokens][W elements]: this lane's row, in 16-byte chunks; 64-byte
                        // rows are stored with the tensor map's 64-byte swizzle (chunk index XOR
                        // (row / 2) % 4), which also keeps the warp's stores off each other's banks
                        constexpr int kChunks = W * static_cast<int>(sizeof(CElem)) / 16;     // 2 or 4
                        constexpr int kPer = 16 / static_cast<int>(sizeof(CElem));            // elements per chunk
#pragma unroll
                        for (int c = 0; c < kChunks; ++c) {
                            uint32_t w4[4];
                            if constexpr (sizeof(CElem) == 4) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) w4[i] = v[c * kPer + i];
                            } else {
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const CElem lo = from_f32<CElem>(__uint_as_float(v[c * kPer + 2 * i]));
                                    const CElem hi = from_f32<CElem>(__uint_as_float(v[c * kPer + 2 * i + 1]));
                                    w4[i] = static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(&lo)) |
                                            (static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(&hi)) << 16);
                                }
                            }
                            const int cs = kChunks == 4 ? (c ^ ((lane >> 1) & 3)) : c;
                            st_shared_v4(stg + lane * (kChunks * 16) + (cs << 4), w4[0], w4[1], w4[2], w4[3]);
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    int32_t crow = static_cast<int32_t>(row0) + c0;
                    if constexpr (H != B) crow = __shfl_sync(0xffffffffu, member, c0 / B) * B + (c0 % B);
                    if (lane == 0) {
                        // row-major: box = 32 tokens x W rows at (token, row); column-major: box =
                        // W columns x 32 tokens at (column, token).  Out-of-range parts are clipped.
                        if constexpr (!CM) tma_store_2d(tm_out, stg, nw, crow);
                        else tma_store_2d(tm_out, stg, crow, nw);
                        bulk_commit_group();
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(acc));
        }
        if (lane == 0) bulk_wait_all<false>();          // this warp's last stores have landed
    }

    if constexpr (DYN) {
        if (warp == 6 && lane == 0) {
            // -------------------------------------------------------------- tile scheduler
            // One request at a time (a request after a failed one is not allowed), up to
            // kSchedDepth tiles ahead of the slowest working warp.
            for (uint32_t r = 0;; ++r) {             // ring entry r = the CTA's tile r + 1
                const int slot = r % kSchedDepth;
                const uint32_t use = r / kSchedDepth;
                if (use > 0 && !mbar_wait(sche_bar(slot), (use - 1u) & 1u, ctl, 6)) break;
                mbar_arrive_expect_tx(schf_bar(slot), 16);
                clc_try_cancel(sched_resp + 16u * slot, schf_bar(slot));
                if (!mbar_wait(schf_bar(slot), use & 1u, ctl, 7)) {
                    // leaving early: the answer of the request just issued must still land in
                    // this CTA's shared memory before the CTA may exit (bounded)
                    mbar_drain_wait(schf_bar(slot), use & 1u, ctl, 22);
                    break;
                }
                uint32_t x;
                if (!clc_query(sched_resp + 16u * slot, &x)) break;      // no CTA left to cancel: the walk ends
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    // launched while the previous grid of the stream was still running: do not finish before it
    if (p.overlap == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (warp == 1) {
        if (*abort_flag) {
            // abort path: let the MMAs this warp's elected lane already issued finish before
            // TMEM is freed (kept out of the role loop above on purpose: placed there it
            // slowed the normal path measurably)
            if (elect_one()) {
                tc_commit(drain_bar);
                mbar_drain_wait(drain_bar, 0, ctl, 23);
            }
            __syncwarp();
        }
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// CAP = the deepest ring the shape is given; the ring actually used also leaves room for the
// epilogue's staging tiles (bcsr_fit_stages).
template <int B, int H, int GROUPS, int CAP, int FMT, int CT, int CM, int DYN>
cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p,
                       int grid, cudaStream_t stream) {
    constexpr int ES = FMT == 3 ? 1 : (FMT == 2 ? 4 : 2);
    constexpr int CS = static_cast<int>(sizeof(typename CType<FMT, CT>::type));
    constexpr int STAGES = bcsr_fit_stages<B, H, GROUPS, CAP, ES, CS, CM>();
    using Cfg = BcsrCfg<B, H, GROUPS, STAGES, ES, CS, CM>;
    auto kfn = bcsr_spmm_kernel<B, H, GROUPS, STAGES, FMT, CT, CM, DYN>;
    // the attribute belongs to the (function, device) pair: set it once per device
    static std::mutex mu;
    static bool attr_done[kMaxDevices] = {};
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu);
        if (!attr_done[dev]) {
            e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
            if (e != cudaSuccess) return e;
            attr_done[dev] = true;
        }
    }
    if (p.overlap == 2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(grid));
        cfg.blockDim = dim3(DYN ? 224 : 192);
        cfg.dynamicSmemBytes = Cfg::kSmemBytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kfn, tmA, tmB, tmB3, tmC, tmP, p);
    }
    kfn<<<grid, DYN ? 224 : 192, Cfg::kSmemBytes, stream>>>(tmA, tmB, tmB3, tmC, tmP, p);
    return cudaGetLastError();
}

template <int FMT, int CT, int CM, int DYN>
cudaError_t launch_shape(int b, int groups, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3,
                         const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    switch (b * 10 + groups) {
        case 161: return launch_one<16, 16, 1, 10, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 162: return launch_one<16, 16, 2, 5, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 164: return launch_one<16, 16, 4, 3, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 321: return launch_one<32, 32, 1, 10, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 322: return launch_one<32, 32, 2, 5, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 324: return launch_one<32, 32, 4, 3, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 641: return launch_one<64, 64, 1, 8, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 642: return launch_one<64, 64, 2, 5, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 644: return launch_one<64, 64, 4, 3, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1281: return launch_one<128, 128, 1, 3, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1282: return launch_one<128, 128, 2, 2, FMT, CT, CM, DYN>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        default: return cudaErrorInvalidValue;
    }
}

// Stacked blocks (row groups): 128 rows x b, token tile 256, four stages of 48 KB.
template <int FMT, int CT, int CM>
cudaError_t launch_stack_shape(int b, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3,
                               const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    switch (b) {
        case 16: return launch_one<16, 128, 2, 4, FMT, CT, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 32: return launch_one<32, 128, 2, 4, FMT, CT, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 64: return launch_one<64, 128, 2, 4, FMT, CT, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        default: return cudaErrorInvalidValue;
    }
}

template <int FMT>
cudaError_t launch_stack_fmt(int b, int c16, int cm, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3,
                             const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    if (cm) return c16 ? launch_stack_shape<FMT, 1, 1>(b, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
                       : launch_stack_shape<FMT, 0, 1>(b, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    return c16 ? launch_stack_shape<FMT, 1, 0>(b, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
               : launch_stack_shape<FMT, 0, 0>(b, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
}

// E4M3 inputs: fp32 C, static schedule; b = 32, 64 or 128 (a block row must hold at least one
// 32-element K step).  Stages are half the bytes of the 16-bit ones.
template <int CM>
cudaError_t launch_fp8(int b, int groups, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3,
                       const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    switch (b * 10 + groups) {
        case 321: return launch_one<32, 32, 1, 10, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 322: return launch_one<32, 32, 2, 10, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 324: return launch_one<32, 32, 4, 6, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 641: return launch_one<64, 64, 1, 10, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 642: return launch_one<64, 64, 2, 10, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 644: return launch_one<64, 64, 4, 5, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1281: return launch_one<128, 128, 1, 6, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1282: return launch_one<128, 128, 2, 4, 3, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        default: return cudaErrorInvalidValue;
    }
}

// TF32 (fp32 storage): fp32 C, static schedule; the deepest rings the stage sizes allow.
template <int CM>
cudaError_t launch_tf32(int b, int groups, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB3,
                        const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    switch (b * 10 + groups) {
        case 161: return launch_one<16, 16, 1, 5, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 162: return launch_one<16, 16, 2, 3, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 321: return launch_one<32, 32, 1, 5, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 322: return launch_one<32, 32, 2, 3, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 641: return launch_one<64, 64, 1, 8, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 642: return launch_one<64, 64, 2, 5, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 644: return launch_one<64, 64, 4, 3, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1281: return launch_one<128, 128, 1, 6, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        case 1282: return launch_one<128, 128, 2, 4, 2, 0, CM, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        default: return cudaErrorInvalidValue;
    }
}

template <int FMT>
cudaError_t launch_fmt(int b, int groups, int c16, int cm, int dyn, const CUtensorMap& tmA, const CUtensorMap& tmB,
                       const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid, cudaStream_t stream) {
    // dynamic scheduling is built for the default output (fp32, row-major) only
    if (dyn) return (c16 || cm) ? cudaErrorInvalidValue : launch_shape<FMT, 0, 0, 1>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    if (cm) return c16 ? launch_shape<FMT, 1, 1, 0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
                       : launch_shape<FMT, 0, 1, 0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    return c16 ? launch_shape<FMT, 1, 0, 0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
               : launch_shape<FMT, 0, 0, 0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
}

}  // namespace

// Widest token tile per block size, in 128-token groups.  b = 64 with row-major fp32 C writes
// the most bytes of C per staged operand byte: there a 256-token tile with five 40 KB stages and
// three staging tiles per epilogue warp measured 3 % faster than 512 tokens with three 72 KB
// stages and one staging tile; every other combination measured equal or slower with 256.
// TF32: elements are twice as wide, so b = 16 / 32 stop at 256 tokens (a 512-token stage of
// several blocks would not fit twice).
int bcsr_token_groups_max(int dtype, int b, int c16, int col_major) {
    if (b == 128) return 2;
    if (dtype == 2 && b <= 32) return 2;
    return (b == 64 && !c16 && !col_major) ? 2 : 4;
}

cudaError_t launch_bcsr(int dtype, int b, int groups, int c16, int col_major, int dynamic, const CUtensorMap& tmA,
                        const CUtensorMap& tmB, const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p,
                        int grid, cudaStream_t stream) {
    if (dtype == 1) return launch_fmt<0>(b, groups, c16, col_major, dynamic, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);   // fp16
    if (dtype == 0) return launch_fmt<1>(b, groups, c16, col_major, dynamic, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);   // bf16
    if (dtype == 3) {
        if (c16 || dynamic) return cudaErrorInvalidValue;
        return col_major ? launch_fp8<1>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
                         : launch_fp8<0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    }
    if (dtype == 2) {
        if (c16 || dynamic) return cudaErrorInvalidValue;
        return col_major ? launch_tf32<1>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream)
                         : launch_tf32<0>(b, groups, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_bcsr_stacked(int dtype, int b, int c16, int col_major, const CUtensorMap& tmA, const CUtensorMap& tmB,
                                const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p, int grid,
                                cudaStream_t stream) {
    if (dtype == 1) return launch_stack_fmt<0>(b, c16, col_major, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);   // fp16
    if (dtype == 0) return launch_stack_fmt<1>(b, c16, col_major, tmA, tmB, tmB3, tmC, tmP, p, grid, stream);   // bf16
    if (dtype == 3 && !c16 && col_major) {
        // E4M3: half the bytes per stage, twice the ring depth
        if (b == 32) return launch_one<32, 128, 2, 8, 3, 0, 1, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
        if (b == 64) return launch_one<64, 128, 2, 8, 3, 0, 1, 0>(tmA, tmB, tmB3, tmC, tmP, p, grid, stream);
    }
    return cudaErrorInvalidValue;
}

namespace {

// One CTA per (split block-row, run of 1024 four-column pieces of its b x N output); a thread sums
// four pieces over the parts, in part order (run-to-run identical results), all loads of a
// piece in flight together.
constexpr int kMergePieces = 4;
__global__ void __launch_bounds__(256) bcsr_merge_kernel(const BcsrMergeParams p) {
    const int i = blockIdx.x;
    const int I = p.row[i], first = p.first[i], nparts = p.nparts[i];
    // the partial tiles belong to the SpMM kernel launched just before on the same stream
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t N = p.N, n4 = N >> 2;                 // N is a multiple of 4 (16-byte rows)
    const int64_t row0 = static_cast<int64_t>(I) * p.b;
    const int64_t rows = min_i64(p.b, p.m - row0);
    const int64_t total = rows * n4;
    const float4* part = reinterpret_cast<const float4*>(p.partial) + static_cast<int64_t>(first) * p.b * n4;
    float4* out = reinterpret_cast<float4*>(p.C + row0 * N);
    const int64_t slot_stride = static_cast<int64_t>(p.b) * n4;
    const int64_t e0 = static_cast<int64_t>(blockIdx.y) * (256 * kMergePieces) + threadIdx.x;
    float4 acc[kMergePieces];
#pragma unroll
    for (int k = 0; k < kMergePieces; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nparts; ++s) {
#pragma unroll
        for (int k = 0; k < kMergePieces; ++k) {
            const int64_t e = e0 + k * 256;
            if (e < total) {
                const float4 v = __ldg(part + s * slot_stride + e);
                acc[k].x += v.x; acc[k].y += v.y; acc[k].z += v.z; acc[k].w += v.w;
            }
        }
    }
#pragma unroll
    for (int k = 0; k < kMergePieces; ++k) {
        const int64_t e = e0 + k * 256;
        if (e < total) out[e] = acc[k];
    }
}

}  // namespace

cudaError_t launch_bcsr_merge(const BcsrMergeParams& p, cudaStream_t stream) {
    if (p.n <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    const int64_t pieces = static_cast<int64_t>(p.b) * (p.N >> 2);
    cfg.gridDim = dim3(static_cast<unsigned>(p.n), static_cast<unsigned>((pieces + 256 * kMergePieces - 1) / (256 * kMergePieces)));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, bcsr_merge_kernel, p);
}

}  // namespace spmm
