// WCSR SpMM kernel for sm_100a (Sec. 3.2 - 3.3 of the paper, re-designed for Blackwell).
//
// Work item: one sub-task of the split plan (a run of `count` condensed columns of one
// 16-row window) times one tile of 128 columns of B ("tokens"; wider B: one pass per tile).  It accumulates
//     D[n, r] += sum_q  B[window_col_idx[q], n0 + n] * values[r, q]
// with the tokens on the 128 TMEM lanes (MMA M side; the gathered B rows are written to
// shared memory in the MN-major 128-byte-swizzled layout tcgen05.mma reads) and the 16
// window rows as the MMA N side (operand = the packed window tile, K-major, un-swizzled).
//
// Roles (PW + 5 warps, persistent CTAs, two or three resident per SM):
//   warps 0..PW-1     gather producers: warp w owns the CTA's fills w, w + PW, ...; per fill
//               every lane reads four column indices and issues one TMA row-gather (four B
//               rows x 128 bytes, hardware swizzle, zero fill for -1 pads) into a STAGES-deep
//               ring; lane 0 also bulk-copies the contiguous packed A tile.  Completion is
//               counted in bytes on the stage's mbarrier, so producers never wait for data.
//   warp PW           MMA issuer (one elected lane): count / b_col tcgen05.mma per stage.
//   warps PW+1..PW+4  epilogue: tcgen05.ld, release the TMEM buffer, store to C (unsplit
//               window) or to the task's partial tile (split window).
// Tasks are dealt to bins by the longest-processing-time rule at creation; CTA c walks bins
// c, c + grid, ...; inside a bin tasks ascend, so all CTAs sweep the matrix top to bottom
// together and neighbouring windows (which share B rows in banded matrices) meet in L2.
// Split windows are summed in slot order by wcsr_merge_kernel, which also zero-fills the C
// rows of empty windows: results are run-to-run identical.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"

namespace spmm {

namespace {

// All K steps of an item accumulate into one 128 x 16 TMEM tile.  (Rotating them over several
// partial accumulators that the epilogue adds was built and measured 4 - 7 % slower: the
// tensor pipe takes a 128 x 16 MMA every 39 cycles whether or not it depends on the previous
// one, and the extra TMEM loads lengthen the epilogue.)

template <int ES, int WH, int KT, int STAGES, bool NARROW = false>
struct WcsrCfg {
    static constexpr int kWH = WH;                          // window height = MMA N
    static constexpr int kKStep = 32 / ES;                  // columns per MMA (= b_col)
    static constexpr int kBnT = 128;                        // tokens per tile = TMEM lanes
    // 128-byte segments per gathered row: all 128 tokens, or (narrow: N <= 64, 2-byte types) one
    static constexpr int kSegs = NARROW ? 1 : kBnT * ES / 128;
    static constexpr int kRowBytes = kSegs * 128;
    static constexpr int kGathers = (KT / 4) * kSegs;       // row-gather instructions per full fill
    static constexpr int kRounds = (kGathers + 31) / 32;    // per lane
    static constexpr int kAtomStride = KT * 128;            // bytes between MN atoms
    static constexpr int kDenseBytes = KT * kRowBytes;
    static constexpr int kABytes = (KT / kKStep) * (kWH * 32);
    static constexpr int kStageBytes = kDenseBytes + kABytes;
    // resident CTAs per SM = bins per SM of the schedule; they must fit the SM's shared memory
    // (1 KB per CTA is reserved by the system) and share its 512 TMEM columns
    static constexpr int kCtasPerSm = wcsr_bins_per_sm(ES, WH);
    static_assert(kCtasPerSm * (STAGES * kStageBytes + 1024 + 256 + 1024) <= 227 * 1024, "shared memory over-subscribed");
    // items with live accumulators
    static constexpr int kNAcc = 4;                         // items with live accumulators
    static constexpr int kAccCols = kWH;                    // TMEM columns of one item
    static constexpr int kTmemCols = kNAcc * kAccCols;      // 64 or 256
    static constexpr int kSmemBytes = STAGES * kStageBytes + 1024 + 256;
    static_assert(KT % 8 == 0 && KT % kKStep == 0 && KT <= 128, "stage shape");
    static_assert(kGathers <= 32, "one gather instruction per lane and fill");
    static_assert(!NARROW || (ES == 2 && WH == 16), "narrow variant: 2-byte types, window height 16");
    static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

// Every role of a CTA walks the same sequence of segments: bins blockIdx.x, +grid, ...; per
// bin one segment per token tile.  A segment is a contiguous range of the (bin-major) fill
// and item arrays, so descriptors are fetched 32 at a time with one coalesced load and
// handed out with warp shuffles.
struct SegIter {
    int b, tt;
    __device__ __forceinline__ void init() { b = blockIdx.x; tt = -1; }
    // advance to the next segment; false when the CTA has no more work
    __device__ __forceinline__ bool next(const WcsrParams& p) {
        if (b >= p.n_bins) return false;
        if (++tt >= p.n_tt) {
            tt = 0;
            b += gridDim.x;
        }
        return b < p.n_bins;
    }
};

// LSU = true: the gathered rows reach shared memory through the load/store units instead of
// TMA -- the cooperative gather with 128-bit loads that Sec. 3.2 describes, here as 16-byte
// cp.async copies that every lane of the producer warp places at the swizzled position the MMA
// expects.  Kept as a selectable variant so that the two gathers can be measured side by side.
template <int ES, int FMT, int WH, int KT, int STAGES, int PW, int CT, bool NARROW, bool LSU = false>
__global__ void __launch_bounds__((PW + 5) * 32, WcsrCfg<ES, WH, KT, STAGES, NARROW>::kCtasPerSm)
wcsr_spmm_kernel(const __grid_constant__ CUtensorMap tmB, const WcsrParams p) {
    using Cfg = WcsrCfg<ES, WH, KT, STAGES, NARROW>;
    constexpr int kWH = WH;
    constexpr int kProducerWarps = PW;          // warps 0 .. PW-1; MMA warp PW; epilogue PW+1 .. PW+4
    constexpr int kMmaWarp = PW;
    // Fill i goes to stage i % STAGES and is produced by warp i % PW.  With STAGES a multiple
    // of PW every stage is always refilled by the same warp, which therefore sees each of its
    // releases in turn: the parity wait on the empty barrier is exact.
    static_assert(STAGES % PW == 0, "every stage must belong to one producer warp");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    static_assert((2 * STAGES + 2 * Cfg::kNAcc + 3) * 8 <= 256, "barrier area is 256 bytes");
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::kStageBytes);
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + Cfg::kNAcc + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 2 * Cfg::kNAcc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 2 * Cfg::kNAcc + 1);
    const uint32_t drain_bar = bar0 + 8u * (2 * STAGES + 2 * Cfg::kNAcc + 2);   // abort path: MMAs still in flight

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WaitCtl ctl{abort_flag, p.status, p.wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < Cfg::kNAcc; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmB);
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // The merge kernel is launched as a programmatic dependent: let its CTAs be scheduled (and
    // fetch their lists) while this grid runs; they block in griddepcontrol.wait until this
    // grid has completed and its writes are visible.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const int64_t N = p.N;
    const int2 kNoDesc = make_int2(0, 0);

    if (LSU && warp < kProducerWarps) {
        // ------------------------------------------------------------------ gather producers, load/store-unit variant
        // Same ownership of fills and stages as below.  A gathered row is kCh 16-byte chunks;
        // one warp-wide issue copies 32 chunks (32 / kCh rows), lane -> (row, chunk) fixed.  The
        // A tile still arrives by bulk copy (its bytes are the barrier's transaction count); the
        // warp's own arrival follows the completion of its cp.async copies.
        if constexpr (LSU) {
            constexpr int kCh = Cfg::kRowBytes / 16;              // 16 (2-byte types) or 32 (TF32)
            constexpr int kE16 = 16 / ES;                         // elements per chunk
            constexpr int kRowsPerIssue = 32 / kCh;
            constexpr int kIssues = KT / kRowsPerIssue;
            constexpr int kIdxRegs = (KT + 31) / 32;
            static_assert(kCh <= 32 && 32 % kCh == 0 && !NARROW, "row of at most 512 bytes");
            const int c = lane % kCh;                             // my chunk inside a gathered row
            const int rsub = lane / kCh;                          // my row inside one issue
            const uint8_t* Bp = static_cast<const uint8_t*>(p.B);
            const size_t row_pitch = static_cast<size_t>(N) * ES;
            auto load_idx = [&](const int2 d, int (&idx)[kIdxRegs]) {
                const int cnt = d.y & 0xFFFF;
#pragma unroll
                for (int j = 0; j < kIdxRegs; ++j)
                    idx[j] = (j * 32 + lane < cnt) ? __ldg(p.col_idx + d.x + j * 32 + lane) : -1;
            };
            SegIter seg;
            seg.init();
            uint32_t it0 = 0, last_it = 0;
            uint32_t n_issued = 0;                       // fills this warp has issued
            bool ok = true;
            int idx_cur[kIdxRegs], idx_nxt[kIdxRegs];
            bool idx_ready = false;
            while (ok && seg.next(p)) {
                const int f0 = __ldg(p.bin_fill + seg.b), f1 = __ldg(p.bin_fill + seg.b + 1);
                const int n0 = seg.tt * Cfg::kBnT;
                int2 win = (f0 + lane < f1) ? __ldg(p.fills + f0 + lane) : kNoDesc;
                for (int wbase = f0; wbase < f1 && ok; wbase += 32) {
                    const int2 nwin = (wbase + 32 + lane < f1) ? __ldg(p.fills + wbase + 32 + lane) : kNoDesc;
                    const uint32_t itw = it0 + static_cast<uint32_t>(wbase - f0);
                    int j = static_cast<int>((static_cast<uint32_t>(warp) + kProducerWarps - itw % kProducerWarps) % kProducerWarps);
                    for (; j < 32 && wbase + j < f1; j += kProducerWarps) {
                        const uint32_t it = itw + j;
                        int2 d;
                        d.x = __shfl_sync(0xffffffffu, win.x, j);
                        d.y = __shfl_sync(0xffffffffu, win.y, j);
                        if (!idx_ready) load_idx(d, idx_cur);
                        const int jn = j + kProducerWarps;        // this warp's next fill, if it is in this segment
                        const bool have_n = wbase + jn < f1;
                        int2 dn;
                        dn.x = __shfl_sync(0xffffffffu, jn < 32 ? win.x : nwin.x, jn & 31);
                        dn.y = __shfl_sync(0xffffffffu, jn < 32 ? win.y : nwin.y, jn & 31);
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1u;
                        const int q = d.x;
                        const int cnt = d.y & 0xFFFF;
                        if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(s), ph ^ 1u, ctl, 11))) { ok = false; break; }
                        const uint32_t sb = smem_base + s * Cfg::kStageBytes;
                        if (lane == 0) {
                            const uint32_t abytes = (cnt / Cfg::kKStep) * (kWH * 32);
                            mbar_expect_tx(full_bar(s), abytes);
                            bulk_load_1d(sb + Cfg::kDenseBytes,
                                         p.packed + static_cast<size_t>(q / Cfg::kKStep) * (kWH * 32), abytes, full_bar(s));
                        }
                        ++n_issued;
                        last_it = it;
#pragma unroll
                        for (int i = 0; i < kIssues; ++i) {
                            const int r = i * kRowsPerIssue + rsub;          // column of the fill = row of the stage
                            // (the register that holds row r's index is known at compile time)
                            const int idx = __shfl_sync(0xffffffffu, idx_cur[(i * kRowsPerIssue) >> 5], r & 31);
                            if (r < cnt && n0 + c * kE16 < N) {
                                uint32_t dst = sb + (c >> 3) * Cfg::kAtomStride + r * 128;
                                if constexpr (ES == 2) {
                                    dst += ((c & 7) ^ (r & 7)) << 4;         // 128-byte swizzle: chunk ^= row % 8
                                } else {
                                    // 128-byte swizzle with 32-byte atoms: 32-byte piece ^= row % 4
                                    dst += ((((c & 7) >> 1) ^ (r & 3)) << 5) + ((c & 1) << 4);
                                }
                                const bool valid = idx >= 0;                  // -1 pads: 16 zero bytes, B is not read
                                const uint8_t* src = Bp + (valid ? static_cast<size_t>(idx) * row_pitch +
                                                                       (static_cast<size_t>(n0) + c * kE16) * ES
                                                                 : 0);
                                cp_async_16(dst, src, valid);
                            }
                        }
                        cp_async_commit();
                        if (have_n) load_idx(dn, idx_nxt);
                        cp_async_wait<0>();
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(full_bar(s));
#pragma unroll
                        for (int jj = 0; jj < kIdxRegs; ++jj) idx_cur[jj] = idx_nxt[jj];
                        idx_ready = have_n;
                    }
                    win = nwin;
                }
                it0 += static_cast<uint32_t>(f1 - f0);
            }
            cp_async_wait<0>();
            if (!ok && lane == 0) {
                // abort path: the bulk copies of the fills this warp issued last (one per stage it
                // owns) may still be in flight
                for (uint32_t k = 0; k < static_cast<uint32_t>(STAGES / PW) && k < n_issued; ++k) {
                    const uint32_t j = last_it - k * kProducerWarps;
                    if (!mbar_drain_wait(full_bar(j % STAGES), (j / STAGES) & 1u, ctl, 31)) break;
                }
            }
        }
    } else if (warp < kProducerWarps) {
        // ------------------------------------------------------------------ gather producers
        // Lane l of the owning warp issues gather u = l (+32 per round): row group u / kSegs
        // (rows 4*rg .. 4*rg+3 of the fill), 128-byte segment u % kSegs of those rows.
        // (with gather hints: also the reuse class of the four columns, one byte)
        const bool hints = p.grp_class != nullptr;
        auto load_idx = [&](const int2 d, int4 (&idx)[Cfg::kRounds], int (&cls)[Cfg::kRounds]) {
            const int cnt = d.y & 0xFFFF;
#pragma unroll
            for (int r = 0; r < Cfg::kRounds; ++r) {
                const int rg = (lane + 32 * r) / Cfg::kSegs;
                idx[r] = (rg * 4 < cnt) ? __ldg(reinterpret_cast<const int4*>(p.col_idx + d.x) + rg)
                                        : make_int4(-1, -1, -1, -1);
                cls[r] = (hints && rg * 4 < cnt) ? __ldg(p.grp_class + (d.x >> 2) + rg) : 0;
            }
        };
        // B rows that many windows gather stay in L2 in preference to everything that streams through
        const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();

        SegIter seg;
        seg.init();
        uint32_t it0 = 0;                            // CTA-wide number of fills before this segment
        uint32_t last_it = 0;
        uint32_t n_issued = 0;                       // fills this warp has issued
        bool ok = true;
        // column indices of this warp's current fill and of its next two fills (requested two
        // fills ahead, so their latency never sits in the issue loop)
        int4 idx_cur[Cfg::kRounds], idx_n1[Cfg::kRounds], idx_n2[Cfg::kRounds];
        int cls_cur[Cfg::kRounds], cls_n1[Cfg::kRounds], cls_n2[Cfg::kRounds];
        bool rdy0 = false, rdy1 = false;
        while (ok && seg.next(p)) {
            const int f0 = __ldg(p.bin_fill + seg.b), f1 = __ldg(p.bin_fill + seg.b + 1);
            const int n0 = seg.tt * Cfg::kBnT;
            const int nvalid = static_cast<int>(min_i64(Cfg::kBnT, N - n0));
            const int nseg = (nvalid * ES + 127) >> 7;       // 128-byte segments that hold tokens < N
            int2 win = (f0 + lane < f1) ? __ldg(p.fills + f0 + lane) : kNoDesc;
            for (int wbase = f0; wbase < f1 && ok; wbase += 32) {
                const int2 nwin = (wbase + 32 + lane < f1) ? __ldg(p.fills + wbase + 32 + lane) : kNoDesc;
                const uint32_t itw = it0 + static_cast<uint32_t>(wbase - f0);   // counter of window slot 0
                int j = static_cast<int>((static_cast<uint32_t>(warp) + kProducerWarps - itw % kProducerWarps) % kProducerWarps);
                for (; j < 32 && wbase + j < f1; j += kProducerWarps) {
                    const uint32_t it = itw + j;
                    int2 d;
                    d.x = __shfl_sync(0xffffffffu, win.x, j);
                    d.y = __shfl_sync(0xffffffffu, win.y, j);
                    // this warp's next two fills, if they are in this segment
                    const int j1 = j + kProducerWarps, j2 = j + 2 * kProducerWarps;
                    const bool have1 = wbase + j1 < f1, have2 = wbase + j2 < f1;
                    int2 d1, d2;
                    d1.x = __shfl_sync(0xffffffffu, j1 < 32 ? win.x : nwin.x, j1 & 31);
                    d1.y = __shfl_sync(0xffffffffu, j1 < 32 ? win.y : nwin.y, j1 & 31);
                    d2.x = __shfl_sync(0xffffffffu, j2 < 32 ? win.x : nwin.x, j2 & 31);
                    d2.y = __shfl_sync(0xffffffffu, j2 < 32 ? win.y : nwin.y, j2 & 31);
                    if (!rdy0) load_idx(d, idx_cur, cls_cur);
                    if (have1 && !rdy1) load_idx(d1, idx_n1, cls_n1);
                    if (have2) load_idx(d2, idx_n2, cls_n2);

                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    const int q = d.x;
                    const int cnt = d.y & 0xFFFF;
                    if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(s), ph ^ 1u, ctl, 11))) { ok = false; break; }
                    const uint32_t sb = smem_base + s * Cfg::kStageBytes;
                    if (lane == 0) {
                        const uint32_t abytes = (cnt / Cfg::kKStep) * (kWH * 32);
                        mbar_arrive_expect_tx(full_bar(s), abytes + (cnt / 4) * nseg * 512);
                        const uint8_t* asrc = p.packed + static_cast<size_t>(q / Cfg::kKStep) * (kWH * 32);
                        if (p.hint_flags & 1) bulk_load_1d_hint(sb + Cfg::kDenseBytes, asrc, abytes, full_bar(s), pol_stream);
                        else bulk_load_1d(sb + Cfg::kDenseBytes, asrc, abytes, full_bar(s));
                    }
                    __syncwarp();
                    ++n_issued;
                    last_it = it;
#pragma unroll
                    for (int r = 0; r < Cfg::kRounds; ++r) {
                        const int u = lane + 32 * r;
                        const int rg = u / Cfg::kSegs, sg = u % Cfg::kSegs;
                        if (rg * 4 < cnt && sg < nseg) {
                            if (hints)
                                tma_gather4_2d_hint(sb + sg * Cfg::kAtomStride + rg * 512, &tmB, full_bar(s), n0 + sg * (128 / ES),
                                                    idx_cur[r].x, idx_cur[r].y, idx_cur[r].z, idx_cur[r].w,
                                                    cls_cur[r] >= p.hot_min ? pol_keep : pol_stream);
                            else
                                tma_gather4_2d(sb + sg * Cfg::kAtomStride + rg * 512, &tmB, full_bar(s),
                                               n0 + sg * (128 / ES), idx_cur[r].x, idx_cur[r].y, idx_cur[r].z, idx_cur[r].w);
                        }
                    }
#pragma unroll
                    for (int r = 0; r < Cfg::kRounds; ++r) {
                        idx_cur[r] = idx_n1[r];
                        idx_n1[r] = idx_n2[r];
                        cls_cur[r] = cls_n1[r];
                        cls_n1[r] = cls_n2[r];
                    }
                    rdy0 = have1;
                    rdy1 = have2;
                }
                win = nwin;
            }
            it0 += static_cast<uint32_t>(f1 - f0);
        }
        if (!ok && lane == 0) {
            // abort path: the fills this warp issued last (one per stage it owns) may still be in flight
            for (uint32_t k = 0; k < static_cast<uint32_t>(STAGES / PW) && k < n_issued; ++k) {
                const uint32_t j = last_it - k * kProducerWarps;
                if (!mbar_drain_wait(full_bar(j % STAGES), (j / STAGES) & 1u, ctl, 32)) break;
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the fill list (descriptor windows via shuffles) and waits for
        // stages and accumulators; one elected lane issues the MMAs and commits.
        // (8-bit floats: format code 0 = E4M3 in both operand fields)
        constexpr uint32_t idesc = make_idesc(FMT == 3 ? 0 : FMT, 128, kWH, 1, 0);
        // narrow variant: only the first 64-token atom is staged; the MMA's second atom is made to
        // alias it (atom stride 0) so that no address outside the stage is read; its TMEM lanes
        // (tokens 64..127) are never stored
        const uint64_t adesc0 = make_smem_desc(0, NARROW ? 0 : Cfg::kAtomStride, ES == 4 ? 512 : 1024, ES == 4 ? SWZ_128B_BASE32B : SWZ_128B);
        const uint64_t bdesc0 = make_smem_desc(0, kWH * 16, 128, SWZ_NONE);
        const bool leader = elect_one();
        SegIter seg;
        seg.init();
        uint32_t it = 0, item = 0, d0 = 0;
        bool fresh = true;                           // the item's accumulator has not been written yet
        int acc = 0;
        bool ok = true;
        while (ok && seg.next(p)) {
            const int f0 = __ldg(p.bin_fill + seg.b), f1 = __ldg(p.bin_fill + seg.b + 1);
            int2 win = (f0 + lane < f1) ? __ldg(p.fills + f0 + lane) : kNoDesc;
            for (int wbase = f0; wbase < f1 && ok; wbase += 32) {
                const int2 nwin = (wbase + 32 + lane < f1) ? __ldg(p.fills + wbase + 32 + lane) : kNoDesc;
                const int nj = min(32, f1 - wbase);
                for (int j = 0; j < nj; ++j, ++it) {
                    const int dy = __shfl_sync(0xffffffffu, win.y, j);
                    const int cnt = dy & 0xFFFF;
                    const bool first = (dy >> 16) & 1, last = (dy >> 17) & 1;
                    // warp-uniform control flow: every lane waits and builds the (uniform)
                    // descriptors, one elected lane issues the tcgen05 instructions
                    if (first) {
                        acc = item % Cfg::kNAcc;
                        const uint32_t aph = (item / Cfg::kNAcc) & 1u;
                        ok = __all_sync(0xffffffffu, mbar_wait(acce_bar(acc), aph ^ 1u, ctl, 12));
                        tc_fence_after_sync();
                        d0 = tmem_base + acc * Cfg::kAccCols;
                        fresh = true;
                    }
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(full_bar(s), ph, ctl, 13));
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t sb = smem_base + s * Cfg::kStageBytes;
                        const int nks = cnt / Cfg::kKStep;
                        // descriptors differ only in their start-address field (bytes >> 4)
                        const uint64_t a0 = adesc0 + (sb >> 4);
                        const uint64_t b0 = bdesc0 + ((sb + Cfg::kDenseBytes) >> 4);
                        auto issue = [&](int ks) {
                            // the item's first MMA overwrites the accumulator: no zeroing pass
                            if (leader)
                                umma_kind<FMT == 3 ? 2 : (FMT == 2 ? 1 : 0)>(d0, a0 + ((ks * (Cfg::kKStep / 8) * 1024) >> 4),
                                                  b0 + ((ks * (kWH * 32)) >> 4), idesc, (ks > 0 || !fresh) ? 1u : 0u);
                        };
                        constexpr int kFullSteps = KT / Cfg::kKStep;
                        if (nks == kFullSteps) {                 // a full stage: straight-line code
#pragma unroll
                            for (int ks = 0; ks < kFullSteps; ++ks) issue(ks);
                        } else {
                            for (int ks = 0; ks < nks; ++ks) issue(ks);
                        }
                        fresh = false;
                        if (leader) {
                            tc_commit(empty_bar(s));
                            if (last) tc_commit(accf_bar(acc));
                        }
                        __syncwarp();
                    }
                    if (last) ++item;
                    if (!ok) break;
                }
                win = nwin;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int qd = warp & 3;
        SegIter seg;
        seg.init();
        uint32_t item = 0;
        bool ok = true;
        while (ok && seg.next(p)) {
            const int i0 = __ldg(p.bin_ptr + seg.b), i1 = __ldg(p.bin_ptr + seg.b + 1);
            const int n0 = seg.tt * Cfg::kBnT;
            const int4 kNoItem = make_int4(0, 0, 0, 0);
            int4 win = (i0 + lane < i1) ? __ldg(p.items + i0 + lane) : kNoItem;
            for (int wbase = i0; wbase < i1 && ok; wbase += 32) {
                const int4 nwin = (wbase + 32 + lane < i1) ? __ldg(p.items + wbase + 32 + lane) : kNoItem;
                const int nj = min(32, i1 - wbase);
                for (int j = 0; j < nj; ++j, ++item) {
                    const int window = __shfl_sync(0xffffffffu, win.x, j);
                    const int slot = __shfl_sync(0xffffffffu, win.y, j);
                    // unsplit window: straight to C (fp32 or the input's 16-bit type); split
                    // window: fp32 partial tile, summed by the merge kernel
                    using CElem = typename CType<FMT, CT>::type;
                    float* out;         // fp32 destination (C when it is fp32, or the partial tile)
                    CElem* outc;        // C in its own type
                    int rows;
                    if (slot < 0) {
                        const int64_t row0 = static_cast<int64_t>(window) * kWH;
                        outc = static_cast<CElem*>(p.C) + row0 * N;
                        out = reinterpret_cast<float*>(outc);
                        rows = static_cast<int>(min_i64(kWH, p.m - row0));
                    } else {
                        out = p.partial + static_cast<int64_t>(slot) * kWH * N;
                        outc = nullptr;
                        rows = kWH;
                    }
                    const int acc = item % Cfg::kNAcc;
                    const uint32_t aph = (item / Cfg::kNAcc) & 1u;
                    if (!__all_sync(0xffffffffu, mbar_wait(accf_bar(acc), aph, ctl, 14))) { ok = false; break; }
                    tc_fence_after_sync();
                    float v[kWH];
                    const uint32_t tbase = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + acc * Cfg::kAccCols;
#pragma unroll
                    for (int c = 0; c < kWH; c += 16) {
                        uint32_t u[16];
                        tmem_ld_x16(tbase + c, u);
                        tmem_ld_wait();
#pragma unroll
                        for (int jr = 0; jr < 16; ++jr) v[c + jr] = __uint_as_float(u[jr]);
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acce_bar(acc));
                    const int n = n0 + qd * 32 + lane;
                    if (n < N) {
                        if (sizeof(CElem) == 4 || slot >= 0) {
#pragma unroll
                            for (int jr = 0; jr < kWH; ++jr)
                                if (jr < rows) out[static_cast<int64_t>(jr) * N + n] = v[jr];
                        } else {
#pragma unroll
                            for (int jr = 0; jr < kWH; ++jr)
                                if (jr < rows) outc[static_cast<int64_t>(jr) * N + n] = from_f32<CElem>(v[jr]);
                        }
                    }
                }
                win = nwin;
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (*abort_flag) {
            // abort path: let the MMAs this warp's elected lane already issued finish before
            // TMEM is freed (kept out of the role loop above on purpose: placed there it
            // slowed the normal path measurably)
            if (elect_one()) {
                tc_commit(drain_bar);
                mbar_drain_wait(drain_bar, 0, ctl, 33);
            }
            __syncwarp();
        }
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// C rows of split windows = sum of their partial tiles in slot order; C rows of empty
// windows = 0.  One CTA per listed window.
template <typename CElem, int WH>
__global__ void __launch_bounds__(256)
wcsr_merge_kernel(const MergeParams p) {
    constexpr int kWH = WH;
    const int i = blockIdx.x;
    const int w = p.window[i];
    const int first = p.first[i];
    const int nparts = p.nparts[i];
    // everything above is creation-time data; the partial tiles and C belong to the SpMM
    // kernel launched just before on the same stream: wait until it has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t N = p.N;
    const int64_t row0 = static_cast<int64_t>(w) * kWH;
    const int rows = static_cast<int>(min_i64(kWH, p.m - row0));
    const int64_t n4 = N >> 2;     // N is a multiple of 4
    const int64_t total = static_cast<int64_t>(rows) * n4;
    const float4* part = reinterpret_cast<const float4*>(p.partial);
    CElem* out = static_cast<CElem*>(p.C) + row0 * N;
    for (int64_t e = threadIdx.x; e < total; e += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < nparts; ++s) {
            const float4 v = part[static_cast<int64_t>(first + s) * kWH * n4 + e];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if constexpr (sizeof(CElem) == 4) {
            reinterpret_cast<float4*>(out)[e] = acc;
        } else {
            alignas(8) CElem q[4] = {from_f32<CElem>(acc.x), from_f32<CElem>(acc.y), from_f32<CElem>(acc.z), from_f32<CElem>(acc.w)};
            reinterpret_cast<uint2*>(out)[e] = *reinterpret_cast<const uint2*>(q);
        }
    }
}

template <int ES, int FMT, int WH, int CT, bool NARROW = false, bool LSU = false>
cudaError_t launch_one(const CUtensorMap& tmB, const WcsrParams& p, int sms, cudaStream_t stream) {
    constexpr int KT = NARROW ? kWcsrNarrowCols : wcsr_stage_cols(ES);
    constexpr int STAGES = wcsr_stages(ES, WH), PW = wcsr_producer_warps(ES, WH);
    using Cfg = WcsrCfg<ES, WH, KT, STAGES, NARROW>;
    auto kfn = wcsr_spmm_kernel<ES, FMT, WH, KT, STAGES, PW, CT, NARROW, LSU>;
    // resident CTAs per SM: shared memory and TMEM columns are checked in WcsrCfg; the
    // register file follows from __launch_bounds__
    static_assert(Cfg::kCtasPerSm * Cfg::kTmemCols <= 512, "TMEM over-subscribed");
    // the attributes belong to the (function, device) pair: set them once per device
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
            e = cudaFuncSetAttribute(kfn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            attr_done[dev] = true;
        }
    }
    int grid = sms * Cfg::kCtasPerSm;
    if (grid > p.n_bins) grid = p.n_bins;
    if (grid < 1) return cudaSuccess;
    kfn<<<grid, (PW + 5) * 32, Cfg::kSmemBytes, stream>>>(tmB, p);
    return cudaGetLastError();
}

template <int WH>
cudaError_t launch_wh(int dtype, int c16, const CUtensorMap& tmB, const WcsrParams& p, int sms, cudaStream_t stream) {
    if (dtype == 2) return launch_one<4, 2, WH, 0>(tmB, p, sms, stream);
    if (dtype == 3) return c16 ? cudaErrorInvalidValue : launch_one<1, 3, WH, 0>(tmB, p, sms, stream);   // E4M3: fp32 C
    if (dtype == 1) return c16 ? launch_one<2, 0, WH, 1>(tmB, p, sms, stream) : launch_one<2, 0, WH, 0>(tmB, p, sms, stream);
    if (dtype == 0) return c16 ? launch_one<2, 1, WH, 1>(tmB, p, sms, stream) : launch_one<2, 1, WH, 0>(tmB, p, sms, stream);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_wcsr(int dtype, int wh, int c16, int narrow, int lsu_gather, const CUtensorMap& tmB, const WcsrParams& p, int sms,
                        cudaStream_t stream) {
    if (lsu_gather) {
        // the comparison variant: window height 16, fp32 C, 128-token stages
        if (wh != 16 || c16 || narrow) return cudaErrorInvalidValue;
        if (dtype == 2) return launch_one<4, 2, 16, 0, false, true>(tmB, p, sms, stream);
        if (dtype == 1) return launch_one<2, 0, 16, 0, false, true>(tmB, p, sms, stream);
        if (dtype == 0) return launch_one<2, 1, 16, 0, false, true>(tmB, p, sms, stream);
        return cudaErrorInvalidValue;
    }
    if (narrow) {
        if (wh != 16 || (dtype != 0 && dtype != 1)) return cudaErrorInvalidValue;
        if (dtype == 1) return c16 ? launch_one<2, 0, 16, 1, true>(tmB, p, sms, stream) : launch_one<2, 0, 16, 0, true>(tmB, p, sms, stream);
        return c16 ? launch_one<2, 1, 16, 1, true>(tmB, p, sms, stream) : launch_one<2, 1, 16, 0, true>(tmB, p, sms, stream);
    }
    if (wh == 16) return launch_wh<16>(dtype, c16, tmB, p, sms, stream);
    if (wh == 64) return launch_wh<64>(dtype, c16, tmB, p, sms, stream);
    return cudaErrorInvalidValue;
}

// Built-in scratch for spmm_wcsr_run_static: partial tiles of split windows, for callers
// that may not allocate device memory.  Every GPU that loads the library holds these
// kStaticScratchBytes until the process exits.  All handles and all calls share it.
constexpr size_t kStaticScratchBytes = size_t{8} << 20;
static __device__ __align__(256) float g_static_scratch[kStaticScratchBytes / sizeof(float)];

cudaError_t wcsr_static_scratch(float** ptr, size_t* bytes) {
    // In host code the array's name is only a stand-in for the device symbol, never a
    // device address: resolve it once per device, with that device current.
    static float* resolved[kMaxDevices] = {};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!resolved[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        resolved[dev] = p;
    }
    *ptr = resolved[dev];
    *bytes = kStaticScratchBytes;
    return cudaSuccess;
}

// ctype: 0 = fp32 C, 1 = fp16, 2 = bf16
cudaError_t launch_wcsr_merge(const MergeParams& p, int wh, int ctype, cudaStream_t stream) {
    if (p.n <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.n));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (wh == 64) {
        if (ctype == 1) return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<__half, 64>, p);
        if (ctype == 2) return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<__nv_bfloat16, 64>, p);
        return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<float, 64>, p);
    }
    if (ctype == 1) return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<__half, 16>, p);
    if (ctype == 2) return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<__nv_bfloat16, 16>, p);
    return cudaLaunchKernelEx(&cfg, wcsr_merge_kernel<float, 16>, p);
}

}  // namespace spmm
