// WCSR SpMM kernel for sm_100a (Sec. 3.2 - 3.3 of the paper, re-designed for Blackwell).
//
// Work item: one sub-task of the split plan (a run of `count` condensed columns of one
// 16-row window) times BN_T = 128 * GROUPS columns of B ("tokens").  It accumulates
//     D[n, r] += sum_q  B[window_col_idx[q], n0 + n] * values[r, q]
// with the tokens on the 128 TMEM lanes (MMA M side; the gathered B rows are written to
// shared memory in the MN-major 128-byte-swizzled layout tcgen05.mma reads) and the 16
// window rows as the MMA N side (operand = the packed window tile, K-major, un-swizzled).
//
// Roles (288 threads, persistent CTAs):
//   warps 0-3   gather producers: per stage read KT column indices and copy the matching
//               B rows with 16-byte cp.async (zero fill for -1 pads) into a STAGES-deep
//               ring; thread 0 also bulk-copies the contiguous packed A tile.  A stage is
//               published LAG fills later (wait_group + proxy fence + mbarrier arrive), so
//               LAG + 1 stages of loads stay in flight per thread.
//   warp 4      MMA issuer (one thread): count / b_col tcgen05.mma per group and stage.
//   warps 5-8   epilogue: tcgen05.ld, release the TMEM buffer, store to C (unsplit window)
//               or to the task's partial tile (split window).
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

constexpr int kWH = 16;
constexpr int kProducerWarps = 4;
constexpr int kNAcc = 4;

template <int ES, int GROUPS, int KT, int STAGES>
struct WcsrCfg {
    static constexpr int kE16 = 16 / ES;                    // elements per 16-byte chunk
    static constexpr int kKStep = 32 / ES;                  // columns per MMA (= b_col)
    static constexpr int kBnT = 128 * GROUPS;
    static constexpr int kRowBytes = kBnT * ES;
    static constexpr int kCh = kRowBytes / 16;              // 16-byte chunks per gathered row
    static constexpr int kIssues = KT * kCh / 32;           // cp.async per lane per fill
    static constexpr int kIdxRegs = (KT + 31) / 32;         // column indices held per lane
    static constexpr int kAtomStride = KT * 128;            // bytes between MN atoms
    static constexpr int kAtomsPerGroup = ES;               // 128 tokens * ES / 128 B
    static constexpr int kDenseBytes = KT * kRowBytes;
    static constexpr int kABytes = (KT / kKStep) * (kWH * 32);
    static constexpr int kStageBytes = kDenseBytes + kABytes;
    static constexpr int kAccCols = GROUPS * kWH;
    static constexpr int kTmemCols = kNAcc * kAccCols < 32 ? 32 : kNAcc * kAccCols;
    static constexpr int kSmemBytes = STAGES * kStageBytes + 1024 + 256;
    static_assert(KT % 8 == 0 && KT % kKStep == 0 && KT <= 64, "stage shape");
    static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

// Walks the fills a CTA owns, in the order every role uses: bins blockIdx.x, +grid, ...;
// inside a bin all token tiles; inside a token tile the bin's fills.
struct FillCursor {
    int sp, tt, f, f_end;
    __device__ __forceinline__ void load_bin(const WcsrParams& p) {
        if (sp < p.n_bins) {
            f = __ldg(p.bin_fill + sp);
            f_end = __ldg(p.bin_fill + sp + 1);
        }
    }
    __device__ __forceinline__ void normalise(const WcsrParams& p) {
        while (sp < p.n_bins && f >= f_end) {
            if (f_end > __ldg(p.bin_fill + sp) && tt + 1 < p.n_tt) {
                ++tt;
                f = __ldg(p.bin_fill + sp);
            } else {
                tt = 0;
                sp += gridDim.x;
                load_bin(p);
            }
        }
    }
    __device__ __forceinline__ void init(const WcsrParams& p) {
        sp = blockIdx.x;
        tt = 0;
        f = f_end = 0;
        load_bin(p);
        normalise(p);
    }
    __device__ __forceinline__ bool done(const WcsrParams& p) const { return sp >= p.n_bins; }
    __device__ __forceinline__ void step(const WcsrParams& p) {
        ++f;
        normalise(p);
    }
};

template <int ES, int FMT, int GROUPS, int KT, int STAGES>
__global__ void __launch_bounds__(288, (WcsrCfg<ES, GROUPS, KT, STAGES>::kSmemBytes + 1024) * 2 <= 227 * 1024 ? 2 : 1)
wcsr_spmm_kernel(const WcsrParams p) {
    using Cfg = WcsrCfg<ES, GROUPS, KT, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::kStageBytes);
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + kNAcc + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 2 * kNAcc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 2 * kNAcc + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WaitCtl ctl{abort_flag, p.status, p.wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 32); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < kNAcc; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 4) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int64_t N = p.N;

    if (warp < kProducerWarps) {
        // ------------------------------------------------------------------ gather producers
        // Warp w fills stages for the CTA's fills w, w + 4, ...; a fill is one warp's job from
        // the index loads to the mbarrier arrive, so four fills are always in progress.
        const int c = lane % Cfg::kCh;               // my 16-byte chunk inside a gathered row
        const int rsub = lane / Cfg::kCh;            // my row inside one issue (kCh < 32)
        constexpr int kRowsPerIssue = Cfg::kCh >= 32 ? 1 : 32 / Cfg::kCh;
        constexpr int kIssuesPerRow = Cfg::kCh > 32 ? Cfg::kCh / 32 : 1;
        const uint8_t* Bp = static_cast<const uint8_t*>(p.B);
        const size_t row_pitch = static_cast<size_t>(N) * ES;

        // Three fills are tracked per warp: `cur` (indices in registers, rows being copied),
        // `n1` (descriptor in registers, indices requested while cur's rows travel) and `n2`
        // (descriptor requested), so neither a descriptor nor an index load stalls the copy loop.
        FillCursor cur;
        cur.init(p);
        for (int i = 0; i < warp && !cur.done(p); ++i) cur.step(p);
        FillCursor n1 = cur;
        for (int i = 0; i < kProducerWarps && !n1.done(p); ++i) n1.step(p);
        uint32_t it = warp;
        bool have = !cur.done(p), have1 = !n1.done(p);
        int2 d_cur = make_int2(0, 0), d_n1 = make_int2(0, 0);
        int idx_cur[Cfg::kIdxRegs];
        if (have) d_cur = __ldg(p.fills + cur.f);
        if (have1) d_n1 = __ldg(p.fills + n1.f);
        if (have) {
            const int cnt = d_cur.y & 0xFFFF;
#pragma unroll
            for (int j = 0; j < Cfg::kIdxRegs; ++j)
                idx_cur[j] = (j * 32 + lane < cnt) ? __ldg(p.col_idx + d_cur.x + j * 32 + lane) : -1;
        }
        bool ok = true;
        while (have) {
            FillCursor n2 = n1;
            for (int i = 0; i < kProducerWarps && !n2.done(p); ++i) n2.step(p);
            const bool have2 = have1 && !n2.done(p);
            int2 d_n2 = make_int2(0, 0);
            if (have2) d_n2 = __ldg(p.fills + n2.f);

            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            const int q = d_cur.x;
            const int cnt = d_cur.y & 0xFFFF;
            const int n0 = cur.tt * Cfg::kBnT;
            if (!mbar_wait(empty_bar(s), ph ^ 1u, ctl, 11)) { ok = false; break; }
            const uint32_t sb = smem_base + s * Cfg::kStageBytes;
            if (lane == 0) {
                const uint32_t abytes = (cnt / Cfg::kKStep) * (kWH * 32);
                mbar_expect_tx(full_bar(s), abytes);
                bulk_load_1d(sb + Cfg::kDenseBytes, p.packed + static_cast<size_t>(q / Cfg::kKStep) * (kWH * 32),
                             abytes, full_bar(s));
            }
#pragma unroll
            for (int i = 0; i < Cfg::kIssues; ++i) {
                const int r = (i / kIssuesPerRow) * kRowsPerIssue + rsub;
                const int cc = c + (i % kIssuesPerRow) * 32;        // chunk inside the row
                // (the register holding row r's index is known at compile time: rsub < kRowsPerIssue)
                const int idx = __shfl_sync(0xffffffffu, idx_cur[((i / kIssuesPerRow) * kRowsPerIssue) >> 5], r & 31);
                if (r < cnt && n0 + cc * Cfg::kE16 < N) {
                    uint32_t dst = sb + (cc >> 3) * Cfg::kAtomStride + r * 128;
                    if constexpr (ES == 2) {
                        // 128-byte swizzle: 16-byte chunk index ^= row % 8
                        dst += ((cc & 7) ^ (r & 7)) << 4;
                    } else {
                        // 128-byte swizzle with 32-byte atoms (the only MN-major layout for
                        // 32-bit operands): 32-byte chunk index ^= row % 4
                        dst += ((((cc & 7) >> 1) ^ (r & 3)) << 5) + ((cc & 1) << 4);
                    }
                    const bool valid = idx >= 0;
                    const uint8_t* src = Bp + (valid ? static_cast<size_t>(idx) * row_pitch +
                                                           (static_cast<size_t>(n0) + cc * Cfg::kE16) * ES
                                                     : 0);
                    cp_async_16(dst, src, valid);
                }
            }
            cp_async_commit();
            // the next fill's indices travel while this fill's rows do
            int idx_n1[Cfg::kIdxRegs];
#pragma unroll
            for (int j = 0; j < Cfg::kIdxRegs; ++j) idx_n1[j] = -1;
            if (have1) {
                const int cn = d_n1.y & 0xFFFF;
#pragma unroll
                for (int j = 0; j < Cfg::kIdxRegs; ++j)
                    if (j * 32 + lane < cn) idx_n1[j] = __ldg(p.col_idx + d_n1.x + j * 32 + lane);
            }
            cp_async_wait<0>();
            fence_proxy_async_smem();
            mbar_arrive(full_bar(s));
            cur = n1;
            n1 = n2;
            d_cur = d_n1;
            d_n1 = d_n2;
#pragma unroll
            for (int j = 0; j < Cfg::kIdxRegs; ++j) idx_cur[j] = idx_n1[j];
            have = have1;
            have1 = have2;
            it += kProducerWarps;
        }
        cp_async_wait<0>();
        if (!ok && lane == 0 && it >= kProducerWarps) {
            // abort path: the A tile of this warp's previous fill may still be in flight
            const uint32_t j = it - kProducerWarps;
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1u) && globaltimer_ns() - t0 < 2000000ull) {}
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(FMT, 128, kWH, 1, 0);
            FillCursor cur;
            cur.init(p);
            uint32_t it = 0, item = 0;
            bool have = !cur.done(p);
            int2 d_cur = make_int2(0, 0);
            if (have) d_cur = __ldg(p.fills + cur.f);
            uint32_t d0 = 0;
            int acc = 0;
            while (have) {
                FillCursor nxt = cur;
                nxt.step(p);
                const bool have_n = !nxt.done(p);
                int2 d_nxt = make_int2(0, 0);
                if (have_n) d_nxt = __ldg(p.fills + nxt.f);

                const int cnt = d_cur.y & 0xFFFF;
                const bool first = (d_cur.y >> 16) & 1, last = (d_cur.y >> 17) & 1;
                const int n0 = cur.tt * Cfg::kBnT;
                const int nvalid = static_cast<int>(min_i64(Cfg::kBnT, N - n0));
                const int ngrp = (nvalid + 127) >> 7;
                if (first) {
                    acc = item % kNAcc;
                    const uint32_t aph = (item / kNAcc) & 1u;
                    if (!mbar_wait(acce_bar(acc), aph ^ 1u, ctl, 12)) break;
                    tc_fence_after_sync();
                    d0 = tmem_base + acc * Cfg::kAccCols;
                }
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1u;
                if (!mbar_wait(full_bar(s), ph, ctl, 13)) break;
                tc_fence_after_sync();
                const uint32_t sb = smem_base + s * Cfg::kStageBytes;
                const int nks = cnt / Cfg::kKStep;
                for (int ks = 0; ks < nks; ++ks) {
                    const uint64_t bdesc = make_smem_desc(sb + Cfg::kDenseBytes + ks * (kWH * 32), kWH * 16, 128, SWZ_NONE);
                    const uint32_t accum = (!first || ks > 0) ? 1u : 0u;
                    for (int g = 0; g < ngrp; ++g) {
                        const uint64_t adesc = make_smem_desc(
                            sb + g * Cfg::kAtomsPerGroup * Cfg::kAtomStride + ks * (Cfg::kKStep / 8) * 1024,
                            Cfg::kAtomStride, ES == 2 ? 1024 : 512, ES == 2 ? SWZ_128B : SWZ_128B_BASE32B);
                        umma_ss<FMT == 2>(d0 + g * kWH, adesc, bdesc, idesc, accum);
                    }
                }
                tc_commit(empty_bar(s));
                if (last) {
                    tc_commit(accf_bar(acc));
                    ++item;
                }
                cur = nxt;
                d_cur = d_nxt;
                have = have_n;
                ++it;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int qd = warp & 3;
        uint32_t item = 0;
        bool ok = true;
        for (int sp = blockIdx.x; sp < p.n_bins && ok; sp += gridDim.x) {
            const int t_begin = p.bin_ptr[sp], t_end = p.bin_ptr[sp + 1];
            for (int tt = 0; tt < p.n_tt && ok; ++tt) {
                const int n0 = tt * Cfg::kBnT;
                for (int ti = t_begin; ti < t_end; ++ti, ++item) {
                    const int t = __ldg(p.bin_tasks + ti);
                    const WcsrDevTask task = p.tasks[t];
                    float* out;
                    int rows;
                    if (task.slot < 0) {
                        const int64_t row0 = static_cast<int64_t>(task.window) * kWH;
                        out = p.C + row0 * N;
                        rows = static_cast<int>(min_i64(kWH, p.m - row0));
                    } else {
                        out = p.partial + static_cast<int64_t>(task.slot) * kWH * N;
                        rows = kWH;
                    }
                    const int acc = item % kNAcc;
                    const uint32_t aph = (item / kNAcc) & 1u;
                    if (!mbar_wait(accf_bar(acc), aph, ctl, 14)) { ok = false; break; }
                    tc_fence_after_sync();
                    uint32_t v[GROUPS][16];
#pragma unroll
                    for (int g = 0; g < GROUPS; ++g)
                        tmem_ld_x16(tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + acc * Cfg::kAccCols + g * kWH, v[g]);
                    tmem_ld_wait();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acce_bar(acc));
#pragma unroll
                    for (int g = 0; g < GROUPS; ++g) {
                        const int n = n0 + g * 128 + qd * 32 + lane;
                        if (n < N) {
#pragma unroll
                            for (int j = 0; j < kWH; ++j)
                                if (j < rows) out[static_cast<int64_t>(j) * N + n] = __uint_as_float(v[g][j]);
                        }
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// C rows of split windows = sum of their partial tiles in slot order; C rows of empty
// windows = 0.  One CTA per listed window.
__global__ void __launch_bounds__(256)
wcsr_merge_kernel(const MergeParams p) {
    const int i = blockIdx.x;
    const int w = p.window[i];
    const int first = p.first[i];
    const int nparts = p.nparts[i];
    const int64_t N = p.N;
    const int64_t row0 = static_cast<int64_t>(w) * kWH;
    const int rows = static_cast<int>(min_i64(kWH, p.m - row0));
    const int64_t n4 = N >> 2;     // N is a multiple of 4
    const int64_t total = static_cast<int64_t>(rows) * n4;
    const float4* part = reinterpret_cast<const float4*>(p.partial);
    float4* out = reinterpret_cast<float4*>(p.C + row0 * N);
    for (int64_t e = threadIdx.x; e < total; e += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < nparts; ++s) {
            const float4 v = part[static_cast<int64_t>(first + s) * kWH * n4 + e];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        out[e] = acc;
    }
}

template <int ES, int FMT, int GROUPS, int KT, int STAGES>
cudaError_t launch_one(const WcsrParams& p, int sms, cudaStream_t stream) {
    using Cfg = WcsrCfg<ES, GROUPS, KT, STAGES>;
    auto kfn = wcsr_spmm_kernel<ES, FMT, GROUPS, KT, STAGES>;
    static int occ = 0;
    if (occ == 0) {
        cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kfn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        // resident CTAs per SM: 227 KB of shared memory (1 KB reserved per CTA), 512 TMEM
        // columns, and the register file (__launch_bounds__ keeps two CTAs of 288 threads)
        int o = (227 * 1024) / (Cfg::kSmemBytes + 1024);
        o = o < 512 / Cfg::kTmemCols ? o : 512 / Cfg::kTmemCols;
        occ = o < 1 ? 1 : (o > 2 ? 2 : o);
    }
    int grid = sms * occ;
    if (grid > p.n_bins) grid = p.n_bins;
    if (grid < 1) return cudaSuccess;
    kfn<<<grid, 288, Cfg::kSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_wcsr(int dtype, int groups, const WcsrParams& p, int sms, cudaStream_t stream) {
    if (dtype == 2) {
        if (groups == 1) return launch_one<4, 2, 1, 32, 6>(p, sms, stream);
        if (groups == 2) return launch_one<4, 2, 2, 32, 6>(p, sms, stream);
    } else if (dtype == 1) {
        if (groups == 1) return launch_one<2, 0, 1, 64, 6>(p, sms, stream);
        if (groups == 2) return launch_one<2, 0, 2, 64, 6>(p, sms, stream);
    } else if (dtype == 0) {
        if (groups == 1) return launch_one<2, 1, 1, 64, 6>(p, sms, stream);
        if (groups == 2) return launch_one<2, 1, 2, 64, 6>(p, sms, stream);
    }
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
    constexpr int kMaxDevices = 64;
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

cudaError_t launch_wcsr_merge(const MergeParams& p, cudaStream_t stream) {
    if (p.n <= 0) return cudaSuccess;
    wcsr_merge_kernel<<<p.n, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace spmm
