// Machine-constant microbenchmarks for the B200 SpMM kernels (a stand-alone program, built beside
// the library; `python bench.py --ubench` runs it).  Three questions the kernel design rests on:
//
//   mma      interval between back-to-back tcgen05.mma (M = 128, K = 32 bytes, both operands in
//            shared memory) as a function of the N extent: one CTA, one issuing thread.
//   load     aggregate rate of TMA tiled loads from an L2-resident array into shared memory, every
//            SM streaming (the operand stream of the BCSR kernel: boxes of 64 rows x 128 bytes).
//   store    aggregate rate of TMA tiled stores from shared memory for several box shapes (what an
//            epilogue staging tile can look like), to a region that stays in L2 ("hot") or
//            streaming through a large array; and of st.global from registers.
//   mix      both at once on every SM, or loads on the even SMs and stores on the odd ones: how
//            much the two streams slow each other down, and whether that happens inside an SM.
//   gather   aggregate rate of TMA row gathers (tile::gather4: four rows x 128 bytes per request,
//            random rows of an L2-resident array), the operand stream of the WCSR kernel, for
//            several numbers of resident CTAs, issuing warps and 16 KB stages in flight.
//
// Every wait is bounded (an iteration limit; on expiry the thread records an error and leaves),
// device memory stays below 1 GB and each case runs for about a millisecond.  Output: one JSON
// line per case on stdout.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

using namespace spmm;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr uint32_t kSpinLimit = 1u << 26;     // polls before a wait gives up (seconds, not forever)

__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, int* err) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    atomicExch(err, 1);
    return false;
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { std::printf("{\"error\": \"%s at %s:%d\"}\n", cudaGetErrorString(e_), __FILE__, __LINE__); std::exit(1); } } while (0)

// ----------------------------------------------------------------------------- mma interval

__global__ void __launch_bounds__(128, 1) mma_kernel(int N, int iters, long long* out, int* err) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ uint64_t bar;
    __shared__ uint32_t tslot;
    for (int i = threadIdx.x; i < 64 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); fence_mbar_init(); }
    if (threadIdx.x < 32) { tmem_alloc(smem_u32(&tslot), 512); tmem_relinquish(); }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tslot;
    if (threadIdx.x < 32) {
        // M-side operand: 128 rows, MN-major, 128-byte swizzle (the token tile of the SpMM kernels);
        // N-side operand: N rows, K-major, 128-byte swizzle (a stored block)
        const uint32_t idesc = make_idesc(0, 128, N, 1, 0);
        const uint64_t ad = make_smem_desc(base, 8192, 1024, SWZ_128B);
        const uint64_t bd = make_smem_desc(base + 32768, 16, 1024, SWZ_128B);
        const int acc_mask = 512 / N - 1;          // accumulators in turn (512 / N is a power of two)
        const long long t0 = clock64();
        if (elect_one()) {
#pragma unroll 8
            for (int i = 0; i < iters; ++i) umma_ss<false>(tm + (i & acc_mask) * N, ad, bd, idesc, 1);
            tc_commit(smem_u32(&bar));
        }
        __syncwarp();
        wait_bounded(smem_u32(&bar), 0, err);
        const long long t1 = clock64();
        if (threadIdx.x == 0) out[0] = t1 - t0;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after_sync(); tmem_dealloc(tm, 512); }
}

// ----------------------------------------------------------------------------- load / store / mix

struct MixArgs {
    int load_slots;        // shared-memory slots of the load ring (0: no loads)
    int load_boxes;        // 8 KB boxes (64 rows x 128 bytes) per slot, one request per slot
    int load_iters;        // requests per loading CTA
    int src_row_tiles, src_col_tiles;
    int store_mode;        // 0 none, 1 TMA tiled store, 2 st.global from registers
    int store_iters;       // tiles per storing warp
    int store_depth;       // staging tiles per warp = TMA stores in flight per warp (1, 2 or 4)
    int tile_cols, tile_rows;   // fp32 elements per row of the store box, rows of the box
    int hot;               // 1: every warp rewrites its own tile (stays in L2); 0: streams through C
    int c_rows, c_cols;    // the fp32 array the stores go to
    int roles;             // 0: every CTA loads and stores; 1: even CTAs load, odd CTAs store
    int mma_n;             // > 0: a sixth warp issues mma_count MMAs (M = 128, N = mma_n, K = 16) on the ring's memory
    int mma_count;
    long long* mma_clk;    // [grid] cycles the MMA warp took
    float* C;
};

template <int kDepth>
__device__ __forceinline__ void store_loop(const CUtensorMap* tmS, const MixArgs& a, uint32_t stg0, int sw, int lane) {
    const int tile_bytes = a.tile_cols * a.tile_rows * 4;
    const int tiles_x = a.c_cols / a.tile_cols, tiles_y = a.c_rows / a.tile_rows;
    // streaming: the grid's warps walk C tile by tile, neighbours in x next to each other
    long long t = (static_cast<long long>(blockIdx.x) * 4 + sw);
    const long long stride = static_cast<long long>(gridDim.x) * 4;
    for (int i = 0; i < a.store_iters; ++i) {
        if (lane == 0) {
            bulk_wait_read<kDepth - 1>();
            const long long tt = a.hot ? (static_cast<long long>(blockIdx.x) * 4 + sw) : (t % (static_cast<long long>(tiles_x) * tiles_y));
            const int tx = static_cast<int>(tt % tiles_x), ty = static_cast<int>(tt / tiles_x);
            tma_store_2d(tmS, stg0 + (i % kDepth) * tile_bytes, tx * a.tile_cols, ty * a.tile_rows);
            bulk_commit_group();
        }
        t += stride;
    }
    if (lane == 0) bulk_wait_all<false>();
}

__global__ void __launch_bounds__(192, 1)
mix_kernel(const __grid_constant__ CUtensorMap tmL, const __grid_constant__ CUtensorMap tmS, const MixArgs a, int* err) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ uint64_t bar[17];
    __shared__ uint32_t tslot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot_bytes = a.load_boxes * 8192;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 17; ++i) mbar_init(smem_u32(&bar[i]), 1);
        fence_mbar_init();
    }
    if (warp == 5 && a.mma_n > 0) { tmem_alloc(smem_u32(&tslot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 5) {
        if (a.mma_n > 0) {
            // operands: the token tile of ring slot 0 (M side, as the SpMM kernel reads it) and 8 KB of
            // slot 1 as the stored block (N side); the data is whatever the loads leave there
            const uint32_t tm = tslot;
            const uint32_t idesc = make_idesc(1, 128, a.mma_n, 1, 0);
            const uint64_t ad = make_smem_desc(base, 8192, 1024, SWZ_128B);
            const uint64_t bd = make_smem_desc(base + slot_bytes, 16, 1024, SWZ_128B);
            const int acc_mask = 512 / a.mma_n - 1;
            // the ring's first loads bring the source array's values into both slots: give them time
            const long long ts = clock64();
            while (clock64() - ts < 30000) { }
            const long long t0 = clock64();
            if (elect_one()) {
#pragma unroll 8
                for (int i = 0; i < a.mma_count; ++i) umma_ss<false>(tm + (i & acc_mask) * a.mma_n, ad + ((i & 3) * 128), bd, idesc, 1);
                tc_commit(smem_u32(&bar[16]));
            }
            __syncwarp();
            wait_bounded(smem_u32(&bar[16]), 0, err);
            if (lane == 0) a.mma_clk[blockIdx.x] = clock64() - t0;
            tc_fence_before_sync();
            __syncwarp();
            tc_fence_after_sync();
            tmem_dealloc(tm, 512);
        }
        return;
    }
    const bool loads = a.load_slots > 0 && (a.roles == 0 || (blockIdx.x & 1) == 0);
    const bool stores = a.store_mode != 0 && (a.roles == 0 || (blockIdx.x & 1) == 1);
    if (warp == 0) {
        if (loads && lane == 0) {
            uint32_t seed = blockIdx.x * 2654435761u + 12345u;
            for (int i = 0; i < a.load_iters + a.load_slots; ++i) {
                const int s = i % a.load_slots;
                if (i >= a.load_slots && !wait_bounded(smem_u32(&bar[s]), ((i / a.load_slots) - 1) & 1, err)) break;
                if (i < a.load_iters) {
                    seed = seed * 1664525u + 1013904223u;
                    const int ct = (seed >> 8) % a.src_col_tiles, rt = (seed >> 20) % a.src_row_tiles;
                    mbar_arrive_expect_tx(smem_u32(&bar[s]), slot_bytes);
                    tma_load_3d(base + s * slot_bytes, &tmL, smem_u32(&bar[s]), 0, rt * 64, ct * a.load_boxes);
                }
            }
        }
    } else if (stores) {
        const int sw = warp - 1;
        const int tile_bytes = a.tile_cols * a.tile_rows * 4;
        const uint32_t stg0 = base + a.load_slots * slot_bytes + sw * a.store_depth * tile_bytes;
        if (a.store_mode == 1) {
            if (a.store_depth == 1) store_loop<1>(&tmS, a, stg0, sw, lane);
            else if (a.store_depth == 2) store_loop<2>(&tmS, a, stg0, sw, lane);
            else store_loop<4>(&tmS, a, stg0, sw, lane);
        } else {
            // st.global from registers: a warp instruction writes 32 consecutive fp32 of one row
            const int tiles_x = a.c_cols / 32, tiles_y = a.c_rows / a.tile_rows;
            long long t = (static_cast<long long>(blockIdx.x) * 4 + sw);
            const long long stride = static_cast<long long>(gridDim.x) * 4;
            for (int i = 0; i < a.store_iters; ++i) {
                const long long tt = a.hot ? (static_cast<long long>(blockIdx.x) * 4 + sw) : (t % (static_cast<long long>(tiles_x) * tiles_y));
                const int tx = static_cast<int>(tt % tiles_x), ty = static_cast<int>(tt / tiles_x);
                float* p = a.C + static_cast<size_t>(ty) * a.tile_rows * a.c_cols + tx * 32 + lane;
                for (int r = 0; r < a.tile_rows; ++r) p[static_cast<size_t>(r) * a.c_cols] = static_cast<float>(i + r);
                t += stride;
            }
        }
    }
}

// ----------------------------------------------------------------------------- row gather

// Every warp owns `slots` stages and refills a stage as soon as its data has landed: lane l < lanes
// requests rows 4 * (l / 2) .. + 3, 128-byte segment l % 2, as the WCSR kernel's producers do (all
// 32 lanes: 64 gathered rows x 256 bytes = 16 KB, the kernel's stage for 2-byte types).  Rows are
// pseudo-random.
__global__ void __launch_bounds__(384, 1)
gather_kernel(const __grid_constant__ CUtensorMap tmG, int slots, int lanes, int iters, int n_rows, int n_col_segs, int* err) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ uint64_t bar[16 * 4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int warps = blockDim.x >> 5;
    if (threadIdx.x == 0) {
        for (int i = 0; i < warps * slots; ++i) mbar_init(smem_u32(&bar[i]), 1);
        fence_mbar_init();
    }
    __syncthreads();
    uint32_t seed = (blockIdx.x * 64u + threadIdx.x / 2) * 2654435761u + 777u;
    const int rg = lane >> 1, sg = lane & 1;
    bool ok = true;
    for (int i = 0; i < iters + slots && ok; ++i) {
        const int sl = i % slots;
        const uint32_t b = smem_u32(&bar[warp * slots + sl]);
        if (i >= slots) ok = __all_sync(0xffffffffu, wait_bounded(b, ((i / slots) - 1) & 1, err));
        if (ok && i < iters) {
            const uint32_t sb = base + (warp * slots + sl) * (lanes * 512);
            if (lane == 0) mbar_arrive_expect_tx(b, lanes * 512);
            __syncwarp();
            int r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) { seed = seed * 1664525u + 1013904223u; r[k] = static_cast<int>((seed >> 8) % static_cast<uint32_t>(n_rows)); }
            seed = seed * 1664525u + 1013904223u;
            const int x = static_cast<int>((seed >> 10) % static_cast<uint32_t>(n_col_segs / 2)) * 128 + sg * 64;
            if (lane < lanes) tma_gather4_2d(sb + sg * (lanes * 256) + rg * 512, &tmG, b, x, r[0], r[1], r[2], r[3]);
        }
    }
}

// bf16 values +-[1, 2) with pseudo-random signs and mantissas
__global__ void fill_random_kernel(uint16_t* p, size_t n) {
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n; i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        uint32_t h = static_cast<uint32_t>(i) * 2654435761u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        p[i] = static_cast<uint16_t>(0x3F80u | (h & 0x7Fu) | ((h >> 8) & 1u) << 15);
    }
}

struct Ctx {
    EncodeTiledFn fn = nullptr;
    void* src = nullptr;        // bf16 [K][N], L2 resident
    float* C = nullptr;
    int* err = nullptr;
    int sms = 148;
    double clk_ghz = 1.965;
    static constexpr uint64_t K = 2048, N = 8192;         // 32 MB
    static constexpr int c_rows = 4096, c_cols = 32768;   // 512 MB of fp32
};

void run_mix(Ctx& cx, const char* name, MixArgs a) {
    CUtensorMap tmL, tmS;
    {
        const cuuint64_t dims[3] = {64, Ctx::K, Ctx::N / 64};
        const cuuint64_t strides[2] = {Ctx::N * 2, 128};
        const cuuint32_t box[3] = {64, 64, static_cast<cuuint32_t>(a.load_boxes > 0 ? a.load_boxes : 1)};
        const cuuint32_t es[3] = {1, 1, 1};
        if (cx.fn(&tmL, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, cx.src, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            std::printf("{\"error\": \"load map\"}\n");
            std::exit(1);
        }
        const cuuint64_t cd[2] = {static_cast<cuuint64_t>(Ctx::c_cols), static_cast<cuuint64_t>(Ctx::c_rows)};
        const cuuint64_t cs[1] = {static_cast<cuuint64_t>(Ctx::c_cols) * 4};
        const cuuint32_t cb[2] = {static_cast<cuuint32_t>(a.tile_cols), static_cast<cuuint32_t>(a.tile_rows)};
        if (cx.fn(&tmS, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, cx.C, cd, cs, cb, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            std::printf("{\"error\": \"store map\"}\n");
            std::exit(1);
        }
    }
    a.src_row_tiles = static_cast<int>(Ctx::K / 64);
    a.src_col_tiles = static_cast<int>(Ctx::N / 64 / (a.load_boxes > 0 ? a.load_boxes : 1));
    a.c_rows = Ctx::c_rows;
    a.c_cols = Ctx::c_cols;
    a.C = cx.C;
    const int smem = a.load_slots * a.load_boxes * 8192 + 4 * a.store_depth * a.tile_cols * a.tile_rows * 4 + 1024;
    if (smem > 227 * 1024) { std::printf("{\"case\": \"%s\", \"error\": \"shared memory\"}\n", name); return; }
    CK(cudaFuncSetAttribute(mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    float best = 1e30f;
    for (int rep = 0; rep < 3; ++rep) {
        CK(cudaEventRecord(e0));
        mix_kernel<<<cx.sms, 192, smem>>>(tmL, tmS, a, cx.err);
        CK(cudaEventRecord(e1));
        CK(cudaDeviceSynchronize());
        float ms;
        CK(cudaEventElapsedTime(&ms, e0, e1));
        if (rep > 0 && ms < best) best = ms;
    }
    int herr = 0;
    CK(cudaMemcpy(&herr, cx.err, 4, cudaMemcpyDeviceToHost));
    const int loaders = a.load_slots > 0 ? (a.roles ? (cx.sms + 1) / 2 : cx.sms) : 0;
    const int storers = a.store_mode ? (a.roles ? cx.sms / 2 : cx.sms) : 0;
    const double lb = double(loaders) * a.load_iters * a.load_boxes * 8192.0;
    const double sb = double(storers) * 4.0 * a.store_iters * a.tile_rows * (a.store_mode == 2 ? 32 : a.tile_cols) * 4.0;
    const double s = best * 1e-3;
    if (a.mma_n > 0) {
        std::vector<long long> clk(cx.sms);
        CK(cudaMemcpy(clk.data(), a.mma_clk, cx.sms * sizeof(long long), cudaMemcpyDeviceToHost));
        double sum = 0;
        for (long long c : clk) sum += double(c);
        std::printf("{\"case\": \"%s\", \"ms\": %.4f, \"load_tbs\": %.2f, \"load_B_per_clk_sm\": %.1f, \"mma_n\": %d, "
                    "\"clk_per_mma\": %.1f, \"wait_ran_out\": %d}\n",
                    name, best, lb / s / 1e12, loaders ? lb / s / loaders / (cx.clk_ghz * 1e9) : 0.0, a.mma_n,
                    sum / cx.sms / a.mma_count, herr);
        std::fflush(stdout);
        CK(cudaEventDestroy(e0));
        CK(cudaEventDestroy(e1));
        return;
    }
    std::printf("{\"case\": \"%s\", \"ms\": %.4f, \"load_tbs\": %.2f, \"store_tbs\": %.2f, \"load_B_per_clk_sm\": %.1f, "
                "\"store_B_per_clk_sm\": %.1f, \"loading_sms\": %d, \"storing_sms\": %d, \"wait_ran_out\": %d}\n",
                name, best, lb / s / 1e12, sb / s / 1e12, loaders ? lb / s / loaders / (cx.clk_ghz * 1e9) : 0.0,
                storers ? sb / s / storers / (cx.clk_ghz * 1e9) : 0.0, loaders, storers, herr);
    std::fflush(stdout);
    CK(cudaEventDestroy(e0));
    CK(cudaEventDestroy(e1));
}

void run_gather(Ctx& cx, const char* name, int ctas_per_sm, int warps, int slots, int lanes, int iters) {
    CUtensorMap tmG;
    const cuuint64_t dims[2] = {Ctx::N, Ctx::K};
    const cuuint64_t strides[1] = {Ctx::N * 2};
    const cuuint32_t box[2] = {64, 1};
    const cuuint32_t es[2] = {1, 1};
    if (cx.fn(&tmG, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cx.src, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
        std::printf("{\"error\": \"gather map\"}\n");
        std::exit(1);
    }
    const int smem = warps * slots * lanes * 512 + 1024;
    if (warps > 12 || warps * slots > 64 || ctas_per_sm * (smem + 1024) > 227 * 1024) {
        std::printf("{\"case\": \"%s\", \"error\": \"shape\"}\n", name);
        return;
    }
    CK(cudaFuncSetAttribute(gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    float best = 1e30f;
    for (int rep = 0; rep < 3; ++rep) {
        CK(cudaEventRecord(e0));
        gather_kernel<<<cx.sms * ctas_per_sm, warps * 32, smem>>>(tmG, slots, lanes, iters, static_cast<int>(Ctx::K), static_cast<int>(Ctx::N / 64), cx.err);
        CK(cudaEventRecord(e1));
        CK(cudaDeviceSynchronize());
        float ms;
        CK(cudaEventElapsedTime(&ms, e0, e1));
        if (rep > 0 && ms < best) best = ms;
    }
    int herr = 0;
    CK(cudaMemcpy(&herr, cx.err, 4, cudaMemcpyDeviceToHost));
    const double bytes = double(cx.sms) * ctas_per_sm * warps * iters * (lanes * 512.0);
    const double sec = best * 1e-3;
    std::printf("{\"case\": \"%s\", \"ms\": %.4f, \"gather_tbs\": %.2f, \"gather_B_per_clk_sm\": %.1f, \"clk_per_request_sm\": %.1f, "
                "\"ctas_per_sm\": %d, \"warps\": %d, \"stages_per_warp\": %d, \"requests_per_stage\": %d, \"KB_in_flight_per_sm\": %d, \"wait_ran_out\": %d}\n",
                name, best, bytes / sec / 1e12, bytes / sec / cx.sms / (cx.clk_ghz * 1e9),
                512.0 / (bytes / sec / cx.sms / (cx.clk_ghz * 1e9)), ctas_per_sm, warps, slots, lanes, ctas_per_sm * warps * slots * lanes / 2, herr);
    std::fflush(stdout);
    CK(cudaEventDestroy(e0));
    CK(cudaEventDestroy(e1));
}

}  // namespace

int main(int argc, char** argv) {
    Ctx cx;
    void* fnp = nullptr;
    cudaDriverEntryPointQueryResult q;
    CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &q));
    cx.fn = reinterpret_cast<EncodeTiledFn>(fnp);
    cudaDeviceProp prop;
    CK(cudaGetDeviceProperties(&prop, 0));
    if (prop.major != 10) { std::printf("{\"error\": \"needs an sm_100 device\"}\n"); return 1; }
    cx.sms = prop.multiProcessorCount;
    int khz = 0;
    CK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0));
    cx.clk_ghz = khz * 1e-6;
    CK(cudaMalloc(&cx.src, Ctx::K * Ctx::N * 2));
    CK(cudaMemset(cx.src, 0, Ctx::K * Ctx::N * 2));
    CK(cudaMalloc(&cx.C, size_t(Ctx::c_rows) * Ctx::c_cols * 4));
    CK(cudaMalloc(&cx.err, 4));
    CK(cudaMemset(cx.err, 0, 4));
    const bool quick = argc > 1 && std::strcmp(argv[1], "--quick") == 0;

    // ---- mma interval
    {
        long long* d;
        CK(cudaMalloc(&d, 8));
        CK(cudaFuncSetAttribute(mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 66 * 1024));
        const int iters = 4000;
        for (int N : {16, 32, 64, 128, 256}) {
            for (int rep = 0; rep < 2; ++rep) {
                mma_kernel<<<1, 128, 66 * 1024>>>(N, iters, d, cx.err);
                CK(cudaDeviceSynchronize());
            }
            long long h = 0;
            CK(cudaMemcpy(&h, d, 8, cudaMemcpyDeviceToHost));
            std::printf("{\"case\": \"mma_m128_n%d_k16_bf16\", \"clk_per_mma\": %.1f, \"smem_operand_bytes\": %d}\n", N, double(h) / iters,
                        128 * 32 + N * 32);
        }
        CK(cudaFree(d));
    }

    // ---- loads alone: ring depth
    MixArgs base{};
    base.load_boxes = 8;           // 64 KB per request, the BCSR kernel's 512-token stage
    base.load_iters = 1500;
    base.store_depth = 2;
    base.tile_cols = 32;
    base.tile_rows = 64;
    for (int slots : {1, 2}) {
        MixArgs a = base;
        a.load_slots = slots;
        char nm[64];
        std::snprintf(nm, sizeof nm, "load_only_%dx64KB", slots);
        run_mix(cx, nm, a);
    }
    {
        MixArgs a = base;
        a.load_boxes = 4; a.load_slots = 4; a.load_iters = 3000;
        run_mix(cx, "load_only_4x32KB", a);
    }

    // ---- row gathers: {resident CTAs per SM, issuing warps per CTA, 16 KB stages per warp}
    {
        struct G { int ctas, warps, slots, lanes; };
        const G gs[] = {{1, 1, 1, 32}, {1, 1, 4, 32}, {1, 4, 1, 32}, {1, 4, 3, 32}, {1, 12, 1, 32}, {3, 4, 1, 32}, {2, 6, 1, 32},
                        {3, 8, 1, 16}, {2, 12, 1, 16}, {3, 12, 1, 8}, {3, 12, 1, 10}, {3, 4, 2, 16}, {3, 8, 2, 8}};
        for (const G& g : gs) {
            char nm[96];
            std::snprintf(nm, sizeof nm, "gather4_%dcta_%dwarps_x%dstages_of_%dreq", g.ctas, g.warps, g.slots, g.lanes);
            run_gather(cx, nm, g.ctas, g.warps, g.slots, g.lanes, 6000 * 32 / (g.ctas * g.warps * g.lanes));      // ~100 MB per SM
        }
    }

    // ---- MMAs beside the loads: do operand reads and TMA writes share shared-memory bandwidth?
    // And does the rate of the MMAs depend on the operand VALUES (all SMs issuing: a power question)?
    {
        long long* dclk;
        CK(cudaMalloc(&dclk, cx.sms * sizeof(long long)));
        for (int random_data : {0, 1}) {
            if (random_data) {
                fill_random_kernel<<<1024, 256>>>(static_cast<uint16_t*>(cx.src), Ctx::K * Ctx::N);
                CK(cudaDeviceSynchronize());
            }
            for (int n : {64, 128, 256}) {
                for (int with_loads : {0, 1}) {
                    MixArgs a = base;
                    a.load_slots = 2;                               // the ring's memory holds the operands either way
                    a.load_iters = with_loads ? 1500 : 2;           // (alone: one load per slot, then nothing)
                    a.mma_n = n;
                    a.mma_count = n == 64 ? 28000 : (n == 128 ? 21000 : 10500);   // about as long as the loads alone
                    a.mma_clk = dclk;
                    char nm[96];
                    std::snprintf(nm, sizeof nm, "mma_n%d%s_%s_operands", n, with_loads ? "_with_loads_2x64KB" : "_alone_all_sms",
                                  random_data ? "random" : "zero");
                    run_mix(cx, nm, a);
                }
            }
        }
        CK(cudaMemset(cx.src, 0, Ctx::K * Ctx::N * 2));
        CK(cudaFree(dclk));
    }

    // ---- stores alone and beside loads, per box shape
    struct Shape { int cols, rows; };
    const Shape shapes[] = {{32, 4}, {32, 8}, {32, 16}, {32, 64}, {64, 32}, {128, 16}, {256, 8}, {128, 64}};
    for (const Shape& sh : shapes) {
        for (int hot : {1, 0}) {
            for (int with_loads : {0, 1}) {
                if (quick && !hot) continue;
                MixArgs a = base;
                a.tile_cols = sh.cols; a.tile_rows = sh.rows;
                a.store_mode = 1;
                a.hot = hot;
                a.store_depth = sh.cols * sh.rows * 4 >= 32768 ? 1 : 2;
                const int tile_bytes = sh.cols * sh.rows * 4;
                a.store_iters = (24 << 20) / 4 / tile_bytes;         // 24 MB per SM
                a.load_slots = with_loads ? 2 : 0;
                a.load_iters = with_loads ? 1200 : 0;                // 75 MB per SM
                char nm[96];
                std::snprintf(nm, sizeof nm, "tma_store_%dx%dB_%s%s", sh.rows, sh.cols * 4, hot ? "hot" : "stream", with_loads ? "_with_loads" : "");
                run_mix(cx, nm, a);
                if (with_loads) {
                    a.roles = 1;
                    std::snprintf(nm, sizeof nm, "tma_store_%dx%dB_%s_loads_on_even_stores_on_odd_sms", sh.rows, sh.cols * 4, hot ? "hot" : "stream");
                    run_mix(cx, nm, a);
                }
            }
        }
    }
    // ---- more stores in flight per warp: 16 x 128 B boxes with four staging tiles per warp
    for (int hot : {1, 0})
        for (int with_loads : {0, 1}) {
            MixArgs a = base;
            a.tile_cols = 32; a.tile_rows = 16; a.store_mode = 1; a.hot = hot; a.store_depth = 4;
            a.store_iters = (24 << 20) / 4 / 2048;
            a.load_slots = with_loads ? 2 : 0;
            a.load_iters = with_loads ? 1200 : 0;
            char nm[96];
            std::snprintf(nm, sizeof nm, "tma_store_16x128B_depth4_%s%s", hot ? "hot" : "stream", with_loads ? "_with_loads" : "");
            run_mix(cx, nm, a);
        }
    // ---- st.global from registers
    for (int hot : {1, 0})
        for (int with_loads : {0, 1}) {
            MixArgs a = base;
            a.store_mode = 2; a.tile_cols = 32; a.tile_rows = 64; a.hot = hot;
            a.store_iters = (24 << 20) / 4 / 8192;
            a.load_slots = with_loads ? 2 : 0;
            a.load_iters = with_loads ? 1200 : 0;
            char nm[96];
            std::snprintf(nm, sizeof nm, "st_global_64x128B_%s%s", hot ? "hot" : "stream", with_loads ? "_with_loads" : "");
            run_mix(cx, nm, a);
        }
    CK(cudaFree(cx.src));
    CK(cudaFree(cx.C));
    CK(cudaFree(cx.err));
    return 0;
}
