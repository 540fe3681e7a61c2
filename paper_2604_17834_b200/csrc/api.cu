// C-ABI layer: handles, format upload, tensor maps, launches (see include/spmm_b200.h).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "format.h"
#include "kernels.h"
#include "spmm_b200.h"

using namespace spmm;

namespace {

// NVTX range around an entry point (a no-op unless a profiler is attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};

inline int elem_size(int dtype) { return dtype == SPMM_TF32 ? 4 : (dtype == SPMM_FP8_E4M3 ? 1 : 2); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

inline CUtensorMapDataType tmap_dtype(int dtype) {
    return dtype == SPMM_FP8_E4M3 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
         : (dtype == SPMM_TF32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
         : (dtype == SPMM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16));
}

// 2-D row-major tensor [rows][cols] of the handle's value type, box [box_rows][box_cols].
int encode_2d(CUtensorMap* map, int dtype, const void* base, uint64_t rows, uint64_t cols,
                    uint32_t box_rows, uint32_t box_cols, CUtensorMapSwizzle swz) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return SPMM_ERR_CUDA;
    const uint64_t es = static_cast<uint64_t>(elem_size(dtype));
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * es};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = tmap_dtype(dtype);
    CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SPMM_OK : SPMM_ERR_CUDA;
}

template <class T>
int upload(T** dptr, const void* src, size_t bytes) {
    *dptr = nullptr;
    const size_t alloc = bytes ? bytes : 16;
    if (cudaMalloc(reinterpret_cast<void**>(dptr), alloc) != cudaSuccess) return SPMM_ERR_ALLOC;
    if (bytes && cudaMemcpy(*dptr, src, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return SPMM_ERR_CUDA;
    return SPMM_OK;
}

}  // namespace

struct spmm_handle_s {
    int format = 0;      // 0 BCSR, 1 WCSR
    int dtype = 0;
    int es = 2;
    int64_t m = 0, k = 0, nnz = 0;
    bool host_only = false;
    bool c16 = false;        // C in the input's 16-bit type (never with TF32, whose input type is fp32)
    bool col_major = false;  // BCSR: B given as X[N][k], C as Y[N][m]
    bool dynamic = false;    // BCSR: tiles handed out at run time through Cluster Launch Control
    bool lsu_gather = false; // WCSR: B rows gathered by the load/store units (comparison variant) instead of TMA
    int cs = 4;              // bytes per C element
    int n_ctas = 148;
    int sms = 148;
    int device = 0;

    BcsrHost bcsr;       // index arrays kept; value array dropped after upload unless host_only
    WcsrHost wcsr;

    // device copies
    int32_t* d_ptr = nullptr;        // block_row_ptr / window_row_ptr
    int32_t* d_idx = nullptr;        // block_col_idx / window_col_idx
    uint8_t* d_vals = nullptr;       // blocks / packed values
    int32_t* d_order = nullptr;      // BCSR row order
    BcsrSchedule sched;              // BCSR tile schedule of the most recent dense width
    // BCSR row groups (stacked 128-row blocks): plan, device arrays and their own tile schedule
    BcsrStack stack;
    int stack_min_fill = 0;          // opts.stack_min_fill
    BcsrSchedule sched_stack;
    int32_t* d_sidx = nullptr;       // block columns of the stacked blocks
    int32_t* d_srows = nullptr;      // [groups][R] member block-rows
    uint8_t* d_svals = nullptr;      // [stacked blocks][128][b]
    int32_t* d_stile_recs = nullptr; // {group, token tile, first stacked block, end}
    int32_t* d_scta_ptr = nullptr;
    CUtensorMap tmAs;                // map of d_svals
    CUtensorMap tmB3s;               // whole-tile map of B for the stacked launch's 256-token tile
    bool tmB3s_ok = false;
    int k_split = 0;                 // opts.k_split (1: cut outlier block-rows into parts)
    int32_t* d_kmerge = nullptr;     // K-split merge lists: row | first slot | parts, each [n_kmerge]
    int n_kmerge = 0;
    CUtensorMap tmP;                 // store map of the K-split partial tiles
    bool tmP_ok = false;
    int32_t* d_tiles = nullptr;      // {block-row, token tile} pairs (the exported schedule)
    int32_t* d_tile_recs = nullptr;  // the kernel's records: {block-row, token tile, first block, end block}
    int32_t* d_cta_ptr = nullptr;
    WcsrDevTask* d_tasks = nullptr;
    int32_t* d_bin_ptr = nullptr;
    int32_t* d_bin_tasks = nullptr;
    int32_t* d_items = nullptr;
    int32_t* d_fills = nullptr;
    int32_t* d_bin_fill = nullptr;
    int32_t* d_fills_narrow = nullptr;    // WCSR narrow-operand variant (2-byte types, height 16)
    int32_t* d_bin_fill_narrow = nullptr;
    uint8_t* d_grp_class = nullptr;  // WCSR: reuse class per group of four padded columns (gather hints)
    int32_t* d_merge = nullptr;      // window | first | nparts, each [n_merge]
    int n_merge = 0;
    int* d_status = nullptr;

    float* d_partial = nullptr;      // WCSR workspace
    size_t partial_bytes = 0;

    // BCSR tensor maps
    CUtensorMap tmA;
    bool tmA_ok = false;
    CUtensorMap tmB;
    CUtensorMap tmB3;                // BCSR: B as [N / 64][k][64] for whole-tile loads
    bool tmB3_ok = false;
    int tmB_groups = 0;
    const void* tmB_ptr = nullptr;
    int64_t tmB_N = -1;
    CUtensorMap tmC;                 // BCSR: the store map of C (or of Y, column-major)
    const void* tmC_ptr = nullptr;
    int64_t tmC_N = -1;

    // staging for spmm_run_host
    void* d_Bstage = nullptr;
    size_t Bstage_bytes = 0;
    float* d_Cstage = nullptr;
    size_t Cstage_bytes = 0;
    // spmm_run_host in column chunks: the copy streams and the events that order them
    static constexpr int kMaxHostChunks = 8;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_in[kMaxHostChunks] = {}, ev_run[kMaxHostChunks] = {};
};

namespace {

void free_handle(spmm_handle_s* h) {
    if (!h) return;
    if (!h->host_only) {
        cudaFree(h->d_ptr);
        cudaFree(h->d_idx);
        cudaFree(h->d_vals);
        cudaFree(h->d_order);
        cudaFree(h->d_tiles);
        cudaFree(h->d_tile_recs);
        cudaFree(h->d_cta_ptr);
        cudaFree(h->d_kmerge);
        cudaFree(h->d_sidx);
        cudaFree(h->d_srows);
        cudaFree(h->d_svals);
        cudaFree(h->d_stile_recs);
        cudaFree(h->d_scta_ptr);
        cudaFree(h->d_tasks);
        cudaFree(h->d_bin_ptr);
        cudaFree(h->d_bin_tasks);
        cudaFree(h->d_items);
        cudaFree(h->d_fills);
        cudaFree(h->d_bin_fill);
        cudaFree(h->d_fills_narrow);
        cudaFree(h->d_bin_fill_narrow);
        cudaFree(h->d_grp_class);
        cudaFree(h->d_merge);
        cudaFree(h->d_status);
        cudaFree(h->d_partial);
        cudaFree(h->d_Bstage);
        cudaFree(h->d_Cstage);
        if (h->s_in) cudaStreamDestroy(h->s_in);
        if (h->s_out) cudaStreamDestroy(h->s_out);
        if (h->ev_start) cudaEventDestroy(h->ev_start);
        for (int i = 0; i < spmm_handle_s::kMaxHostChunks; ++i) {
            if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
            if (h->ev_run[i]) cudaEventDestroy(h->ev_run[i]);
        }
    }
    delete h;
}

int device_setup(spmm_handle_s* h, const spmm_opts_t* opts) {
    if (h->host_only) {
        h->sms = 148;
        h->n_ctas = (opts && opts->n_ctas > 0) ? opts->n_ctas : 148;
        return SPMM_OK;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPMM_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SPMM_ERR_CUDA;
    if (prop.major != 10) return SPMM_ERR_UNSUPPORTED;   // sm_100a code only
    h->device = dev;
    h->sms = prop.multiProcessorCount;
    h->n_ctas = (opts && opts->n_ctas > 0) ? opts->n_ctas : h->sms;
    if (cudaMalloc(reinterpret_cast<void**>(&h->d_status), 4 * sizeof(int)) != cudaSuccess) return SPMM_ERR_ALLOC;
    if (cudaMemset(h->d_status, 0, 4 * sizeof(int)) != cudaSuccess) return SPMM_ERR_CUDA;
    return SPMM_OK;
}

int check_opts(const spmm_opts_t* opts) {
    if (!opts) return SPMM_OK;
    if (opts->c_type != SPMM_C_FP32 && opts->c_type != SPMM_C_SAME_AS_INPUT) return SPMM_ERR_INVALID_ARG;
    if (opts->layout != SPMM_ROWMAJOR && opts->layout != SPMM_COLMAJOR) return SPMM_ERR_INVALID_ARG;
    if (opts->schedule != SPMM_SCHED_STATIC && opts->schedule != SPMM_SCHED_DYNAMIC) return SPMM_ERR_INVALID_ARG;
    if (opts->gather != SPMM_GATHER_TMA && opts->gather != SPMM_GATHER_LSU) return SPMM_ERR_INVALID_ARG;
    return SPMM_OK;
}

// Option checks shared by the host and the device builder; on success *hp is a fresh handle.
int new_bcsr_handle(spmm_handle_s** hp, int64_t m, int64_t k, int dtype, int block, const spmm_opts_t* opts) {
    if (dtype != SPMM_BF16 && dtype != SPMM_FP16 && dtype != SPMM_FP8_E4M3 && dtype != SPMM_TF32) return SPMM_ERR_UNSUPPORTED;
    if (int orc = check_opts(opts)) return orc;
    // TF32 (Sec. 3.1's k8 shape, the type of Sec. 4.1's BCSR evaluation): static schedule only
    if (dtype == SPMM_TF32 && opts && opts->schedule != SPMM_SCHED_STATIC) return SPMM_ERR_UNSUPPORTED;
    if (dtype == SPMM_FP8_E4M3) {
        // 8-bit inputs: fp32 C, static schedule; a block row must hold a whole 32-element K step;
        // with column-major operands the rows of X are k bytes and must be multiples of 16
        if (opts && (opts->c_type != SPMM_C_FP32 || opts->schedule != SPMM_SCHED_STATIC)) return SPMM_ERR_UNSUPPORTED;
        if (block < 32) return SPMM_ERR_UNSUPPORTED;
        if (opts && opts->layout == SPMM_COLMAJOR && k % 16 != 0) return SPMM_ERR_UNSUPPORTED;
    }
    spmm_handle_s* h = new (std::nothrow) spmm_handle_s;
    if (!h) return SPMM_ERR_ALLOC;
    h->format = 0;
    h->dtype = dtype;
    h->es = elem_size(dtype);
    h->m = m;
    h->k = k;
    h->host_only = opts && opts->host_only;
    h->c16 = opts && opts->c_type == SPMM_C_SAME_AS_INPUT && dtype != SPMM_TF32;   // TF32's own type is fp32
    h->cs = h->c16 ? 2 : 4;
    h->col_major = opts && opts->layout == SPMM_COLMAJOR;
    h->dynamic = opts && opts->schedule == SPMM_SCHED_DYNAMIC;
    h->stack_min_fill = opts ? opts->stack_min_fill : 0;
    h->k_split = opts ? opts->k_split : 0;
    if (h->stack_min_fill > 100) { delete h; return SPMM_ERR_INVALID_ARG; }
    if (h->dynamic && (h->c16 || h->col_major)) { delete h; return SPMM_ERR_UNSUPPORTED; }
    // column-major operands: rows of X (k elements) and of Y (m elements) must be multiples of
    // 16 bytes for the tensor map and for the 16-byte pieces the epilogue writes
    if (h->col_major && (m % 8 != 0 || (k * h->es) % 16 != 0)) { delete h; return SPMM_ERR_UNSUPPORTED; }
    *hp = h;
    return SPMM_OK;
}

// Tensor map of the stored blocks: box rows of min(b * es, 128) bytes, swizzle = the row bytes.
int encode_tmA(spmm_handle_s* h) {
    const BcsrHost& f = h->bcsr;
    if (f.nnzb <= 0) return SPMM_OK;
    if (static_cast<int64_t>(f.nnzb) * f.b >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    // (a stage unit's rows: the whole block row, or one column slice of it, at most 128 bytes per piece)
    const int unit_bytes = f.b / bcsr_k_split(f.b, h->es) * h->es;
    const int row_bytes = unit_bytes < 128 ? unit_bytes : 128;
    const int bw = row_bytes / h->es;
    const CUtensorMapSwizzle swz = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    int rc = encode_2d(&h->tmA, h->dtype, h->d_vals, static_cast<uint64_t>(f.nnzb) * f.b, f.b,
                             static_cast<uint32_t>(f.b * bcsr_blocks_per_stage(f.b)), bw, swz);
    h->tmA_ok = rc == SPMM_OK;
    return rc;
}

// Row groups: the plan from the index arrays, then (unless host_only) the stacked values built on
// the device from the uploaded blocks, the groups' index arrays and the map of the stacked values.
int setup_stack(spmm_handle_s* h) {
    const BcsrHost& f = h->bcsr;
    // static schedule only; b = 128 blocks already are 128 rows high
    // (row groups exist for the 16-bit types, and for E4M3 with column-major operands)
    const bool eligible = !h->dynamic && f.b < 128 && h->stack_min_fill >= 0 && h->dtype != SPMM_TF32 &&
                          !(h->dtype == SPMM_FP8_E4M3 && !h->col_major);
    int rc = build_bcsr_stack(f, eligible ? h->stack_min_fill : -1, &h->stack);
    if (rc || h->host_only || h->stack.ng == 0) return rc;
    const BcsrStack& st = h->stack;
    rc = stack_bcsr_device(h->d_vals, st, f.b, h->es, &h->d_svals);
    if (!rc) rc = upload(&h->d_sidx, st.col_idx.data(), st.col_idx.size() * 4);
    if (!rc) rc = upload(&h->d_srows, st.rows.data(), st.rows.size() * 4);
    if (rc) return rc;
    std::vector<int32_t>().swap(h->stack.src);        // only needed to build the values
    const int row_bytes = f.b * h->es;                // <= 128 for b <= 64
    const CUtensorMapSwizzle swz = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    return encode_2d(&h->tmAs, h->dtype, h->d_svals, static_cast<uint64_t>(st.ns) * kStackRows, f.b, kStackRows, f.b, swz);
}

int create_bcsr(spmm_handle_t* out, const CsrView& a, int dtype, int block, const spmm_opts_t* opts) {
    spmm_handle_s* h = nullptr;
    int rc = new_bcsr_handle(&h, a.m, a.k, dtype, block, opts);
    if (rc) return rc;
    rc = validate_csr(a);
    if (rc) { delete h; return rc; }
    h->nnz = a.nnz;
    rc = device_setup(h, opts);
    if (rc) { free_handle(h); return rc; }
    try {
        rc = build_bcsr(a, block, &h->bcsr);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) { free_handle(h); return rc; }
    if (!h->host_only) {
        const BcsrHost& f = h->bcsr;
        if (static_cast<int64_t>(f.nnzb) * f.b >= (int64_t{1} << 31)) { free_handle(h); return SPMM_ERR_TOO_LARGE; }
        rc = upload(&h->d_ptr, f.block_row_ptr.data(), f.block_row_ptr.size() * 4);
        if (!rc) rc = upload(&h->d_idx, f.block_col_idx.data(), f.block_col_idx.size() * 4);
        if (!rc) rc = upload(&h->d_vals, f.blocks.data(), f.blocks.size());
        if (!rc) rc = upload(&h->d_order, f.row_order.data(), f.row_order.size() * 4);
        if (!rc) rc = encode_tmA(h);
        if (rc) { free_handle(h); return rc; }
        std::vector<uint8_t>().swap(h->bcsr.blocks);   // the device copy is the one that counts
    }
    try {
        rc = setup_stack(h);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) { free_handle(h); return rc; }
    *out = h;
    return SPMM_OK;
}

// The same handle from a CSR matrix in device memory: the format is built by GPU kernels.
int create_bcsr_device(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx,
                       const void* d_vals, int dtype, int block, const spmm_opts_t* opts, cudaStream_t stream) {
    if (opts && opts->host_only) return SPMM_ERR_INVALID_ARG;
    spmm_handle_s* h = nullptr;
    int rc = new_bcsr_handle(&h, m, k, dtype, block, opts);
    if (rc) return rc;
    rc = device_setup(h, opts);
    if (rc) { free_handle(h); return rc; }
    try {
        rc = build_bcsr_device(m, k, d_row_ptr, d_col_idx, static_cast<const uint8_t*>(d_vals), h->es, block, stream,
                               &h->bcsr, &h->nnz, &h->d_ptr, &h->d_idx, &h->d_vals);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (!rc) rc = upload(&h->d_order, h->bcsr.row_order.data(), h->bcsr.row_order.size() * 4);
    if (!rc) rc = encode_tmA(h);
    if (!rc) {
        try {
            rc = setup_stack(h);
        } catch (const std::bad_alloc&) {
            rc = SPMM_ERR_ALLOC;
        }
    }
    if (rc) { free_handle(h); return rc; }
    *out = h;
    return SPMM_OK;
}

// Uploads the schedule arrays of a WCSR handle (everything but the three format arrays).
int upload_wcsr_plan(spmm_handle_s* h) {
    const WcsrHost& f = h->wcsr;
    std::vector<WcsrDevTask> dt(f.tasks.size());
    for (size_t i = 0; i < f.tasks.size(); ++i) {
        dt[i].col_begin = f.window_row_ptr[f.tasks[i].window] + f.tasks[i].q0;
        dt[i].count = f.tasks[i].count;
        dt[i].window = f.tasks[i].window;
        dt[i].slot = f.tasks[i].slot;
    }
    const size_t nm = f.merge_window.size();
    std::vector<int32_t> mg(3 * nm);
    for (size_t i = 0; i < nm; ++i) {
        mg[i] = f.merge_window[i];
        mg[nm + i] = f.merge_first[i];
        mg[2 * nm + i] = f.merge_nparts[i];
    }
    h->n_merge = static_cast<int>(nm);
    int rc = upload(&h->d_tasks, dt.data(), dt.size() * sizeof(WcsrDevTask));
    if (!rc) rc = upload(&h->d_bin_ptr, f.bin_ptr.data(), f.bin_ptr.size() * 4);
    if (!rc) rc = upload(&h->d_bin_tasks, f.bin_tasks.data(), f.bin_tasks.size() * 4);
    if (!rc) {
        std::vector<int32_t> items(4 * f.bin_tasks.size(), 0);
        for (size_t i = 0; i < f.bin_tasks.size(); ++i) {
            items[4 * i] = f.tasks[f.bin_tasks[i]].window;
            items[4 * i + 1] = f.tasks[f.bin_tasks[i]].slot;
            items[4 * i + 2] = f.tasks[f.bin_tasks[i]].count;
        }
        rc = upload(&h->d_items, items.data(), items.size() * 4);
    }
    if (!rc) rc = upload(&h->d_fills, f.fills.data(), f.fills.size() * 4);
    if (!rc) rc = upload(&h->d_bin_fill, f.bin_fill.data(), f.bin_fill.size() * 4);
    if (!rc && !f.bin_fill_narrow.empty()) {
        rc = upload(&h->d_fills_narrow, f.fills_narrow.data(), f.fills_narrow.size() * 4);
        if (!rc) rc = upload(&h->d_bin_fill_narrow, f.bin_fill_narrow.data(), f.bin_fill_narrow.size() * 4);
    }
    if (!rc) rc = upload(&h->d_merge, mg.data(), mg.size() * 4);
    if (!rc && !f.grp_class.empty()) {
        rc = upload(&h->d_grp_class, f.grp_class.data(), f.grp_class.size());
        if (!rc) std::vector<uint8_t>().swap(h->wcsr.grp_class);
    }
    return rc;
}

// Option and size checks shared by the host and the device builder; on success *hp is a fresh handle.
int new_wcsr_handle(spmm_handle_s** hp, int64_t m, int64_t k, int dtype, const spmm_opts_t* opts, int* b_col_out, int* T_out) {
    if (dtype != SPMM_BF16 && dtype != SPMM_FP16 && dtype != SPMM_TF32 && dtype != SPMM_FP8_E4M3) return SPMM_ERR_UNSUPPORTED;
    if (int orc = check_opts(opts)) return orc;
    if (opts && opts->layout == SPMM_COLMAJOR) return SPMM_ERR_UNSUPPORTED;   // BCSR only
    // 8-bit inputs: fp32 C, the TMA gather
    if (dtype == SPMM_FP8_E4M3 && opts && (opts->c_type != SPMM_C_FP32 || opts->gather != SPMM_GATHER_TMA)) return SPMM_ERR_UNSUPPORTED;
    if (opts && opts->schedule == SPMM_SCHED_DYNAMIC) return SPMM_ERR_UNSUPPORTED;
    const int es = elem_size(dtype);
    const int b_col_default = 32 / es;
    const int b_col = (opts && opts->b_col > 0) ? opts->b_col : b_col_default;
    if (b_col != b_col_default) return SPMM_ERR_UNSUPPORTED;
    const int T = (opts && opts->split_cols > 0) ? opts->split_cols : 0;   // 0: chosen from the matrix
    if (T % b_col != 0) return SPMM_ERR_INVALID_ARG;
    spmm_handle_s* h = new (std::nothrow) spmm_handle_s;
    if (!h) return SPMM_ERR_ALLOC;
    h->format = 1;
    h->dtype = dtype;
    h->es = es;
    h->m = m;
    h->k = k;
    h->host_only = opts && opts->host_only;
    h->c16 = opts && opts->c_type == SPMM_C_SAME_AS_INPUT && dtype != SPMM_TF32;
    h->cs = h->c16 ? 2 : 4;
    h->lsu_gather = opts && opts->gather == SPMM_GATHER_LSU;
    if (h->lsu_gather && h->c16) { delete h; return SPMM_ERR_UNSUPPORTED; }   // the comparison variant writes fp32 C
    *hp = h;
    *b_col_out = b_col;
    *T_out = T;
    return SPMM_OK;
}

int create_wcsr(spmm_handle_t* out, const CsrView& a, int dtype, int wh, const spmm_opts_t* opts) {
    spmm_handle_s* h = nullptr;
    int b_col = 0, T = 0;
    int rc = new_wcsr_handle(&h, a.m, a.k, dtype, opts, &b_col, &T);
    if (rc) return rc;
    if (h->lsu_gather && wh != 16) { delete h; return SPMM_ERR_UNSUPPORTED; }
    rc = validate_csr(a);
    if (rc) { delete h; return rc; }
    h->nnz = a.nnz;
    rc = device_setup(h, opts);
    if (rc) { free_handle(h); return rc; }
    try {
        rc = build_wcsr(a, wh, b_col, T, h->n_ctas * wcsr_bins_per_sm(h->es, wh), &h->wcsr);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) { free_handle(h); return rc; }
    if (!h->host_only) {
        const WcsrHost& f = h->wcsr;
        rc = upload(&h->d_ptr, f.window_row_ptr.data(), f.window_row_ptr.size() * 4);
        if (!rc) rc = upload(&h->d_idx, f.window_col_idx.data(), f.window_col_idx.size() * 4);
        if (!rc) rc = upload(&h->d_vals, f.packed.data(), f.packed.size());
        if (!rc) rc = upload_wcsr_plan(h);
        if (rc) { free_handle(h); return rc; }
        std::vector<uint8_t>().swap(h->wcsr.packed);
    }
    *out = h;
    return SPMM_OK;
}

// The same handle from a CSR matrix in device memory: the format arrays are built by GPU kernels.
int create_wcsr_device(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx,
                       const void* d_vals, int dtype, int wh, const spmm_opts_t* opts, cudaStream_t stream) {
    if (opts && opts->host_only) return SPMM_ERR_INVALID_ARG;
    spmm_handle_s* h = nullptr;
    int b_col = 0, T = 0;
    int rc = new_wcsr_handle(&h, m, k, dtype, opts, &b_col, &T);
    if (rc) return rc;
    if (h->lsu_gather && wh != 16) { delete h; return SPMM_ERR_UNSUPPORTED; }
    rc = device_setup(h, opts);
    if (rc) { free_handle(h); return rc; }
    try {
        rc = build_wcsr_device(m, k, d_row_ptr, d_col_idx, static_cast<const uint8_t*>(d_vals), h->es, wh, b_col, T,
                               h->n_ctas * wcsr_bins_per_sm(h->es, wh), stream, &h->wcsr, &h->nnz, &h->d_ptr, &h->d_idx,
                               &h->d_vals, &h->d_grp_class);
        if (!rc) rc = upload_wcsr_plan(h);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) { free_handle(h); return rc; }
    *out = h;
    return SPMM_OK;
}

int make_view(CsrView* v, int64_t m, int64_t k, const int64_t* row_ptr, const int32_t* col_idx, const void* vals,
              int dtype) {
    if (dtype < 0 || dtype > 3) return SPMM_ERR_INVALID_ARG;
    if (m < 0 || k < 0 || !row_ptr) return SPMM_ERR_INVALID_ARG;
    if (m >= (int64_t{1} << 31) || k >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    v->m = m;
    v->k = k;
    v->row_ptr = row_ptr;
    v->nnz = row_ptr[m];
    v->col_idx = col_idx;
    v->vals = static_cast<const uint8_t*>(vals);
    v->es = elem_size(dtype);
    return SPMM_OK;
}

// Map of B for the WCSR row gather: box = one row x 128 bytes.
int encode_gather_map(CUtensorMap* map, int dtype, const void* base, uint64_t rows, uint64_t cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return SPMM_ERR_CUDA;
    const uint32_t es = static_cast<uint32_t>(elem_size(dtype));
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * es};
    const cuuint32_t box[2] = {128 / es, 1};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = tmap_dtype(dtype);
    const CUtensorMapSwizzle swz = dtype == SPMM_TF32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
    const CUtensorMapL2promotion promo = cols * es >= 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_NONE;
    CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                    promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SPMM_OK : SPMM_ERR_CUDA;
}

int ensure_tmB(spmm_handle_s* h, const void* B, int64_t N, int groups) {
    if (h->tmB_ptr == B && h->tmB_N == N && h->tmB_groups == groups) return SPMM_OK;
    int rc;
    if (h->format == 1) {
        rc = encode_gather_map(&h->tmB, h->dtype, B, static_cast<uint64_t>(h->k), static_cast<uint64_t>(N));
    } else if (h->col_major) {
        // X as [N][k]: box = 128 tokens x min(b, 64) elements, swizzle = the box's row bytes;
        // and the same memory as [N / 128][128][k] so that one request brings all token groups
        // of a tile (whole groups only; a ragged last tile uses the 2-D map, zero filled)
        // (per stage unit: the block's k extent, or one column slice of it -- bcsr_k_split)
        const uint32_t unit_bytes = h->bcsr.b / bcsr_k_split(h->bcsr.b, h->es) * h->es;
        const uint32_t row_bytes = unit_bytes < 128 ? unit_bytes : 128;
        const uint32_t bw = row_bytes / h->es;
        const CUtensorMapSwizzle swz = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                      : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
        rc = encode_2d(&h->tmB, h->dtype, B, static_cast<uint64_t>(N), static_cast<uint64_t>(h->k), 128, bw, swz);
        EncodeTiledFn fn = get_encode_fn();
        auto whole_tile_map = [&](int g, CUtensorMap* out, bool* ok) {
            *ok = false;
            *out = h->tmB;
            if (rc || !fn || N < 128) return;
            const cuuint64_t dims[3] = {static_cast<cuuint64_t>(h->k), 128, static_cast<cuuint64_t>(N / 128)};
            const cuuint64_t strides[2] = {static_cast<cuuint64_t>(h->k) * h->es, static_cast<cuuint64_t>(h->k) * 128 * h->es};
            const cuuint32_t box[3] = {bw, 128, static_cast<cuuint32_t>(g)};
            const cuuint32_t estr[3] = {1, 1, 1};
            const CUtensorMapDataType dt = tmap_dtype(h->dtype);
            CUresult r = fn(out, dt, 3, const_cast<void*>(B), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            *ok = r == CUDA_SUCCESS;
            if (!*ok) *out = h->tmB;
        };
        whole_tile_map(groups, &h->tmB3, &h->tmB3_ok);
        if (h->stack.ng > 0) whole_tile_map(kStackGroups, &h->tmB3s, &h->tmB3s_ok);
    } else {
        // B as [k][N]: box = kb rows (the block's k extent, or one column slice of A's block:
        // bcsr_k_split) x 128 bytes of tokens; 4-byte elements take the 128-byte swizzle with
        // 32-byte atoms, which is what a token-major (MN-major) tensor-core operand of that
        // width reads
        const uint32_t tok = 128u / static_cast<uint32_t>(h->es);          // tokens per box row
        const uint32_t kb = static_cast<uint32_t>(h->bcsr.b / bcsr_k_split(h->bcsr.b, h->es));
        const CUtensorMapSwizzle swz = h->es == 4 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
        rc = encode_2d(&h->tmB, h->dtype, B, static_cast<uint64_t>(h->k), static_cast<uint64_t>(N), kb, tok, swz);
        // the same memory as [N / tok][k][tok]: one request then brings a whole token tile
        // (es * groups boxes); only full groups of tok tokens are covered, a ragged tail uses tmB
        EncodeTiledFn fn = get_encode_fn();
        auto whole_tile_map = [&](int g, CUtensorMap* out, bool* ok) {
            *ok = false;
            *out = h->tmB;
            if (rc || !fn || N < static_cast<int64_t>(tok)) return;
            const cuuint64_t dims[3] = {tok, static_cast<cuuint64_t>(h->k), static_cast<cuuint64_t>(N / tok)};
            const cuuint64_t strides[2] = {static_cast<cuuint64_t>(N) * h->es, 128};
            const cuuint32_t box[3] = {tok, kb, static_cast<cuuint32_t>(h->es * g)};
            const cuuint32_t estr[3] = {1, 1, 1};
            CUresult r = fn(out, tmap_dtype(h->dtype), 3, const_cast<void*>(B), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            *ok = r == CUDA_SUCCESS;
            if (!*ok) *out = h->tmB;
        };
        whole_tile_map(groups, &h->tmB3, &h->tmB3_ok);
        if (h->stack.ng > 0) whole_tile_map(kStackGroups, &h->tmB3s, &h->tmB3s_ok);
    }
    if (rc) return rc;
    h->tmB_ptr = B;
    h->tmB_N = N;
    h->tmB_groups = groups;
    return SPMM_OK;
}

// Store map of C for the BCSR epilogue (shared-memory staging tile -> TMA store).
int ensure_tmC(spmm_handle_s* h, void* C, int64_t N) {
    if (h->tmC_ptr == C && h->tmC_N == N) return SPMM_OK;
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return SPMM_ERR_CUDA;
    const uint32_t w = static_cast<uint32_t>(bcsr_epi_cols(h->bcsr.b, h->c16, h->col_major));
    const CUtensorMapDataType dt = !h->c16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : (h->dtype == SPMM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
    const cuuint32_t estr[2] = {1, 1};
    CUresult r;
    if (h->col_major) {
        const cuuint64_t dims[2] = {static_cast<cuuint64_t>(h->m), static_cast<cuuint64_t>(N)};
        const cuuint64_t strides[1] = {static_cast<cuuint64_t>(h->m) * h->cs};
        const cuuint32_t box[2] = {w, 32};
        const CUtensorMapSwizzle swz = w * h->cs == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE;
        r = fn(&h->tmC, dt, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(h->m)};
        const cuuint64_t strides[1] = {static_cast<cuuint64_t>(N) * h->cs};
        const cuuint32_t box[2] = {32, w};
        r = fn(&h->tmC, dt, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return SPMM_ERR_CUDA;
    h->tmC_ptr = C;
    h->tmC_N = N;
    return SPMM_OK;
}

// Tile width, slab width and the tile schedule for dense width N (cached for the last N).
int ensure_schedule(spmm_handle_s* h, int64_t N) {
    if (h->sched.N == N) return SPMM_OK;
    const BcsrHost& f = h->bcsr;
    // token tile: the largest of 512 / 256 / 128 columns that divides N (Sec. 4.3: pick a tile
    // width that divides the dense width so that no padded columns are computed); otherwise
    // the largest tile, whose ragged last tile is predicated.
    const int gmax = bcsr_token_groups_max(h->dtype, f.b, h->c16 ? 1 : 0, h->col_major ? 1 : 0);
    int groups = 0;
    for (int g = gmax; g >= 1; g >>= 1)
        if (N % (128 * g) == 0) { groups = g; break; }
    if (!groups) groups = N >= 128 * gmax ? gmax : (N > 128 ? 2 : 1);
    // keep at least ~8 tiles per CTA so that the schedule has something to balance
    while (groups > 1 && f.nbr * ((N + 128 * groups - 1) / (128 * groups)) < 8 * h->n_ctas) groups >>= 1;
    const int bnt = 128 * groups;
    const int n_tt = static_cast<int>((N + bnt - 1) / bnt);
    // slab: token tiles whose B rows (k x slab columns) stay within ~16 MB of L2 (C streams through the same cache)
    const int64_t slab_cols = (int64_t{16} << 20) / (h->k * h->es > 0 ? h->k * h->es : 1);
    int64_t sw = slab_cols / bnt;
    if (sw < 1) sw = 1;
    if (sw > n_tt) sw = n_tt;
    BcsrSchedule sc, ss;
    const BcsrStack& st = h->stack;
    int rc;
    try {
        // dynamic scheduling: one list in the global order (slab by slab, longest block-row first)
        // b = 64 gains little per stacked block (its MMAs, not the operand traffic, bound it), so
        // its row groups are used only when they make at least one tile per CTA
        const int64_t n_tt_groups = (N + 128 * kStackGroups - 1) / (128 * kStackGroups);
        const bool use_groups = st.ng > 0 && (f.b <= 32 || st.ng * n_tt_groups >= h->n_ctas);
        if (!use_groups) {
            // K-split of outlier block-rows: static schedule, fp32 row-major C (the parts' partial
            // tiles are fp32 and go through the same epilogue as C)
            rc = SPMM_OK;
            // (opt-in: measured 2 - 7 % slower than the uncut plan on the skewed sweep -- the parts'
            // extra epilogues and the merge launch cost more than the better balance returns)
            if (!h->dynamic && !h->c16 && !h->col_major && h->k_split > 0)
                rc = build_bcsr_ksplit(f, n_tt, h->n_ctas, &sc.units, &sc.n_slots, &sc.cap);
            if (!rc && !sc.units.empty()) {
                const int32_t nu = static_cast<int32_t>(sc.units.size() / 4);
                std::vector<int32_t> order(static_cast<size_t>(nu)), lens(static_cast<size_t>(nu));
                for (int32_t u = 0; u < nu; ++u) order[u] = u;
                auto ulen = [&](int32_t u) { return sc.units[4 * u + 2] - sc.units[4 * u + 1]; };
                std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return ulen(x) > ulen(y); });
                for (int32_t r = 0; r < nu; ++r) lens[r] = ulen(order[r]);
                rc = build_tile_schedule(order, lens, kTileFixedCost, n_tt, static_cast<int>(sw), h->n_ctas, &sc);
            } else if (!rc) {
                rc = build_bcsr_schedule(f, n_tt, static_cast<int>(sw), h->dynamic ? 1 : h->n_ctas, &sc);
            }
        } else {
            // The row groups get a launch and a schedule of their own; the launch of the remaining
            // block-rows starts on the SMs the first one leaves idle, CTA after CTA as they free up.
            // CTAs are dispatched in index order, so CTA j of the second launch starts when the
            // j-th lightest CTA of the first one is done: its list is dealt with that head start.
            const int bnt_s = 128 * kStackGroups;
            const int n_tt_s = static_cast<int>((N + bnt_s - 1) / bnt_s);
            int64_t sws = slab_cols / bnt_s;
            if (sws < 1) sws = 1;
            if (sws > n_tt_s) sws = n_tt_s;
            std::vector<int32_t> units, lens;
            for (int64_t g = 0; g < st.ng; ++g) {
                units.push_back(static_cast<int32_t>(g));
                lens.push_back(st.ptr[g + 1] - st.ptr[g]);
            }
            std::vector<int64_t> loads;
            rc = build_tile_schedule(units, lens, kStackTileFixedCost, n_tt_s, static_cast<int>(sws), h->n_ctas, &ss,
                                     bcsr_stack_block_cost(), nullptr, &loads);
            ss.groups = kStackGroups;
            ss.N = N;
            if (!rc) {
                std::sort(loads.begin(), loads.end());
                units.clear();
                lens.clear();
                for (int64_t r = 0; r < f.nbr; ++r) {
                    const int32_t I = f.row_order[r];
                    if (st.stacked[I]) continue;
                    units.push_back(I);
                    lens.push_back(f.block_row_ptr[I + 1] - f.block_row_ptr[I]);
                }
                rc = build_tile_schedule(units, lens, kTileFixedCost, n_tt, static_cast<int>(sw), h->n_ctas, &sc,
                                         bcsr_block_cost(f.b, groups), &loads);
            }
        }
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) return rc;
    sc.groups = groups;
    sc.N = N;
    if (!h->host_only) {
        if (h->d_tiles) {   // a previous schedule may still be in use by a running kernel
            if (cudaDeviceSynchronize() != cudaSuccess) return SPMM_ERR_CUDA;
            cudaFree(h->d_tiles);
            cudaFree(h->d_tile_recs);
            cudaFree(h->d_cta_ptr);
            cudaFree(h->d_stile_recs);
            cudaFree(h->d_scta_ptr);
            cudaFree(h->d_kmerge);
            h->d_tiles = h->d_tile_recs = h->d_cta_ptr = h->d_stile_recs = h->d_scta_ptr = h->d_kmerge = nullptr;
            h->n_kmerge = 0;
            h->tmP_ok = false;
        }
        rc = upload(&h->d_tiles, sc.tiles.data(), sc.tiles.size() * 4);
        if (!rc) {
            // self-contained records, so that a role needs one load per tile (and can fetch it a tile ahead)
            const size_t nt = sc.tiles.size() / 2;
            std::vector<int32_t> recs(4 * nt);
            for (size_t i = 0; i < nt; ++i) {
                recs[4 * i + 1] = sc.tiles[2 * i + 1];
                if (sc.units.empty()) {
                    const int32_t I = sc.tiles[2 * i];
                    recs[4 * i] = I;
                    recs[4 * i + 2] = f.block_row_ptr[I];
                    recs[4 * i + 3] = f.block_row_ptr[I + 1];
                } else {
                    // K-split: the tile names a unit {block-row, first block, end block, slot}; a part
                    // carries -1 - slot in place of the block-row
                    const int32_t* u = &sc.units[4 * static_cast<size_t>(sc.tiles[2 * i])];
                    recs[4 * i] = u[3] < 0 ? u[0] : -1 - u[3];
                    recs[4 * i + 2] = u[1];
                    recs[4 * i + 3] = u[2];
                }
            }
            rc = upload(&h->d_tile_recs, recs.data(), recs.size() * 4);
        }
        if (!rc && sc.n_slots > 0) {
            // merge lists (split block-rows in ascending order: their slots are consecutive), the
            // partial tiles' workspace and its store map
            // (the parts of a block-row are consecutive units, in part order)
            std::vector<int32_t> rows, firsts, parts;
            for (size_t u = 0; u < sc.units.size() / 4; ++u) {
                const int32_t I = sc.units[4 * u], slot = sc.units[4 * u + 3];
                if (slot < 0) continue;
                if (rows.empty() || rows.back() != I) { rows.push_back(I); firsts.push_back(slot); parts.push_back(0); }
                parts.back()++;
            }
            std::vector<int32_t> mg;
            mg.insert(mg.end(), rows.begin(), rows.end());
            mg.insert(mg.end(), firsts.begin(), firsts.end());
            mg.insert(mg.end(), parts.begin(), parts.end());
            h->n_kmerge = static_cast<int>(rows.size());
            rc = upload(&h->d_kmerge, mg.data(), mg.size() * 4);
            const size_t need = static_cast<size_t>(sc.n_slots) * f.b * static_cast<size_t>(N) * 4;
            if (!rc && need > h->partial_bytes) {
                cudaFree(h->d_partial);
                h->d_partial = nullptr;
                h->partial_bytes = 0;
                if (cudaMalloc(reinterpret_cast<void**>(&h->d_partial), need) != cudaSuccess) rc = SPMM_ERR_ALLOC;
                else h->partial_bytes = need;
            }
            if (!rc) {
                EncodeTiledFn fn = get_encode_fn();
                const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(sc.n_slots) * f.b};
                const cuuint64_t strides[1] = {static_cast<cuuint64_t>(N) * 4};
                const cuuint32_t box[2] = {32, static_cast<cuuint32_t>(bcsr_epi_cols(f.b, false, false))};
                const cuuint32_t estr[2] = {1, 1};
                if (!fn || fn(&h->tmP, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, h->d_partial, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                    rc = SPMM_ERR_CUDA;
                else
                    h->tmP_ok = true;
            }
        }
        if (!rc) rc = upload(&h->d_cta_ptr, sc.cta_ptr.data(), sc.cta_ptr.size() * 4);
        if (!rc && !ss.tiles.empty()) {
            const size_t nt = ss.tiles.size() / 2;
            std::vector<int32_t> recs(4 * nt);
            for (size_t i = 0; i < nt; ++i) {
                const int32_t g = ss.tiles[2 * i];
                recs[4 * i] = g;
                recs[4 * i + 1] = ss.tiles[2 * i + 1];
                recs[4 * i + 2] = st.ptr[g];
                recs[4 * i + 3] = st.ptr[g + 1];
            }
            rc = upload(&h->d_stile_recs, recs.data(), recs.size() * 4);
            if (!rc) rc = upload(&h->d_scta_ptr, ss.cta_ptr.data(), ss.cta_ptr.size() * 4);
        }
        if (rc) return rc;
    }
    h->sched_stack = std::move(ss);
    h->sched = std::move(sc);
    return SPMM_OK;
}

int run_bcsr(spmm_handle_s* h, const void* B, void* C, int64_t N, cudaStream_t stream) {
    const BcsrHost& f = h->bcsr;
    // the box of the dense operand is 64 tokens wide (128 with column-major operands or 1-byte values)
    if (N < ((h->col_major || h->es == 1) ? 128 : 64)) return SPMM_ERR_UNSUPPORTED;
    if (f.nbr == 0) return SPMM_OK;
    int rc = ensure_schedule(h, N);
    if (rc) return rc;
    BcsrParams p;
    p.block_row_ptr = h->d_ptr;
    p.block_col_idx = h->d_idx;
    p.tiles = reinterpret_cast<const int4*>(h->d_tile_recs);
    p.cta_ptr = h->d_cta_ptr;
    p.C = C;
    p.m = h->m;
    p.N = N;
    p.status = h->d_status;
    p.wait_limit_ns = g_wait_limit_ns.load();
    p.stack_rows = nullptr;
    p.overlap = 0;
    CUtensorMap tmA = h->tmA;
    if (!h->tmA_ok) {
        // no stored block at all: the kernel never touches A, any valid map will do
        rc = encode_2d(&tmA, h->dtype, h->d_vals, 8, 8, 8, 8, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (rc) return rc;
    }
    rc = ensure_tmB(h, B, N, h->sched.groups);
    if (rc) return rc;
    p.use_3d = h->tmB3_ok ? 1 : 0;
    rc = ensure_tmC(h, C, N);
    if (rc) return rc;
    if (!h->sched_stack.tiles.empty()) {
        // the row groups first (the longest block-rows are among them), then everything else
        BcsrParams ps = p;
        ps.block_col_idx = h->d_sidx;
        ps.tiles = reinterpret_cast<const int4*>(h->d_stile_recs);
        ps.cta_ptr = h->d_scta_ptr;
        ps.stack_rows = h->d_srows;
        ps.use_3d = h->tmB3s_ok ? 1 : 0;
        ps.overlap = 1;
        p.overlap = 2;
        cudaError_t es = launch_bcsr_stacked(h->dtype, f.b, h->c16, h->col_major, h->tmAs, h->tmB, h->tmB3s, h->tmC, h->tmC, ps,
                                             h->n_ctas, stream);
        if (es != cudaSuccess) return SPMM_ERR_CUDA;
        if (h->sched.tiles.empty()) return SPMM_OK;
    }
    // dynamic: one CTA per tile, the schedule was built as a single list in the global order
    const int grid = h->dynamic ? static_cast<int>(h->sched.tiles.size() / 2) : h->n_ctas;
    if (grid <= 0) return SPMM_OK;
    const bool ksplit = h->sched.n_slots > 0 && h->tmP_ok;
    if (ksplit) p.overlap = 1;          // the merge kernel's CTAs may be placed while this grid runs
    cudaError_t e = launch_bcsr(h->dtype, f.b, h->sched.groups, h->c16, h->col_major, h->dynamic, tmA, h->tmB, h->tmB3,
                                h->tmC, ksplit ? h->tmP : h->tmC, p, grid, stream);
    if (e != cudaSuccess) return SPMM_ERR_CUDA;
    if (ksplit) {
        BcsrMergeParams mp;
        mp.row = h->d_kmerge;
        mp.first = h->d_kmerge + h->n_kmerge;
        mp.nparts = h->d_kmerge + 2 * h->n_kmerge;
        mp.partial = h->d_partial;
        mp.C = static_cast<float*>(C);
        mp.m = h->m;
        mp.N = N;
        mp.n = h->n_kmerge;
        mp.b = f.b;
        if (launch_bcsr_merge(mp, stream) != cudaSuccess) return SPMM_ERR_CUDA;
    }
    return SPMM_OK;
}

int64_t wcsr_workspace_bytes(const spmm_handle_s* h, int64_t N) {
    return h->wcsr.n_slots * int64_t{h->wcsr.wh} * N * 4;
}

int launch_wcsr_all(spmm_handle_s* h, const void* B, void* C, float* partial, int64_t N, cudaStream_t stream) {
    const WcsrHost& f = h->wcsr;
    const int bnt = 128;                    // tokens per tile; wider B takes one pass per tile
    WcsrParams p;
    p.bin_ptr = h->d_bin_ptr;
    p.items = reinterpret_cast<const int4*>(h->d_items);
    // narrow dense operand: the variant whose stages hold more columns
    const bool narrow = h->d_bin_fill_narrow != nullptr && N <= kWcsrNarrowMaxN && !h->lsu_gather;
    p.fills = reinterpret_cast<const int2*>(narrow ? h->d_fills_narrow : h->d_fills);
    p.bin_fill = narrow ? h->d_bin_fill_narrow : h->d_bin_fill;
    p.col_idx = h->d_idx;
    // Gather hints: B rows whose reuse class fits half of a 126 MB L2 at this dense width are
    // fetched evict-last, everything else evict-first.  Class c holds at most
    // kWcsrTopClassRows << (7 - c) rows of N * es bytes each.
    p.grp_class = h->lsu_gather ? nullptr : h->d_grp_class;
    p.hot_min = 8;
    for (int c = 1; c <= 7; ++c)
        if ((static_cast<int64_t>(kWcsrTopClassRows) << (7 - c)) * N * h->es <= (int64_t{64} << 20)) { p.hot_min = c; break; }
    // (measured on the R-MAT configuration at N = 128: DRAM reads 2.84 -> 2.53 GB, L2 sector hit rate
    // 50 -> 53 %, time unchanged -- the kernel is bound by the latency of its gathers, not by DRAM
    // bytes; storing C evict-first as well measured 1 - 5 % slower and is left off)
    p.hint_flags = 1;
    p.packed = h->d_vals;
    p.B = B;
    p.C = C;
    p.partial = partial;
    p.m = h->m;
    p.N = N;
    p.n_bins = static_cast<int32_t>(f.bin_ptr.size()) - 1;
    p.n_tt = static_cast<int32_t>((N + bnt - 1) / bnt);
    p.status = h->d_status;
    p.wait_limit_ns = g_wait_limit_ns.load();
    if (!f.tasks.empty()) {
        int rc = ensure_tmB(h, B, N, 1);
        if (rc) return rc;
        cudaError_t e = launch_wcsr(h->dtype, f.wh, h->c16, narrow ? 1 : 0, h->lsu_gather ? 1 : 0, h->tmB, p, h->sms, stream);
        if (e != cudaSuccess) return SPMM_ERR_CUDA;
    }
    MergeParams mp;
    mp.window = h->d_merge;
    mp.first = h->d_merge + h->n_merge;
    mp.nparts = h->d_merge + 2 * h->n_merge;
    mp.partial = partial;
    mp.C = C;
    mp.m = h->m;
    mp.N = N;
    mp.n = h->n_merge;
    cudaError_t e = launch_wcsr_merge(mp, f.wh, h->c16 ? (h->dtype == SPMM_FP16 ? 1 : 2) : 0, stream);
    return e == cudaSuccess ? SPMM_OK : SPMM_ERR_CUDA;
}

// The handle's workspace for the partial tiles of split windows at dense width N (grown, never shrunk).
int ensure_wcsr_workspace(spmm_handle_s* h, int64_t N) {
    const size_t need = static_cast<size_t>(wcsr_workspace_bytes(h, N));
    if (need > h->partial_bytes) {
        if (h->d_partial) {
            if (cudaDeviceSynchronize() != cudaSuccess) return SPMM_ERR_CUDA;
            cudaFree(h->d_partial);
            h->d_partial = nullptr;
            h->partial_bytes = 0;
        }
        if (cudaMalloc(reinterpret_cast<void**>(&h->d_partial), need) != cudaSuccess) return SPMM_ERR_ALLOC;
        h->partial_bytes = need;
    }
    return SPMM_OK;
}

int run_wcsr(spmm_handle_s* h, const void* B, void* C, int64_t N, cudaStream_t stream) {
    if (int rc = ensure_wcsr_workspace(h, N)) return rc;
    return launch_wcsr_all(h, B, C, h->d_partial, N, stream);
}

int check_run_args(spmm_handle_s* h, const void* B, const void* C, int64_t N) {
    if (!h || !B || !C || N <= 0) return SPMM_ERR_INVALID_ARG;
    if (h->host_only) return SPMM_ERR_HOST_ONLY;
    // the handle's arrays, tensor maps and kernel attributes belong to the device it was created on
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPMM_ERR_CUDA;
    if (dev != h->device) return SPMM_ERR_INVALID_ARG;
    // row-major B and C have N elements per row: rows must stay 16-byte aligned (column-major
    // operands have k and m elements per row, checked at creation)
    if (!h->col_major && (N * h->es) % 16 != 0) return SPMM_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(B) & 15) || (reinterpret_cast<uintptr_t>(C) & 15)) return SPMM_ERR_UNSUPPORTED;
    if (N >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    return SPMM_OK;
}

}  // namespace

// ============================================================================= C ABI

extern "C" {

int spmm_bcsr_create_csr(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* row_ptr, const int32_t* col_idx,
                         const void* vals, int dtype, int block, const spmm_opts_t* opts) {
    NvtxRange nvtx_range("spmm_bcsr_create_csr");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    CsrView v;
    int rc = make_view(&v, m, k, row_ptr, col_idx, vals, dtype);
    if (rc) return rc;
    return create_bcsr(out, v, dtype, block, opts);
}

int spmm_bcsr_create_csr_device(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* row_ptr_dev,
                                const int32_t* col_idx_dev, const void* vals_dev, int dtype, int block,
                                const spmm_opts_t* opts, void* stream) {
    NvtxRange nvtx_range("spmm_bcsr_create_csr_device");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    if (dtype < 0 || dtype > 3 || m < 0 || k < 0 || !row_ptr_dev) return SPMM_ERR_INVALID_ARG;
    if (m >= (int64_t{1} << 31) || k >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    return create_bcsr_device(out, m, k, row_ptr_dev, col_idx_dev, vals_dev, dtype, block, opts, static_cast<cudaStream_t>(stream));
}

int spmm_wcsr_create_csr_device(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* row_ptr_dev,
                                const int32_t* col_idx_dev, const void* vals_dev, int dtype, int window_height,
                                const spmm_opts_t* opts, void* stream) {
    NvtxRange nvtx_range("spmm_wcsr_create_csr_device");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    if (dtype < 0 || dtype > 3 || m < 0 || k < 0 || !row_ptr_dev) return SPMM_ERR_INVALID_ARG;
    if (m >= (int64_t{1} << 31) || k >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    return create_wcsr_device(out, m, k, row_ptr_dev, col_idx_dev, vals_dev, dtype, window_height, opts, static_cast<cudaStream_t>(stream));
}

int spmm_bcsr_create_coo(spmm_handle_t* out, int64_t m, int64_t k, int64_t nnz, const int32_t* rows,
                         const int32_t* cols, const void* vals, int dtype, int block, const spmm_opts_t* opts) {
    NvtxRange nvtx_range("spmm_bcsr_create_coo");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    if (dtype < 0 || dtype > 3) return SPMM_ERR_INVALID_ARG;
    CsrOwned o;
    int rc;
    try {
        rc = coo_to_csr(m, k, nnz, rows, cols, static_cast<const uint8_t*>(vals), elem_size(dtype), &o);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) return rc;
    return spmm_bcsr_create_csr(out, m, k, o.row_ptr.data(), o.col_idx.data(), o.vals.data(), dtype, block, opts);
}

int spmm_wcsr_create_csr(spmm_handle_t* out, int64_t m, int64_t k, const int64_t* row_ptr, const int32_t* col_idx,
                         const void* vals, int dtype, int window_height, const spmm_opts_t* opts) {
    NvtxRange nvtx_range("spmm_wcsr_create_csr");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    CsrView v;
    int rc = make_view(&v, m, k, row_ptr, col_idx, vals, dtype);
    if (rc) return rc;
    return create_wcsr(out, v, dtype, window_height, opts);
}

int spmm_wcsr_create_coo(spmm_handle_t* out, int64_t m, int64_t k, int64_t nnz, const int32_t* rows,
                         const int32_t* cols, const void* vals, int dtype, int window_height,
                         const spmm_opts_t* opts) {
    NvtxRange nvtx_range("spmm_wcsr_create_coo");
    if (!out) return SPMM_ERR_INVALID_ARG;
    *out = nullptr;
    if (dtype < 0 || dtype > 3) return SPMM_ERR_INVALID_ARG;
    CsrOwned o;
    int rc;
    try {
        rc = coo_to_csr(m, k, nnz, rows, cols, static_cast<const uint8_t*>(vals), elem_size(dtype), &o);
    } catch (const std::bad_alloc&) {
        rc = SPMM_ERR_ALLOC;
    }
    if (rc) return rc;
    return spmm_wcsr_create_csr(out, m, k, o.row_ptr.data(), o.col_idx.data(), o.vals.data(), dtype, window_height,
                                opts);
}

int spmm_run(spmm_handle_t h, const void* B_dev, void* C_dev, int64_t N, void* stream) {
    NvtxRange nvtx_range("spmm_run");
    int rc = check_run_args(h, B_dev, C_dev, N);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (h->format == 0) return run_bcsr(h, B_dev, C_dev, N, st);
    return run_wcsr(h, B_dev, C_dev, N, st);
}

int spmm_bcsr_plan(spmm_handle_t h, int64_t N) {
    NvtxRange nvtx_range("spmm_bcsr_plan");
    if (!h || N <= 0) return SPMM_ERR_INVALID_ARG;
    if (h->format != 0) return SPMM_ERR_INVALID_ARG;
    if (N < ((h->col_major || h->es == 1) ? 128 : 64) || (!h->col_major && (N * h->es) % 16 != 0)) return SPMM_ERR_UNSUPPORTED;
    return ensure_schedule(h, N);
}

int spmm_prepare(spmm_handle_t h, int64_t N) {
    NvtxRange nvtx_range("spmm_prepare");
    if (!h || N <= 0) return SPMM_ERR_INVALID_ARG;
    if (h->format == 0) return spmm_bcsr_plan(h, N);
    if ((N * h->es) % 16 != 0) return SPMM_ERR_UNSUPPORTED;
    if (N >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
    if (h->host_only) return SPMM_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPMM_ERR_CUDA;
    if (dev != h->device) return SPMM_ERR_INVALID_ARG;
    return ensure_wcsr_workspace(h, N);
}

int spmm_wcsr_run_static(spmm_handle_t h, const void* B_dev, void* C_dev, int64_t N, void* stream) {
    NvtxRange nvtx_range("spmm_wcsr_run_static");
    int rc = check_run_args(h, B_dev, C_dev, N);
    if (rc) return rc;
    if (h->format != 1) return SPMM_ERR_INVALID_ARG;
    float* scratch = nullptr;
    size_t cap = 0;
    if (wcsr_static_scratch(&scratch, &cap) != cudaSuccess) return SPMM_ERR_CUDA;
    if (static_cast<size_t>(wcsr_workspace_bytes(h, N)) > cap) return SPMM_ERR_TOO_LARGE;
    return launch_wcsr_all(h, B_dev, C_dev, scratch, N, static_cast<cudaStream_t>(stream));
}

int spmm_run_host(spmm_handle_t h, const void* B_host, void* C_host, int64_t N, void* stream) {
    NvtxRange nvtx_range("spmm_run_host");
    if (!h || !B_host || !C_host || N <= 0) return SPMM_ERR_INVALID_ARG;
    if (h->host_only) return SPMM_ERR_HOST_ONLY;
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) return SPMM_ERR_CUDA;
        if (dev != h->device) return SPMM_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bbytes = static_cast<size_t>(h->k) * N * h->es;
    const size_t cbytes = static_cast<size_t>(h->m) * N * h->cs;
    if (bbytes > h->Bstage_bytes) {
        cudaFree(h->d_Bstage);
        h->d_Bstage = nullptr;
        h->Bstage_bytes = 0;
        if (cudaMalloc(&h->d_Bstage, bbytes ? bbytes : 16) != cudaSuccess) return SPMM_ERR_ALLOC;
        h->Bstage_bytes = bbytes;
    }
    if (cbytes > h->Cstage_bytes) {
        cudaFree(h->d_Cstage);
        h->d_Cstage = nullptr;
        h->Cstage_bytes = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&h->d_Cstage), cbytes ? cbytes : 16) != cudaSuccess) return SPMM_ERR_ALLOC;
        h->Cstage_bytes = cbytes;
    }
    // Large operands go in column chunks (token chunks), so that the copy of one chunk's result to
    // the host overlaps the copy of the next chunk's operand to the device (the two directions of
    // the link are independent) and the kernels in between.  Chunks are whole slices of N that the
    // kernels accept by themselves; each is staged as its own contiguous array, so the kernels
    // run unchanged on it.  Row-major operands: a chunk is a column range, copied with 2-D
    // copies whose rows are at least 256 bytes; column-major: a contiguous range of tokens.
    int nchunks = 1;
    if (bbytes + cbytes >= (size_t{8} << 20)) {
        for (int c = spmm_handle_s::kMaxHostChunks; c >= 2; c >>= 1) {
            if (N % c != 0) continue;
            const int64_t nc = N / c;
            const bool ok = h->col_major ? (nc >= 128)
                                         : (nc * h->es >= 256 && (nc * h->es) % 16 == 0 && (nc * h->cs) % 16 == 0 &&
                                            (h->format == 1 || nc >= 64));
            if (ok) { nchunks = c; break; }
        }
    }
    if (nchunks == 1) {
        if (cudaMemcpyAsync(h->d_Bstage, B_host, bbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SPMM_ERR_CUDA;
        int rc = spmm_run(h, h->d_Bstage, h->d_Cstage, N, stream);
        if (rc) return rc;
        if (cudaMemcpyAsync(C_host, h->d_Cstage, cbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPMM_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return SPMM_ERR_CUDA;
        return SPMM_OK;
    }
    if (!h->s_in) {
        if (cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) != cudaSuccess)
            return SPMM_ERR_CUDA;
        for (int i = 0; i < spmm_handle_s::kMaxHostChunks; ++i)
            if (cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&h->ev_run[i], cudaEventDisableTiming) != cudaSuccess)
                return SPMM_ERR_CUDA;
    }
    const int64_t nc = N / nchunks;
    const size_t bchunk = bbytes / nchunks, cchunk = cbytes / nchunks;
    const uint8_t* Bh = static_cast<const uint8_t*>(B_host);
    uint8_t* Chost = static_cast<uint8_t*>(C_host);
    uint8_t* dB = static_cast<uint8_t*>(h->d_Bstage);
    uint8_t* dC = reinterpret_cast<uint8_t*>(h->d_Cstage);
    bool bad = false;
    // the staging buffers may still be read by work queued on `stream` earlier
    bad |= cudaEventRecord(h->ev_start, st) != cudaSuccess;
    bad |= cudaStreamWaitEvent(h->s_in, h->ev_start, 0) != cudaSuccess;
    for (int c = 0; c < nchunks && !bad; ++c) {
        if (h->col_major)
            bad |= cudaMemcpyAsync(dB + c * bchunk, Bh + c * bchunk, bchunk, cudaMemcpyHostToDevice, h->s_in) != cudaSuccess;
        else
            bad |= cudaMemcpy2DAsync(dB + c * bchunk, nc * h->es, Bh + static_cast<size_t>(c) * nc * h->es, N * h->es, nc * h->es,
                                     static_cast<size_t>(h->k), cudaMemcpyHostToDevice, h->s_in) != cudaSuccess;
        bad |= cudaEventRecord(h->ev_in[c], h->s_in) != cudaSuccess;
    }
    int rc = SPMM_OK;
    for (int c = 0; c < nchunks && !bad && !rc; ++c) {
        bad |= cudaStreamWaitEvent(st, h->ev_in[c], 0) != cudaSuccess;
        if (bad) break;
        rc = spmm_run(h, dB + c * bchunk, dC + c * cchunk, nc, stream);
        if (rc) break;
        bad |= cudaEventRecord(h->ev_run[c], st) != cudaSuccess;
        bad |= cudaStreamWaitEvent(h->s_out, h->ev_run[c], 0) != cudaSuccess;
        if (h->col_major)
            bad |= cudaMemcpyAsync(Chost + c * cchunk, dC + c * cchunk, cchunk, cudaMemcpyDeviceToHost, h->s_out) != cudaSuccess;
        else
            bad |= cudaMemcpy2DAsync(Chost + static_cast<size_t>(c) * nc * h->cs, N * h->cs, dC + c * cchunk, nc * h->cs, nc * h->cs,
                                     static_cast<size_t>(h->m), cudaMemcpyDeviceToHost, h->s_out) != cudaSuccess;
    }
    // nothing of this call may still be in flight when it returns, whatever happened above
    const bool s1 = cudaStreamSynchronize(h->s_in) == cudaSuccess;
    const bool s2 = cudaStreamSynchronize(st) == cudaSuccess;
    const bool s3 = cudaStreamSynchronize(h->s_out) == cudaSuccess;
    if (rc) return rc;
    return (bad || !s1 || !s2 || !s3) ? SPMM_ERR_CUDA : SPMM_OK;
}

int spmm_check(spmm_handle_t h) {
    if (!h) return SPMM_ERR_INVALID_ARG;
    if (h->host_only) return SPMM_ERR_HOST_ONLY;
    int st[4] = {0, 0, 0, 0};
    if (cudaMemcpy(st, h->d_status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return SPMM_ERR_CUDA;
    if (st[0] != 0) {
        cudaMemset(h->d_status, 0, sizeof(st));
        if (st[0] == 2) return SPMM_ERR_DEV_BOUNDS;
        return st[3] != 0 ? SPMM_ERR_DEV_UNDRAINED : SPMM_ERR_DEV_TIMEOUT;
    }
    return SPMM_OK;
}

int spmm_get_info(spmm_handle_t h, int64_t N, spmm_info_t* info) {
    if (!h || !info || N < 0) return SPMM_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof(*info));
    info->format = h->format;
    info->dtype = h->dtype;
    info->m = h->m;
    info->k = h->k;
    info->nnz = h->nnz;
    info->n_ctas = h->n_ctas;
    const double s = h->es, n = static_cast<double>(N);
    if (h->format == 0) {
        const BcsrHost& f = h->bcsr;
        info->block = f.b;
        info->n_units = f.nnzb;
        info->stored_values = f.nnzb * f.b * f.b;
        info->n_rows_units = f.nbr;
        info->n_empty = f.n_empty;
        int64_t rows_touched = f.distinct_bcols * f.b;
        if (rows_touched > h->k) rows_touched = h->k;
        info->distinct_b_rows = rows_touched;
        info->bytes_a = static_cast<double>(info->stored_values) * s;
        info->bytes_idx = static_cast<double>(f.nbr + 1 + f.nnzb) * 4.0;
        info->bytes_gather = static_cast<double>(f.nnzb) * f.b * n * s;
        info->n_stacked_rows = static_cast<int32_t>(h->stack.rows.size());
        info->n_stack_blocks = h->stack.ns;
        if (h->sched.N >= 0) {
            info->n_slots = h->sched.n_slots;
            info->n_split = h->n_kmerge;
            if (h->host_only && h->sched.n_slots > 0) {
                int64_t ns = 0, last = -1;
                for (size_t u = 0; u < h->sched.units.size() / 4; ++u)
                    if (h->sched.units[4 * u + 3] >= 0 && h->sched.units[4 * u] != last) { last = h->sched.units[4 * u]; ++ns; }
                info->n_split = ns;
            }
            info->n_tasks = static_cast<int64_t>(h->sched.units.size() / 4);
            info->split_cols = h->sched.cap;
            info->workspace_bytes = h->sched.n_slots * f.b * h->sched.N * 4;
            info->plan_n = h->sched.N;
            info->plan_token_tile = 128 * h->sched.groups;
            info->plan_slab_tiles = h->sched.slab_w;
        }
    } else {
        const WcsrHost& f = h->wcsr;
        info->block = f.wh;
        info->b_col = f.b_col;
        info->n_units = f.P;
        info->stored_values = f.P * f.wh;
        info->n_rows_units = f.nwin;
        info->n_empty = f.n_empty;
        info->n_tasks = static_cast<int64_t>(f.tasks.size());
        info->n_split = f.n_split;
        info->n_slots = f.n_slots;
        info->split_cols = f.T;
        info->n_bins = static_cast<int32_t>(f.bin_ptr.size()) - 1;
        info->distinct_b_rows = f.distinct_cols;
        info->bytes_a = static_cast<double>(info->stored_values) * s;
        info->bytes_idx = static_cast<double>(f.nwin + 1 + f.P) * 4.0;
        info->bytes_gather = static_cast<double>(f.P) * n * s;
        info->workspace_bytes = wcsr_workspace_bytes(h, N);
    }
    info->fill_ratio = info->stored_values ? static_cast<double>(h->nnz) / static_cast<double>(info->stored_values) : 0.0;
    info->bytes_b_touched = static_cast<double>(info->distinct_b_rows) * n * s;
    info->bytes_c = static_cast<double>(h->m) * n * h->cs;
    info->flops_stored = 2.0 * static_cast<double>(info->stored_values) * n;
    return SPMM_OK;
}

int spmm_export(spmm_handle_t h, int which, void* host_dst, size_t cap, size_t* need) {
    if (!h || !need) return SPMM_ERR_INVALID_ARG;
    const void* dev_src = nullptr;    // device array in canonical layout, or
    const void* host_src = nullptr;   // host array in canonical layout
    size_t bytes = 0;
    bool unpack_wcsr = false;
    bool host_copy = false;           // the array is kept on the host even when the handle is on the device
    std::vector<int32_t> tmp;
    if (h->format == 0) {
        const BcsrHost& f = h->bcsr;
        switch (which) {
            case SPMM_X_BCSR_BLOCK_ROW_PTR: bytes = f.block_row_ptr.size() * 4; dev_src = h->d_ptr; host_src = f.block_row_ptr.data(); break;
            case SPMM_X_BCSR_BLOCK_COL_IDX: bytes = f.block_col_idx.size() * 4; dev_src = h->d_idx; host_src = f.block_col_idx.data(); break;
            case SPMM_X_BCSR_BLOCKS: bytes = static_cast<size_t>(f.nnzb) * f.b * f.b * h->es; dev_src = h->d_vals; host_src = f.blocks.data(); break;
            case SPMM_X_BCSR_ROW_ORDER: bytes = f.row_order.size() * 4; dev_src = h->d_order; host_src = f.row_order.data(); break;
            case SPMM_X_BCSR_TILE_PTR:
                if (h->sched.N < 0) return SPMM_ERR_INVALID_ARG;
                bytes = h->sched.cta_ptr.size() * 4; dev_src = h->d_cta_ptr; host_src = h->sched.cta_ptr.data(); break;
            case SPMM_X_BCSR_TILES:
                if (h->sched.N < 0) return SPMM_ERR_INVALID_ARG;
                bytes = h->sched.tiles.size() * 4; dev_src = h->d_tiles; host_src = h->sched.tiles.data(); break;
            case SPMM_X_BCSR_UNITS:
                if (h->sched.N < 0) return SPMM_ERR_INVALID_ARG;
                bytes = h->sched.units.size() * 4; host_src = h->sched.units.data(); host_copy = true; break;
            // the row-group plan lives on the host in every mode
            case SPMM_X_BCSR_STACK_ROWS: bytes = h->stack.rows.size() * 4; host_src = h->stack.rows.data(); host_copy = true; break;
            case SPMM_X_BCSR_STACK_PTR: bytes = h->stack.ptr.size() * 4; host_src = h->stack.ptr.data(); host_copy = true; break;
            case SPMM_X_BCSR_STACK_COL_IDX: bytes = h->stack.col_idx.size() * 4; host_src = h->stack.col_idx.data(); host_copy = true; break;
            case SPMM_X_BCSR_STACK_TILE_PTR:
                if (h->sched.N < 0) return SPMM_ERR_INVALID_ARG;
                bytes = h->sched_stack.cta_ptr.size() * 4; host_src = h->sched_stack.cta_ptr.data(); host_copy = true; break;
            case SPMM_X_BCSR_STACK_TILES:
                if (h->sched.N < 0) return SPMM_ERR_INVALID_ARG;
                bytes = h->sched_stack.tiles.size() * 4; host_src = h->sched_stack.tiles.data(); host_copy = true; break;
            default: return SPMM_ERR_INVALID_ARG;
        }
    } else {
        const WcsrHost& f = h->wcsr;
        switch (which) {
            case SPMM_X_WCSR_WINDOW_ROW_PTR: bytes = f.window_row_ptr.size() * 4; dev_src = h->d_ptr; host_src = f.window_row_ptr.data(); break;
            case SPMM_X_WCSR_WINDOW_COL_IDX: bytes = static_cast<size_t>(f.P) * 4; dev_src = h->d_idx; host_src = f.window_col_idx.data(); break;
            case SPMM_X_WCSR_VALUES: bytes = static_cast<size_t>(f.P) * f.wh * h->es; unpack_wcsr = true; break;
            case SPMM_X_WCSR_TASKS: bytes = f.tasks.size() * 16; break;
            case SPMM_X_WCSR_BIN_PTR: bytes = f.bin_ptr.size() * 4; dev_src = h->d_bin_ptr; host_src = f.bin_ptr.data(); break;
            case SPMM_X_WCSR_BIN_TASKS: bytes = f.bin_tasks.size() * 4; dev_src = h->d_bin_tasks; host_src = f.bin_tasks.data(); break;
            case SPMM_X_WCSR_GROUP_CLASS: bytes = static_cast<size_t>(f.P / 4); dev_src = h->d_grp_class; host_src = f.grp_class.data(); break;
            default: return SPMM_ERR_INVALID_ARG;
        }
    }
    *need = bytes;
    if (!host_dst) return SPMM_OK;
    if (cap < bytes) return SPMM_ERR_INVALID_ARG;
    if (bytes == 0) return SPMM_OK;
    if (unpack_wcsr) {
        const WcsrHost& f = h->wcsr;
        std::vector<uint8_t> packed_dl;
        const uint8_t* packed = f.packed.data();
        if (!h->host_only) {
            packed_dl.resize(bytes);
            if (cudaMemcpy(packed_dl.data(), h->d_vals, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return SPMM_ERR_CUDA;
            packed = packed_dl.data();
        }
        uint8_t* dst = static_cast<uint8_t*>(host_dst);
        for (int r = 0; r < f.wh; ++r)
            for (int64_t q = 0; q < f.P; ++q)
                std::memcpy(dst + (static_cast<size_t>(r) * f.P + q) * h->es,
                            packed + wcsr_packed_offset(f.wh, f.b_col, h->es, r, q), h->es);
        return SPMM_OK;
    }
    if (h->format == 1 && which == SPMM_X_WCSR_TASKS) {
        const WcsrHost& f = h->wcsr;
        int32_t* dst = static_cast<int32_t*>(host_dst);
        if (h->host_only) {
            for (size_t i = 0; i < f.tasks.size(); ++i) {
                dst[4 * i + 0] = f.tasks[i].window;
                dst[4 * i + 1] = f.tasks[i].q0;
                dst[4 * i + 2] = f.tasks[i].count;
                dst[4 * i + 3] = f.tasks[i].slot;
            }
        } else {
            std::vector<WcsrDevTask> dt(f.tasks.size());
            if (cudaMemcpy(dt.data(), h->d_tasks, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return SPMM_ERR_CUDA;
            for (size_t i = 0; i < dt.size(); ++i) {
                dst[4 * i + 0] = dt[i].window;
                dst[4 * i + 1] = dt[i].col_begin - f.window_row_ptr[dt[i].window];
                dst[4 * i + 2] = dt[i].count;
                dst[4 * i + 3] = dt[i].slot;
            }
        }
        return SPMM_OK;
    }
    if (h->host_only || host_copy) {
        std::memcpy(host_dst, host_src, bytes);
        return SPMM_OK;
    }
    return cudaMemcpy(host_dst, dev_src, bytes, cudaMemcpyDeviceToHost) == cudaSuccess ? SPMM_OK : SPMM_ERR_CUDA;
}

int spmm_destroy(spmm_handle_t h) {
    free_handle(h);
    return SPMM_OK;
}

const char* spmm_status_string(int code) {
    switch (code) {
        case SPMM_OK: return "ok";
        case SPMM_ERR_INVALID_ARG: return "invalid argument";
        case SPMM_ERR_UNSORTED: return "unsorted or duplicate entries";
        case SPMM_ERR_OUT_OF_RANGE: return "index out of range";
        case SPMM_ERR_UNSUPPORTED: return "unsupported size, dtype, alignment or device";
        case SPMM_ERR_ALLOC: return "allocation failed";
        case SPMM_ERR_CUDA: return "CUDA call failed (is there a B200 and a usable context?)";
        case SPMM_ERR_DEV_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case SPMM_ERR_HOST_ONLY: return "handle was created host_only";
        case SPMM_ERR_TOO_LARGE: return "size exceeds a fixed capacity";
        case SPMM_ERR_DEV_BOUNDS: return "a kernel met an index outside its range";
        case SPMM_ERR_DEV_UNDRAINED: return "a bounded wait inside a kernel ran out and so did the wait for its work in flight";
        default: return "unknown status";
    }
}


int spmm_set_wait_limit_ns(uint64_t ns) {
    g_wait_limit_ns.store(ns);
    return SPMM_OK;
}

}  // extern "C"
