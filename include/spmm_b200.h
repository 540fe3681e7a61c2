/*
 * spmm_b200 -- sparse x dense matrix multiplication C = A x B on one NVIDIA
 * B200 (sm_100a), with A held in one of the two formats of the AsyncSparse
 * paper (Sec. 2.3 "Sparse Formats"):
 *
 *   BCSR  Block Compressed Sparse Row: A is tiled into b x b blocks and only
 *         blocks holding at least one stored entry are kept, each as a dense
 *         tile.  The kernel runs one tensor-core micro-GEMM per stored block
 *         (Sec. 3.1 - 3.3).
 *   WCSR  Window Compressed Sparse Row: rows are grouped into windows of
 *         fixed height; per window the union of the column indices is kept
 *         and padded to a multiple of b_col.  The kernel gathers the matching
 *         rows of B and multiplies them with the packed window tile; long
 *         windows are cut into fixed-size sub-tasks (Sec. 3.2 - 3.3).
 *
 * Conventions
 *   - A is m x k, B is k x N row-major (B[r*N + c]), C is m x N row-major,
 *     fp32 -- unless the handle was created with opts.layout (both operands
 *     column-major, BCSR) or opts.c_type (C in the input's 16-bit type).  C is
 *     overwritten completely (no alpha / beta; Sec. 2.3 states the problem as
 *     C = A x B).
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA
 *     device memory of the current device.  The library never frees or keeps
 *     a caller's pointer beyond the call that receives it.
 *   - Every function returns 0 (SPMM_OK) or a negative spmm_status_t.  No
 *     exception crosses this boundary.
 *   - There is no CPU fallback: without a CUDA device every create call that
 *     is not host_only, and every run call, fails with SPMM_ERR_CUDA.
 */
#ifndef SPMM_B200_H
#define SPMM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spmm_handle_s *spmm_handle_t;

typedef enum {
    SPMM_OK = 0,
    SPMM_ERR_INVALID_ARG = -1,   /* null pointer, negative size, bad enum value              */
    SPMM_ERR_UNSORTED = -2,      /* CSR columns not strictly ascending / duplicate COO entry  */
    SPMM_ERR_OUT_OF_RANGE = -3,  /* row or column index outside the matrix                    */
    SPMM_ERR_UNSUPPORTED = -4,   /* block / window size, N, dtype or alignment not supported  */
    SPMM_ERR_ALLOC = -5,         /* host or device allocation failed                          */
    SPMM_ERR_CUDA = -6,          /* a CUDA call or a launch failed (no device, bad context)   */
    SPMM_ERR_DEV_TIMEOUT = -7,   /* a bounded wait inside a kernel ran out (see spmm_check)   */
    SPMM_ERR_HOST_ONLY = -8,     /* the handle was created host_only and cannot run           */
    SPMM_ERR_TOO_LARGE = -9,     /* a size exceeds a fixed capacity (int32 index, scratch)    */
    SPMM_ERR_DEV_BOUNDS = -10,   /* a kernel met an index outside its range and stopped using
                                    it (reported by spmm_check; cannot happen with a handle
                                    this library built)                                       */
    SPMM_ERR_DEV_UNDRAINED = -11 /* as SPMM_ERR_DEV_TIMEOUT, and the wait for the copies or
                                    tensor-core work the kernel had in flight when it gave up
                                    ran out as well: it left while they may still have been
                                    writing shared or tensor memory, so kernels that ran on the
                                    device afterwards may be affected too (spmm_check)        */
} spmm_status_t;

/* Value type of A and B.  Accumulation is always fp32 (C: see spmm_ctype_t). */
typedef enum {
    SPMM_BF16 = 0,               /* 2-byte bfloat16 storage                                   */
    SPMM_FP16 = 1,               /* 2-byte IEEE half storage                                  */
    SPMM_TF32 = 2,               /* 4-byte fp32 storage, TF32 tensor-core arithmetic (the
                                    k8 instruction shape of Sec. 3.1; Sec. 4.1 evaluates both
                                    formats in it).  WCSR, and BCSR with every block size and
                                    both layouts; C is fp32, the BCSR schedule static, and
                                    BCSR row groups are not formed.                           */
    SPMM_FP8_E4M3 = 3            /* 1-byte E4M3 storage (Sec. 5 names 8-bit inputs as the next
                                    step); fp32 C.  BCSR: static schedule, block 32, 64 or
                                    128; row-major operands need N >= 128 and N % 16 == 0,
                                    SPMM_COLMAJOR needs k % 16 == 0 (row groups are formed with
                                    SPMM_COLMAJOR only).  WCSR: windows padded to 32 columns
                                    (b_col = 32), the TMA gather, N % 16 == 0.                */
} spmm_dtype_t;

/* Element type of C (opts.c_type).  Accumulation is fp32 either way. */
typedef enum {
    SPMM_C_FP32 = 0,             /* fp32 (default; the type the paper's kernels write)        */
    SPMM_C_SAME_AS_INPUT = 1     /* bf16 / fp16 handles: C in that type, rounded to nearest
                                    even from the fp32 accumulator.  TF32 handles: fp32.      */
} spmm_ctype_t;

/* Operand layout (opts.layout), BCSR only. */
typedef enum {
    SPMM_ROWMAJOR = 0,           /* B is k x N, C is m x N, both row-major (default)          */
    SPMM_COLMAJOR = 1            /* B and C column-major, i.e. the caller holds X = B^T as a
                                    row-major N x k array and receives Y = C^T as a row-major
                                    N x m array: the layout of the paper's BCSR kernel
                                    (Sec. 3.2) and of a linear layer Y = X W^T with a sparse
                                    weight W = A (Sec. 4.4).  Needs m % 8 == 0, k % 8 == 0 and
                                    N >= 128; N itself is unconstrained.                      */
} spmm_layout_t;

/* How the BCSR kernel's tiles (block-row x token tile) reach the CTAs (opts.schedule). */
typedef enum {
    SPMM_SCHED_STATIC = 0,       /* dealt to the persistent CTAs ahead of time (default)     */
    SPMM_SCHED_DYNAMIC = 1       /* one CTA per tile in the grid; running CTAs take over the
                                    tiles of CTAs that have not started yet (Cluster Launch
                                    Control), in the schedule's global order.  BCSR, fp32
                                    row-major C only.  Sec. 3.6 / Sec. 5: the paper's dynamic
                                    scheduler used an atomic counter and lost to the hardware
                                    block scheduler; this is the hardware queue itself.       */
} spmm_sched_t;

/* How the WCSR kernel brings the gathered rows of B into shared memory (opts.gather). */
typedef enum {
    SPMM_GATHER_TMA = 0,         /* TMA row gather (four rows x 128 bytes per request), the
                                    default: the indirect load Sec. 3.2 says TMA cannot do is
                                    available on this architecture                            */
    SPMM_GATHER_LSU = 1          /* the paper's own scheme (Sec. 3.2): the producer warps copy
                                    the rows with 128-bit loads through the load/store units
                                    (16-byte cp.async) to the swizzled positions the MMA reads.
                                    Kept for the side-by-side measurement; window height 16,
                                    fp32 C.                                                   */
} spmm_gather_t;

/* Optional creation parameters; pass NULL for all defaults.  Zero = default. */
typedef struct {
    int32_t b_col;       /* WCSR: pad every window to a multiple of this many columns.
                            Default (and only supported value): 16 for 2-byte types, 8 for
                            TF32, 32 for E4M3 -- the K extent of one tensor-core instruction
                            (Sec. 2.3, Sec. 4.1 uses 8 with TF32).                           */
    int32_t split_cols;  /* WCSR: sub-task size T in columns (Sec. 3.3); multiple of b_col.
                            Default: the largest of one bin's share of the padded columns, its
                            half, quarter and eighth (rounded down to a multiple of 64, clamped
                            to [128, 65536]) whose longest-first assignment of the sub-tasks to
                            the bins ends within 2 % of the best of the four: as few split
                            windows as the balance allows.                                    */
    int32_t host_only;   /* 1: build the format on the host only (no CUDA call at all); the
                            handle serves spmm_export / spmm_get_info, spmm_run fails.       */
    int32_t n_ctas;      /* persistent grid size the schedule is built for; default = the
                            device's SM count (148 when host_only).                          */
    int32_t c_type;      /* spmm_ctype_t                                                      */
    int32_t layout;      /* spmm_layout_t; SPMM_COLMAJOR with a WCSR handle is UNSUPPORTED    */
    int32_t schedule;    /* spmm_sched_t; with SPMM_SCHED_DYNAMIC the exported tile list is a
                            single range (TILE_PTR = {0, n_tiles}) in the global order       */
    int32_t stack_min_fill; /* BCSR row groups (no counterpart in the paper): where 128 / b
                            block-rows store blocks in mostly the same block columns, the
                            kernel computes them together from 128-row stacked blocks (absent
                            sub-blocks zero), so that each slice of the dense operand is staged
                            once for all of them.  Grouping is by similarity: in ROW_ORDER, every
                            block-row not yet grouped is offered the 128 / b - 1 ungrouped
                            block-rows that share the most block columns with it (they may
                            lie anywhere in the matrix); the candidate is taken when at least
                            this percentage of its sub-blocks is stored (the search is capped
                            at 2^27 visited stored blocks).  0 = default (30 / 45 / 75
                            for b = 16 / 32 / 64), -1 = off, 1..100 = threshold.  A private
                            second copy of the grouped rows' values is kept on the device; the
                            exported format arrays and nnz_stored are unaffected.  Ignored for
                            b = 128 and the dynamic schedule.                                 */
    int32_t gather;      /* spmm_gather_t; WCSR only (a BCSR handle ignores it)              */
    int32_t k_split;     /* BCSR: 1 = a block-row whose stored blocks exceed a quarter of one
                            CTA's mean load for the dense width at hand is cut into contiguous
                            ranges of its stored blocks; each part computes a partial tile and
                            a second kernel adds the parts in order (the same rule as the WCSR
                            merge: run-to-run identical).  The optional counterpart of
                            Sec. 3.3's task split for the structured path, where Sec. 3.5 - 3.6
                            report the imbalance.  Static schedule, fp32 row-major C, no row
                            groups in use.  0 = off (default: the uncut plan measured faster on
                            the benchmark configurations).                                    */
    int32_t reserved[6];
} spmm_opts_t;

typedef struct {
    int32_t format;          /* 0 = BCSR, 1 = WCSR                                            */
    int32_t dtype;           /* spmm_dtype_t                                                  */
    int64_t m, k, nnz;       /* matrix shape and number of stored CSR/COO entries             */
    int32_t block;           /* BCSR block size b, or WCSR window height                      */
    int32_t b_col;           /* WCSR column padding (0 for BCSR)                              */
    int64_t n_units;         /* BCSR: stored blocks; WCSR: padded columns P                   */
    int64_t stored_values;   /* BCSR: blocks*b*b; WCSR: height*P  ("nnz_stored")              */
    double  fill_ratio;      /* nnz / stored_values (Sec. 2.3)                                */
    int64_t n_rows_units;    /* BCSR: block-rows; WCSR: windows                               */
    int64_t n_empty;         /* empty block-rows / windows                                    */
    int64_t n_tasks;         /* WCSR sub-tasks; BCSR: K-split units of the current plan (0 if no
                                block-row is cut)                                             */
    int64_t n_split;         /* WCSR windows / BCSR block-rows cut into more than one part    */
    int64_t n_slots;         /* partial-sum tiles (WCSR sub-tasks of split windows; BCSR parts) */
    int32_t split_cols;      /* WCSR T in effect; BCSR: the K-split cap in stored blocks      */
    int32_t n_ctas;          /* grid size the schedule was built for                          */
    int64_t distinct_b_rows; /* rows of B that A touches (distinct stored columns)            */
    /* bytes the roofline model charges for one spmm_run at the given N: */
    double  bytes_a, bytes_idx, bytes_b_touched, bytes_c;
    double  bytes_gather;    /* B bytes that must enter shared memory (no reuse assumed)      */
    double  flops_stored;    /* 2 * stored_values * N                                         */
    int64_t workspace_bytes; /* device scratch spmm_run needs at this N (partial tiles; for BCSR
                                at the planned N)                                             */
    /* BCSR tile schedule currently held (spmm_bcsr_plan or the last spmm_run); 0 if none:   */
    int64_t plan_n;          /* dense width it was built for                                  */
    int32_t plan_token_tile; /* columns of B per tile: 128, 256 or 512                        */
    int32_t plan_slab_tiles; /* token tiles per L2 slab                                       */
    int32_t n_bins;          /* WCSR: bins of the static task schedule (0 for BCSR): n_ctas x
                                the resident CTAs per SM of the kernel for this value type     */
    int32_t n_stacked_rows;  /* BCSR: block-rows computed as members of row groups            */
    int64_t n_stack_blocks;  /* BCSR: 128-row stacked blocks those groups hold                 */
} spmm_info_t;

/* Arrays spmm_export can return, in their canonical (paper) layout. */
typedef enum {
    SPMM_X_BCSR_BLOCK_ROW_PTR = 0,  /* int32 [ceil(m/b)+1]                                   */
    SPMM_X_BCSR_BLOCK_COL_IDX = 1,  /* int32 [n_blocks], ascending inside a block-row         */
    SPMM_X_BCSR_BLOCKS = 2,         /* dtype [n_blocks][b][b] row-major, zero filled          */
    SPMM_X_BCSR_ROW_ORDER = 3,      /* int32 [block-rows]: schedule order, longest first      */
    SPMM_X_BCSR_TILE_PTR = 4,       /* int32 [n_ctas+1]: per-CTA ranges of TILES (needs a plan) */
    SPMM_X_BCSR_TILES = 5,          /* int32 [n_tiles][2]: block-row, token tile; CTA-major
                                       (block-rows outside the row groups only)               */
    SPMM_X_BCSR_STACK_ROWS = 6,     /* int32 [groups][128/b]: block-rows of every row group     */
    SPMM_X_BCSR_STACK_PTR = 7,      /* int32 [groups+1]: ranges of STACK_COL_IDX                */
    SPMM_X_BCSR_STACK_COL_IDX = 8,  /* int32 [n_stack_blocks]: block columns of a group's union,
                                       ascending                                              */
    SPMM_X_BCSR_STACK_TILE_PTR = 9, /* int32 [n_ctas+1]: per-CTA ranges of STACK_TILES (needs a
                                       plan)                                                  */
    SPMM_X_BCSR_STACK_TILES = 20,   /* int32 [n][2]: row group, 256-column token tile; CTA-major */
    SPMM_X_BCSR_UNITS = 21,         /* int32 [n_units][4]: block-row, first stored block, end
                                       stored block, partial slot (-1: the unit is a whole block-row
                                       and writes C).  Empty unless the plan cut a block-row
                                       (opts.k_split); TILES[.][0] then indexes this array instead
                                       of naming a block-row                                    */
    SPMM_X_WCSR_WINDOW_ROW_PTR = 10,/* int32 [ceil(m/h)+1], in columns                        */
    SPMM_X_WCSR_WINDOW_COL_IDX = 11,/* int32 [P], -1 on padding                               */
    SPMM_X_WCSR_VALUES = 12,        /* dtype [h][P] row-major                                 */
    SPMM_X_WCSR_TASKS = 13,         /* int32 [n_tasks][4]: window, first col in window,
                                       column count, partial slot (-1 = writes C directly)    */
    SPMM_X_WCSR_BIN_PTR = 14,       /* int32 [n_bins+1]: ranges of BIN_TASKS, n_bins = 2*n_ctas */
    SPMM_X_WCSR_BIN_TASKS = 15,     /* int32 [n_tasks]: task indices bin by bin (the static
                                       schedule: CTA c runs bins c, c + grid, ...)            */
    SPMM_X_WCSR_GROUP_CLASS = 16    /* uint8 [P / 4]: reuse class of every four padded columns
                                       (7 = among the 16 Ki most gathered rows of B, each class
                                       below twice as many, 0 = the rest): the kernel's L2
                                       hint for the gathers, no effect on results             */
} spmm_export_t;

/*
 * Create a BCSR handle from CSR (Sec. 2.3, BCSR paragraph).
 *   out      receives the handle (NULL on failure).
 *   m, k     matrix shape; need not be multiples of `block` (ragged edge is zero padded).
 *   row_ptr  host int64 [m+1], row_ptr[0] = 0, non-decreasing.
 *   col_idx  host int32 [nnz], strictly ascending inside each row, in [0, k).
 *   vals     host, nnz elements of `dtype` (2 or 4 bytes each; bf16/fp16 as raw 16-bit).
 *   block    16, 32, 64 or 128.
 * A block is kept when any stored entry falls inside it, whatever its value.
 * The arrays are copied; the caller keeps ownership.  The handle owns its device memory.
 */
int spmm_bcsr_create_csr(spmm_handle_t *out, int64_t m, int64_t k, const int64_t *row_ptr,
                         const int32_t *col_idx, const void *vals, int dtype, int block,
                         const spmm_opts_t *opts);

/*
 * Same handle, built on the GPU from a CSR matrix that already lives in DEVICE memory
 * (block mask, index and value packing of Sec. 2.3 as kernels; the paper builds its formats
 * offline).  row_ptr_dev / col_idx_dev / vals_dev are device pointers with the layout of
 * spmm_bcsr_create_csr; the caller keeps them.  The CSR is validated on the device (same
 * error codes).  The call runs on `stream` (a cudaStream_t as void*, NULL = default) and
 * synchronises it; opts.host_only is not allowed.  Limit: ceil(k / block) <= 819,200.
 */
int spmm_bcsr_create_csr_device(spmm_handle_t *out, int64_t m, int64_t k, const int64_t *row_ptr_dev,
                                const int32_t *col_idx_dev, const void *vals_dev, int dtype, int block,
                                const spmm_opts_t *opts, void *stream);

/*
 * The WCSR counterpart: window condensation and value packing on the GPU from a device-resident
 * CSR (sort / unique of (window, column) keys); arguments as spmm_bcsr_create_csr_device with
 * window_height in place of block.  nnz must be below 2^31.
 */
int spmm_wcsr_create_csr_device(spmm_handle_t *out, int64_t m, int64_t k, const int64_t *row_ptr_dev,
                                const int32_t *col_idx_dev, const void *vals_dev, int dtype,
                                int window_height, const spmm_opts_t *opts, void *stream);

/* Same from COO: host int32 rows[nnz], cols[nnz] in any order, no duplicate (row, col). */
int spmm_bcsr_create_coo(spmm_handle_t *out, int64_t m, int64_t k, int64_t nnz,
                         const int32_t *rows, const int32_t *cols, const void *vals, int dtype,
                         int block, const spmm_opts_t *opts);

/*
 * Create a WCSR handle (Sec. 2.3, WCSR paragraph; task split of Sec. 3.3).
 * Arguments as above; window_height is 16 (the benchmark configurations; Sec. 5 names
 * finer-than-64 windows as the redesign this library performs) or 64 (the paper's own
 * window, Sec. 4.1).
 * Per window the kept columns are ascending, then -1 pads up to a multiple of b_col.
 */
int spmm_wcsr_create_csr(spmm_handle_t *out, int64_t m, int64_t k, const int64_t *row_ptr,
                         const int32_t *col_idx, const void *vals, int dtype, int window_height,
                         const spmm_opts_t *opts);

int spmm_wcsr_create_coo(spmm_handle_t *out, int64_t m, int64_t k, int64_t nnz,
                         const int32_t *rows, const int32_t *cols, const void *vals, int dtype,
                         int window_height, const spmm_opts_t *opts);

/*
 * BCSR only: build (and keep) the static tile schedule for dense width N -- the one
 * spmm_run(h, ., ., N, .) uses -- so that it can be inspected with spmm_export / spmm_get_info.
 * The schedule answers the load imbalance Sec. 3.5 and Sec. 4.2 (opt6) report for a persistent
 * kernel with a fixed tile order: tiles (block-row x token tile) are dealt to the CTAs ahead
 * of time, longest block-row first, each to the least loaded CTA.  A handle with row groups
 * (opts.stack_min_fill) gets two such lists: STACK_TILES for the groups (256-token tiles), whose
 * launch goes first, and TILES for the other block-rows, dealt with the head start that the
 * j-th lightest CTA of the first launch leaves to CTA j of the second (loads counted in bytes
 * staged per block).  Works on host_only handles.
 * spmm_run builds the same schedule on its first call with a new N (that call allocates and
 * may synchronise the device).
 */
int spmm_bcsr_plan(spmm_handle_t h, int64_t N);

/*
 * Both formats (an addition of this library): do ahead of time what the first spmm_run with a
 * new dense width N would do besides launching -- BCSR: spmm_bcsr_plan (schedule, its device
 * arrays, the workspace of a K-split plan); WCSR: grow the handle's partial-tile workspace to
 * what N needs.  May allocate and synchronise the device.  Afterwards spmm_run(h, ., ., N', .)
 * with N' = N (BCSR) or N' <= N (WCSR) makes no allocating or synchronising call of its own
 * (the CUDA runtime may still load a kernel variant's code on that variant's first launch).
 * Same argument rules as spmm_run for N; a host_only WCSR handle returns SPMM_OK and does nothing.
 */
int spmm_prepare(spmm_handle_t h, int64_t N);

/*
 * C = A x B (Sec. 2.3; kernels of Sec. 3).  Asynchronous on `stream` (a cudaStream_t passed
 * as void*; NULL = the default stream); never synchronises.
 *   B_dev  device, k x N row-major, elements of the handle's dtype, 16-byte aligned.
 *   C_dev  device, m x N row-major, fp32 (or the handle's 16-bit type with
 *          SPMM_C_SAME_AS_INPUT), 16-byte aligned; every element is written.
 *   N      dense width; N * element size must be a multiple of 16 bytes.  A BCSR handle
 *          with row-major operands also needs N >= 64 (SPMM_ERR_UNSUPPORTED below that; the
 *          same holds for spmm_bcsr_plan); WCSR accepts any such N.
 * With SPMM_COLMAJOR (BCSR): B_dev is X, N x k row-major, and C_dev is Y, N x m row-major,
 * Y[n][i] = sum_j A[i][j] * X[n][j]; any N >= 128.
 * The handle must be run with the device it was created on current (SPMM_ERR_INVALID_ARG
 * otherwise, nothing is launched).
 * WCSR keeps the partial tiles of split windows in a device workspace owned by the handle;
 * it is (re)allocated here the first time a given N needs more than it holds, so two runs
 * of one handle must not overlap on the GPU, and the first run at a new N may synchronise.
 * Split windows are merged by a fixed-order sum, so results are run-to-run identical.
 * A BCSR handle with row groups launches its kernel twice (groups, then the other block-rows;
 * the second launch starts on the SMs the first leaves idle and does not finish before it).
 * A BCSR plan that cuts long block-rows (opts.k_split) keeps the parts' partial tiles in a
 * workspace of the handle as well (allocated with the plan) and adds a small merge kernel.
 */
int spmm_run(spmm_handle_t h, const void *B_dev, void *C_dev, int64_t N, void *stream);

/*
 * WCSR only; the paper has no counterpart (an addition of this library).  Same result as
 * spmm_run, but the call allocates nothing: the partial tiles of split windows go to a
 * scratch array that is built into the library (8 MiB of device memory, held by every GPU
 * that loads the library until the process exits) instead of a workspace allocated on
 * demand.  It is meant for callers that must not allocate device memory at the time of the
 * call: code that runs inside a framework whose memory pool already owns the device, or a
 * latency-critical loop that cannot afford the device-wide synchronisation an allocation
 * or a free can cause.
 *   - The partial tiles need n_slots * window_height * N * 4 bytes (spmm_get_info:
 *     workspace_bytes; a 64-row handle needs four times what a 16-row one does).  More than
 *     8 MiB returns SPMM_ERR_TOO_LARGE and nothing is launched; choose a larger split_cols at
 *     creation, a smaller N, or use spmm_run.
 *   - The first call on each device looks up the scratch array's device address, and the
 *     first launch of each kernel variant (value type, window height, C type, N <= 64 or
 *     wider) on a device sets that kernel's attributes and may load its code.  Make one
 *     warm-up call per handle type and N class outside any stream capture and outside the
 *     loop that must not stall.  Later calls only launch kernels.
 *   - The array is shared by all handles and all calls and keeps the previous call's
 *     contents; every partial tile a call reads is first written by that same call, so
 *     nothing needs clearing.  Two calls that overlap on the GPU (different streams, or
 *     different host threads) race on it: serialise them.
 *   - Returns SPMM_ERR_INVALID_ARG for a BCSR handle.
 * Arguments and all other behaviour as spmm_run.
 */
int spmm_wcsr_run_static(spmm_handle_t h, const void *B_dev, void *C_dev, int64_t N, void *stream);

/*
 * Same result as spmm_run, for callers that hold HOST buffers: copies B to the device,
 * runs, copies C back and synchronises `stream` before returning.  B_host / C_host are
 * ordinary or pinned host memory of k*N elements / m*N elements of C's type, in the
 * handle's layout; the device staging buffers
 * belong to the handle and are reused between calls.
 * Operands of 8 MB and more travel in up to eight equal chunks of N (column ranges of
 * row-major operands, moved with 2-D copies of at least 256 bytes per row; token ranges of
 * column-major ones), each computed by its own kernel launch on `stream`, so that a
 * chunk's result goes back to the host while the next chunk's operand comes in: two
 * copy streams owned by the handle carry the transfers, ordered against `stream` with
 * events.  The result does not depend on the chunking.  Pinned host memory is needed for
 * the copies to overlap.
 */
int spmm_run_host(spmm_handle_t h, const void *B_host, void *C_host, int64_t N, void *stream);

/*
 * After the caller has synchronised the stream: reads the handle's device status word.
 * Every wait inside the kernels is bounded; a wait that ran out makes the kernel leave
 * early and this call return SPMM_ERR_DEV_TIMEOUT (the output is then undefined).
 * The status word is cleared by the call.
 */
int spmm_check(spmm_handle_t h);

/* Fill *info; the byte / flop model fields are evaluated for dense width N (N may be 0). */
int spmm_get_info(spmm_handle_t h, int64_t N, spmm_info_t *info);

/*
 * Copy one canonical array to host memory.  *need receives its size in bytes; when
 * host_dst is NULL or cap < *need nothing is copied (SPMM_ERR_INVALID_ARG if cap is too
 * small and host_dst non-NULL).  Arrays are read back from the device copy the kernels
 * use (and un-permuted where the device layout is private), so what is checked is what runs.
 */
int spmm_export(spmm_handle_t h, int which, void *host_dst, size_t cap, size_t *need);

/* Free the handle and everything it owns.  NULL is accepted. */
int spmm_destroy(spmm_handle_t h);

/* Static, never-NULL description of a status code. */
const char *spmm_status_string(int code);

/*
 * Upper bound, in nanoseconds, of any single wait inside a kernel (default 2e9).  Process
 * wide.  0 makes every wait that is not satisfied on its first poll run out at once: a hook
 * for testing the failure path (the kernel leaves early, spmm_check reports
 * SPMM_ERR_DEV_TIMEOUT, the context stays usable).
 */
int spmm_set_wait_limit_ns(uint64_t ns);

#ifdef __cplusplus
}
#endif
#endif /* SPMM_B200_H */
