// Launch interfaces between the C-ABI layer (api.cu) and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spmm {

// per-device caches (kernel attributes, the built-in scratch address) are arrays of this length
constexpr int kMaxDevices = 64;

struct BcsrParams {
    const int32_t* block_row_ptr;
    const int32_t* block_col_idx;
    const int4* tiles;        // {block-row, token tile, first stored block, end block}, CTA-major
    const int32_t* cta_ptr;   // [grid+1] ranges of tiles
    void* C;            // fp32 or the input's 16-bit type; [m][N], or [N][m] with column-major operands
    int64_t m, N;
    int* status;
    uint64_t wait_limit_ns;
    int32_t use_3d;     // tmB3 is valid: whole token tiles are fetched with one 3-D request
    // stacked launch only: [groups][128 / b] block-rows of every row group (see BcsrStack); the
    // tile records then name {group, token tile, first stacked block, end stacked block} and
    // block_col_idx is the stacked blocks' column index
    const int32_t* stack_rows;
    // 1: this grid lets the next launch of the stream start while it runs (its first
    // instruction after set-up is griddepcontrol.launch_dependents); 2: this grid was launched
    // that way behind another one and waits for it (griddepcontrol.wait) before its CTAs exit
    int32_t overlap;
};

// dtype: 0 bf16, 1 fp16, 2 tf32 (fp32 storage; fp32 C, static schedule), 3 E4M3 (column-major
// operands, fp32 C).  groups: token tile = 128 * groups columns of B (1, 2 or 4).
// c16: C in the input's 16-bit type.  With es = bytes per element, t = 128 / es tokens per
// 128-byte box row and kb = b / bcsr_k_split(b, es) rows of B per stage unit --
// row-major operands: tmB = B as [k][N], box kb x t; tmB3 = B as [N / t][k][t], box
// (es * groups) x kb x t; 128-byte swizzle (with 32-byte atoms for es = 4).  Column-major operands
// (col_major): tmB = X as [N][k], box 128 tokens x min(kb * es, 128) bytes; tmB3 = X as
// [N / 128][128][k], box groups x 128 x the same; both with the swizzle of that row length.
// tmA: the stored blocks as [blocks * b][b], box (b * blocks per stage) rows x min(kb * es, 128) bytes.
// tmC: C as [m][N], box 32 x bcsr_epi_cols, no swizzle; or Y as [N][m], box bcsr_epi_cols x 32,
// 64-byte swizzle when a box row is 64 bytes.
// dynamic: the grid is one CTA per tile (grid = number of tiles, p.tiles in the schedule's global
// order, p.cta_ptr unused) and CTAs steal tiles through Cluster Launch Control; fp32 row-major only.
cudaError_t launch_bcsr(int dtype, int b, int groups, int c16, int col_major, int dynamic, const CUtensorMap& tmA,
                        const CUtensorMap& tmB, const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP,
                        const BcsrParams& p, int grid, cudaStream_t stream);
// Row groups: the same kernel with 128 x b stacked blocks (MMA N = 128) and a 256-token tile.
// tmA: the stacked values as [blocks * 128][b], box 128 x b; tmB3 built for groups = 2; b = 16, 32, 64.
constexpr int kStackRows = 128;
constexpr int kStackGroups = 2;
cudaError_t launch_bcsr_stacked(int dtype, int b, int c16, int col_major, const CUtensorMap& tmA, const CUtensorMap& tmB,
                                const CUtensorMap& tmB3, const CUtensorMap& tmC, const CUtensorMap& tmP, const BcsrParams& p,
                                int grid, cudaStream_t stream);
// K-split: tmP = the partial tiles as [slots * b][N] fp32, box as tmC's (the tile record of a
// part holds -1 - slot in place of the block-row); pass tmC where the plan has no parts.
// The merge: C rows of every split block-row = sum of its parts' partial tiles in part order.
struct BcsrMergeParams {
    const int32_t* row;      // [n] split block-rows
    const int32_t* first;    // first slot
    const int32_t* nparts;
    const float* partial;    // [slots][b][N]
    float* C;                // [m][N]
    int64_t m, N;
    int32_t n, b;
};
cudaError_t launch_bcsr_merge(const BcsrMergeParams& p, cudaStream_t stream);
int bcsr_token_groups_max(int dtype, int b, int c16, int col_major);
// Accumulator columns (= rows of A's block) an epilogue warp handles at a time: it stages them
// in a 2 KB (1 KB for b = 16 with 16-bit C) shared-memory tile and stores the tile with one TMA
// request whose box is 32 tokens x this many rows (row-major C) or this many columns x 32 tokens
// (column-major Y).  Larger tiles (up to 64 rows) were measured slower: the stage ring needs the room.
constexpr int bcsr_epi_cols(int b, bool c16, bool col_major) { return (b < 32 || !c16) ? 16 : 32; }
// stored blocks that share one pipeline stage (and one A request): 4 / 2 for b = 16 / 32
constexpr int bcsr_blocks_per_stage(int b) { return b == 16 ? 4 : (b == 32 ? 2 : 1); }
// Column slices a stored block is cut into, one pipeline stage each: blocks of 4-byte elements
// with rows longer than 128 bytes (TF32, b = 64 / 128) go through the ring 32 columns at a time;
// every other block is one unit.
constexpr int bcsr_k_split(int b, int es) { return (es == 4 && b > 32) ? b / 32 : 1; }

// WCSR pipeline shape, shared by the host schedule (fills are cut to the stage size) and the
// kernel.  A stage holds 128 / es columns (64 of a 2-byte type, 32 of TF32) of one 128-token
// tile: 16 KB of gathered B rows + the A tile (2 KB at window height 16, 8 KB at 64).  Per value
// size and window height: ring depth, producer warps (each owns STAGES / PW stages) and resident
// CTAs per SM, which is also the number of bins per SM of the static schedule (every resident
// CTA walks one bin).  Measured on B200 at height 16: 2-byte types run fastest as three small
// CTAs per SM (4 stages, 4 producer warps), TF32 as two deeper ones (6 stages, 6 producer warps);
// both fill the SM's shared memory.  Height 64: two CTAs per SM, 4 stages of 24 KB, 4 producer
// warps (the accumulators of two CTAs fill the 512 TMEM columns).
#ifndef WCSR_STAGE_ROW_BYTES
#define WCSR_STAGE_ROW_BYTES 128
#endif
constexpr int wcsr_stage_cols(int es) { return WCSR_STAGE_ROW_BYTES / es; }
// Narrow dense operands (2-byte types, window height 16, N <= 64): a gathered row is one 128-byte
// segment instead of two, so a stage of the same size class holds 96 columns (12 KB of rows +
// 3 KB of A): a third fewer stage hand-shakes per column, which is what bounds the narrow case.
constexpr int kWcsrNarrowCols = 96;
constexpr int kWcsrNarrowMaxN = 64;
constexpr int wcsr_stages(int es, int wh) { return wh == 64 ? 4 : (es == 4 ? 6 : 4); }
constexpr int wcsr_producer_warps(int es, int wh) { return wh == 64 ? 4 : (es == 4 ? 6 : 4); }
constexpr int wcsr_bins_per_sm(int es, int wh) { return wh == 64 ? 2 : (es == 4 ? 2 : 3); }

// Device task descriptor of the WCSR kernel (one per sub-task of the split plan).
struct WcsrDevTask {
    int32_t col_begin;   // absolute position of the task's first padded column
    int32_t count;       // columns (multiple of b_col)
    int32_t window;
    int32_t slot;        // partial tile index, or -1: write C directly
};

struct WcsrParams {
    const int32_t* bin_ptr;      // [n_bins+1] ranges of items
    const int4* items;           // {window, partial slot or -1, columns, 0} of every task, bin-major
    const int2* fills;           // {first padded column, count | first<<16 | last<<17}, bin-major (cut to the launch's stage size)
    const int32_t* bin_fill;     // [n_bins+1] fill ranges
    const int32_t* col_idx;      // window_col_idx [P]
    const uint8_t* grp_class;    // reuse class of every four padded columns [P / 4], or null: no gather hints
    int32_t hot_min;             // groups of this class and above are gathered with the evict-last priority
    int32_t hint_flags;          // 1: the packed A tiles are fetched evict-first
    const uint8_t* packed;       // packed A values
    const void* B;               // k x N row-major
    void* C;                     // [m][N] fp32, or the input's 16-bit type
    float* partial;              // [n_slots][window height][N]
    int64_t m, N;
    int32_t n_bins;
    int32_t n_tt;                // token tiles = ceil(N / (128 * groups))
    int* status;
    uint64_t wait_limit_ns;
};

// dtype: 0 bf16, 1 fp16, 2 tf32, 3 E4M3 (fp32 C).  tmB: 2-D map of B (k rows x N), box = 128
// bytes x 1 row, 128-byte swizzle (32-byte atoms for tf32), used in row-gather mode.
// narrow: the N <= 64 variant for 2-byte types at window height 16 (p.fills / p.bin_fill cut to kWcsrNarrowCols).
// lsu_gather: the comparison variant whose producers gather B rows with 16-byte cp.async copies through the
// load/store units instead of TMA (window height 16, fp32 C, not narrow); tmB is then unused.
cudaError_t launch_wcsr(int dtype, int wh, int c16, int narrow, int lsu_gather, const CUtensorMap& tmB, const WcsrParams& p,
                        int sms, cudaStream_t stream);

struct MergeParams {
    const int32_t* window;   // [n] windows the merge writes
    const int32_t* first;    // first slot or -1
    const int32_t* nparts;   // slots to add (0 = zero fill)
    const float* partial;
    void* C;
    int64_t m, N;
    int32_t n;
};
cudaError_t launch_wcsr_merge(const MergeParams& p, int wh, int ctype, cudaStream_t stream);   // ctype: 0 fp32, 1 fp16, 2 bf16

// Device address and size in bytes of the library's built-in partial-tile scratch on the
// current device (resolved on the first call per device).
cudaError_t wcsr_static_scratch(float** ptr, size_t* bytes);

}  // namespace spmm
