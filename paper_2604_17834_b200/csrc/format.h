// Host-side format construction: CSR/COO canonicalisation, BCSR block mask and
// packing, WCSR window condensation and column remap, long-window split plan and
// the static schedules (Sec. 2.3 formats; Sec. 3.3 task decomposition).
#pragma once

#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

namespace spmm {

struct CsrView {
    int64_t m = 0, k = 0, nnz = 0;
    const int64_t* row_ptr = nullptr;
    const int32_t* col_idx = nullptr;
    const uint8_t* vals = nullptr;   // nnz * es bytes
    int es = 2;                      // element size in bytes
};

// Owning CSR, produced from COO.
struct CsrOwned {
    std::vector<int64_t> row_ptr;
    std::vector<int32_t> col_idx;
    std::vector<uint8_t> vals;
};

struct BcsrHost {
    int b = 0;
    int64_t nbr = 0, nbc = 0, nnzb = 0, n_empty = 0, distinct_bcols = 0;
    std::vector<int32_t> block_row_ptr;   // [nbr+1]
    std::vector<int32_t> block_col_idx;   // [nnzb], ascending inside a block-row
    std::vector<uint8_t> blocks;          // [nnzb][b][b] * es, zero filled
    std::vector<int32_t> row_order;       // [nbr] block-rows, most stored blocks first (stable)
};

// Row stacking (device-private; no counterpart in the paper, whose blocks are all b x b).  A
// stored block costs the kernel one b-row slice of the token tile however few rows of A it has,
// so with small blocks the operand traffic into shared memory, not the arithmetic, bounds it.
// Where R = 128 / b block-rows store blocks in mostly the same block columns, they are computed
// as one "row group": for every block column of the union one stacked block of 128 rows x b
// (absent sub-blocks zero), so that the slice of the token tile is fetched once for all R rows
// and one MMA with N = 128 replaces R MMAs with N = b.
// Rule (a pure function of the index arrays; grouping by similarity): walk row_order (most stored
// blocks first).  A non-empty block-row not yet in a group is a seed; its partners are the R - 1
// other free block-rows that share the most block columns with it (at least one; ties: the one
// earlier in row_order).  The candidate is accepted when
// 100 * (stored blocks of the R rows) >= min_fill_pct * R * (block columns in their union);
// a rejected candidate leaves all its rows free.  The search stops once the work charged -- per
// seed, the number of stored blocks in the seed's block columns -- would pass kBcsrGroupWorkLimit.
struct BcsrStack {
    int R = 0;                          // block-rows per group; 0: no stacking for this handle
    int min_fill_pct = 0;
    int64_t ng = 0, ns = 0;             // row groups, stacked blocks
    std::vector<int32_t> rows;          // [ng][R] member block-rows, in row_order order
    std::vector<int32_t> ptr;           // [ng+1] ranges of stacked blocks
    std::vector<int32_t> col_idx;       // [ns] block columns of the union, ascending inside a group
    std::vector<int32_t> src;           // [ns][R] stored block behind each sub-block, or -1
    std::vector<uint8_t> stacked;       // [nbr] 1: the block-row belongs to a group
};
// default acceptance threshold per block size, from the bytes a stacked and an unstacked block
// bring into shared memory per unit of work (and measured on the Bernoulli sweep)
constexpr int64_t kBcsrGroupWorkLimit = int64_t{1} << 27;
constexpr int bcsr_stack_default_fill(int b) { return b == 16 ? 30 : (b == 32 ? 45 : 75); }
int build_bcsr_stack(const BcsrHost& f, int min_fill_pct, BcsrStack* out);

// Static tile schedule of the BCSR kernel for one dense width: a tile is (block-row, token
// tile).  Tiles are taken slab by slab (a slab = slab_w consecutive token tiles, sized so the
// B rows it touches stay in L2) and, inside a slab, block-rows with the most stored blocks
// first; each tile goes to the CTA whose load is smallest at that moment (ties: lowest CTA),
// load = sum of (stored blocks + kTileFixedCost).  Loads carry over from slab to slab.
struct BcsrSchedule {
    int64_t N = -1;
    int groups = 0, n_tt = 0, slab_w = 0, n_ctas = 0;
    std::vector<int32_t> cta_ptr;    // [n_ctas+1]
    std::vector<int32_t> tiles;      // 2 * n_tiles: {block-row (or K-split unit, below), token tile}, CTA-major
    // K-split of outlier block-rows (empty when no block-row exceeds the cap): 4 * n_units
    // {block-row, first stored block, end stored block, slot}; tiles[] then names units.
    std::vector<int32_t> units;
    int64_t n_slots = 0;             // partial tiles (one per part of a split block-row)
    int32_t cap = 0;
};
// K-split: a block-row with more stored blocks than cap = max(kKSplitMinCap, ceil(n_tt * sum over
// all block-rows of (stored blocks + kTileFixedCost) / (4 * n_ctas))) -- a quarter of a CTA's mean
// load -- is cut into ceil(len / cap) contiguous ranges of its stored blocks, part j = blocks
// [j * len / parts, (j + 1) * len / parts).  Each part computes a partial C tile (fp32, slot =
// running index over the parts of split block-rows in ascending block-row order); the parts are
// summed in part order by the merge kernel.  Units are listed block-rows in row_order, parts in
// order; they are scheduled most stored blocks first (stable).  Returns the units (empty: no split).
constexpr int kKSplitMinCap = 8;
int build_bcsr_ksplit(const BcsrHost& f, int n_tt, int n_ctas, std::vector<int32_t>* units, int64_t* n_slots, int32_t* cap);
// a tile's fixed cost in stored-block units: its epilogue writes b x BN x 4 bytes of C, a stored
// block brings b x BN x 2 bytes of B (measured best of 2 / 4 / 6 / 10 on the skewed sweep)
constexpr int kTileFixedCost = 4;

struct WcsrTask { int32_t window, q0, count, slot; };

struct WcsrHost {
    int wh = 0, b_col = 0, T = 0;
    int64_t nwin = 0, P = 0, n_empty = 0, n_split = 0, n_slots = 0, distinct_cols = 0;
    std::vector<int32_t> window_row_ptr;  // [nwin+1], in columns
    std::vector<int32_t> window_col_idx;  // [P], -1 on pads
    // Device-private packing of values[wh][P]: one chunk of wh x b_col values per group of
    // b_col consecutive padded columns; inside a chunk the order is
    // [16-byte K half (2)][8-row group (wh/8)][row in group (8)][16 bytes], which is the
    // un-swizzled K-major core-matrix layout tcgen05.mma reads.  chunk bytes = wh * 32.
    std::vector<uint8_t> packed;
    std::vector<WcsrTask> tasks;          // window order; chunks of a window consecutive
    // Static schedule: tasks are dealt to n_bins bins by the longest-processing-time rule
    // (cost = columns + kTaskFixedCost; heaviest task first, always into the lightest bin, ties
    // to the lowest bin index); inside a bin tasks run in ascending order.  CTA c runs bins
    // c, c + grid, ...
    std::vector<int32_t> bin_ptr;         // [n_bins+1]
    std::vector<int32_t> bin_tasks;       // [n_tasks] task indices, bin-major
    // Device-private pipeline schedule: every task cut into "fills" of at most kt columns (one
    // shared-memory stage each), stored bin-major in the bins' task order.
    // fills[i] = {first padded column, count | first<<16 | last<<17} where first / last mark
    // the first / last fill of a task; bin_fill[j] = index of the first fill of bin j.
    int kt = 0;
    std::vector<int32_t> fills;           // 2 * n_fills
    std::vector<int32_t> bin_fill;        // [n_bins+1]
    // the same for the narrow-operand kernel variant (stages of kWcsrNarrowCols columns); empty
    // unless the value type is 2 bytes wide and the window height 16
    std::vector<int32_t> fills_narrow, bin_fill_narrow;
    // Device-private gather hint (no effect on results): reuse class of every group of four
    // consecutive padded columns, one byte each.  A column's class says how high its B row ranks
    // by the number of windows that gather it: 7 = among the 16 Ki most gathered rows, 6 = 32 Ki,
    // ... 1 = 1 Mi, 0 = below that or gathered once; a group takes the highest class of its four
    // columns.  At run time the rows whose class reaches the level that fits half of L2 at the
    // dense width in use are gathered with the evict-last priority, the others with evict-first.
    std::vector<uint8_t> grp_class;       // [P / 4]
    // finalisation lists: windows whose C rows the merge kernel writes
    std::vector<int32_t> merge_window;    // split windows then empty windows
    std::vector<int32_t> merge_first;     // first slot (split) or -1 (empty)
    std::vector<int32_t> merge_nparts;    // number of slots (split) or 0 (empty)
};

// All return 0 or a negative spmm_status_t value.
int validate_csr(const CsrView& a);
int coo_to_csr(int64_t m, int64_t k, int64_t nnz, const int32_t* rows, const int32_t* cols,
               const uint8_t* vals, int es, CsrOwned* out);
int build_bcsr(const CsrView& a, int b, BcsrHost* out);
// Fills row_order, n_empty and distinct_bcols from the index arrays.
void finish_bcsr_host(BcsrHost* out);
// The same format built on the GPU from a CSR matrix in device memory (format_gpu.cu): validates the
// CSR, allocates and fills the three device arrays (owned by the caller afterwards), and leaves the
// index arrays and counts in *out (out->blocks stays empty).  Synchronises `stream`.
int build_bcsr_device(int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx, const uint8_t* d_vals,
                      int es, int b, cudaStream_t stream, BcsrHost* out, int64_t* nnz_out, int32_t** d_block_row_ptr,
                      int32_t** d_block_col_idx, uint8_t** d_blocks);
// Allocates and fills the stacked values [ns][128][b] on the device from the stored blocks and
// st.src (format_gpu.cu); *d_stacked is owned by the caller afterwards.  Synchronises the device.
int stack_bcsr_device(const uint8_t* d_blocks, const BcsrStack& st, int b, int es, uint8_t** d_stacked);
int build_bcsr_schedule(const BcsrHost& f, int n_tt, int slab_w, int n_ctas, BcsrSchedule* out);
// The same rule over any list of units (block-rows or row groups) given in schedule order with
// their lengths in stored blocks; tiles = {unit, token tile}.
// A tile's load is (length + fixed_cost) * unit_cost; CTA c starts with load initial[c] (all zero
// when initial is null); *final_loads (optional) receives the CTAs' loads at the end.
int build_tile_schedule(const std::vector<int32_t>& units, const std::vector<int32_t>& lens, int fixed_cost, int n_tt,
                        int slab_w, int n_ctas, BcsrSchedule* out, int64_t unit_cost = 1,
                        const std::vector<int64_t>* initial = nullptr, std::vector<int64_t>* final_loads = nullptr);
// Relative cost of one stored block in the two launches of a handle with row groups, in bytes
// staged per block divided by b: a stacked block brings 256 tokens x b and 128 x b of A, a b x b
// block 128 * groups tokens x b and b x b of A (both launches are bound by that traffic).
constexpr int64_t bcsr_stack_block_cost() { return 2 * (256 + 128); }
constexpr int64_t bcsr_block_cost(int b, int groups) { return 2 * (128 * groups + b); }
// a row group's tile writes 128 rows of C whatever its length
constexpr int kStackTileFixedCost = 8;
// T = 0 picks the sub-task size from the matrix (default_split_cols): the largest of one bin's
// share of the padded columns, its half, quarter and eighth (each rounded down to a multiple of 64
// and clamped to [128, 65536]) whose longest-processing-time assignment ends within 2 % of the
// best of the four: as few split windows as the balance allows.
int default_split_cols(const std::vector<int32_t>& window_row_ptr, int64_t nwin, int64_t P, int n_bins);
int build_wcsr(const CsrView& a, int wh, int b_col, int T, int n_bins, WcsrHost* out);
// Reuse classes of the column groups (WcsrHost::grp_class) from window_col_idx [P] and k.
constexpr int kWcsrTopClassRows = 16384;   // rows in class 7; every class below doubles it
void wcsr_reuse_classes(const int32_t* window_col_idx, int64_t P, int64_t k, std::vector<uint8_t>* grp_class);
// Second half of build_wcsr: split plan, bins, fills and merge lists from out->window_row_ptr / out->P.
int plan_wcsr(WcsrHost* out, int T, int n_bins, int es);
// The WCSR format arrays built on the GPU from a CSR matrix in device memory (format_gpu.cu):
// validates the CSR, allocates and fills window_row_ptr, window_col_idx and the packed values on
// the device (owned by the caller afterwards) together with the column groups' reuse classes
// (*d_grp_class, the rule of wcsr_reuse_classes), leaves window_row_ptr, P and distinct_cols in *out
// (out->window_col_idx, out->packed and out->grp_class stay empty) and runs plan_wcsr.
// Synchronises `stream`.
int build_wcsr_device(int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx, const uint8_t* d_vals,
                      int es, int wh, int b_col, int T, int n_bins, cudaStream_t stream, WcsrHost* out, int64_t* nnz_out,
                      int32_t** d_window_row_ptr, int32_t** d_window_col_idx, uint8_t** d_packed, uint8_t** d_grp_class);

// Byte offset of element (row r, padded column q) inside the packed WCSR value array.
#ifdef __CUDACC__
__host__ __device__
#endif
inline size_t wcsr_packed_offset(int wh, int b_col, int es, int r, int64_t q) {
    const int64_t chunk = q / b_col;
    const int c = static_cast<int>(q % b_col);
    const int byte_in_row = c * es;                  // 0 .. 31
    return static_cast<size_t>(chunk) * (static_cast<size_t>(wh) * 32) +
           static_cast<size_t>(byte_in_row / 16) * (static_cast<size_t>(wh) * 16) +
           static_cast<size_t>(r / 8) * 128 + static_cast<size_t>(r % 8) * 16 +
           static_cast<size_t>(byte_in_row % 16);
}

// Cost, in column equivalents, that the span partition charges per task on top of its columns.
constexpr int kTaskFixedCost = 32;

}  // namespace spmm
