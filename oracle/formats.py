"""Format oracle: BCSR, WCSR and the long-window split plan.  TEST INFRASTRUCTURE ONLY.

Each function writes out the definition from the paper (Sec. 2.3 "Sparse
Formats"; Sec. 3.3 for the task decomposition) with numpy primitives
(repeat, unique, bincount, cumsum, fancy-index scatter).  There is no
blocking, threading or device code here, and nothing is shared with the
CUDA library's own format construction.

Readings taken where the paper is silent or garbled (all listed again in the
design notes):
  * a block / a window column is kept when any *stored* CSR entry falls in
    it, whatever its value (structural, Sec. 2.3 "contain at least one
    nonzero");
  * m and k need not be multiples of the block / window size: counts use
    ceilings and the ragged edge is zero padded;
  * blocks inside a block-row and columns inside a window are ascending;
  * WCSR ``values`` is ONE row-major 2-D array [b_row, padded_nnz_cols]
    (the second of the two shapes printed in Sec. 2.3);
  * an empty window has length 0 (no pad group);
  * a long window is cut into consecutive chunks of T columns (Sec. 3.3
    "fixed-size sub-tasks"); T is a multiple of b_col.

Values are moved, never computed with, so any dtype works (bf16 travels as
uint16 bit patterns).

Pins (tests/test_oracle_formats.py): brute-force per-element Python
constructions on tiny inputs, round trips to dense, the array-length and
fill-ratio formulas of Sec. 2.3, dense / block-diagonal / diagonal /
identical-row special cases, wh = 1 degenerating to padded CSR.
"""
from __future__ import annotations

import numpy as np


def _csr_rows(row_ptr):
    row_ptr = np.asarray(row_ptr, dtype=np.int64)
    m = row_ptr.shape[0] - 1
    return np.repeat(np.arange(m, dtype=np.int64), np.diff(row_ptr))


def _cdiv(a, b):
    return -(-a // b)


# --------------------------------------------------------------------------- BCSR


def bcsr_from_csr(m, k, row_ptr, col_idx, vals, b):
    """CSR -> BCSR with b x b blocks (Sec. 2.3, BCSR paragraph).

    Returns dict(block_row_ptr int32 [ceil(m/b)+1], block_col_idx int32 [nnzb],
    blocks [nnzb, b, b] of vals.dtype, zero filled).
    """
    vals = np.asarray(vals)
    col = np.asarray(col_idx, dtype=np.int64)
    rows = _csr_rows(row_ptr)
    nbr, nbc = _cdiv(m, b), _cdiv(k, b)
    key = (rows // b) * nbc + (col // b)
    ukeys = np.unique(key)                       # ascending => block-row major, block-col ascending
    nnzb = ukeys.shape[0]
    counts = np.bincount(ukeys // nbc, minlength=nbr)
    block_row_ptr = np.zeros(nbr + 1, dtype=np.int64)
    block_row_ptr[1:] = np.cumsum(counts)
    blocks = np.zeros((nnzb, b, b), dtype=vals.dtype)
    pos = np.searchsorted(ukeys, key)
    blocks[pos, rows % b, col % b] = vals
    return dict(
        block_row_ptr=block_row_ptr.astype(np.int32),
        block_col_idx=(ukeys % nbc).astype(np.int32),
        blocks=blocks,
    )


def bcsr_to_dense(m, k, b, block_row_ptr, block_col_idx, blocks):
    """Expand BCSR back to a dense m x k array (stored zeros become zeros)."""
    nbr = block_row_ptr.shape[0] - 1
    nbc = _cdiv(k, b)
    D = np.zeros((nbr * b, nbc * b), dtype=blocks.dtype)
    for I in range(nbr):
        for p in range(block_row_ptr[I], block_row_ptr[I + 1]):
            J = int(block_col_idx[p])
            D[I * b:(I + 1) * b, J * b:(J + 1) * b] = blocks[p]
    return D[:m, :k]


def bcsr_block_count(m, k, row_ptr, col_idx, b):
    """Number of stored blocks of the BCSR form (Sec. 2.3) without building it: the count of
    distinct (row // b, column // b) pairs over the stored entries."""
    col = np.asarray(col_idx, dtype=np.int64)
    rows = _csr_rows(row_ptr)
    return int(np.unique((rows // b) * _cdiv(k, b) + (col // b)).shape[0])


def fill_ratio_bcsr(nnz, nnzb, b):
    """nnz / (nnz_blocks * b_row * b_col)  (Sec. 2.3)."""
    return nnz / float(nnzb * b * b) if nnzb else 0.0


# --------------------------------------------------------------------------- WCSR


def wcsr_from_csr(m, k, row_ptr, col_idx, vals, wh, b_col):
    """CSR -> WCSR with window height wh and column padding b_col (Sec. 2.3, WCSR paragraph).

    Returns dict(window_row_ptr int32 [ceil(m/wh)+1] in units of columns,
    window_col_idx int32 [P] (-1 on pads), values [wh, P] of vals.dtype).
    """
    vals = np.asarray(vals)
    col = np.asarray(col_idx, dtype=np.int64)
    rows = _csr_rows(row_ptr)
    nwin = _cdiv(m, wh)
    key = (rows // wh) * k + col
    ukeys = np.unique(key)                        # window major, columns ascending
    uwin = ukeys // k
    cnt = np.bincount(uwin, minlength=nwin).astype(np.int64)
    length = _cdiv(cnt, b_col) * b_col            # 0 stays 0
    wptr = np.zeros(nwin + 1, dtype=np.int64)
    wptr[1:] = np.cumsum(length)
    P = int(wptr[-1])
    if P >= 2 ** 31:
        raise ValueError("padded column count does not fit int32")
    first = np.zeros(nwin + 1, dtype=np.int64)
    first[1:] = np.cumsum(cnt)
    rank = np.arange(ukeys.shape[0], dtype=np.int64) - first[uwin]
    ppos = wptr[uwin] + rank                      # padded position of every kept column
    wcol = np.full(P, -1, dtype=np.int32)
    wcol[ppos] = (ukeys % k).astype(np.int32)
    values = np.zeros((wh, P), dtype=vals.dtype)
    values[rows % wh, ppos[np.searchsorted(ukeys, key)]] = vals
    return dict(window_row_ptr=wptr.astype(np.int32), window_col_idx=wcol, values=values)


def wcsr_to_dense(m, k, wh, window_row_ptr, window_col_idx, values):
    """Expand WCSR back to a dense m x k array."""
    nwin = window_row_ptr.shape[0] - 1
    D = np.zeros((nwin * wh, k), dtype=values.dtype)
    for w in range(nwin):
        for q in range(window_row_ptr[w], window_row_ptr[w + 1]):
            c = int(window_col_idx[q])
            if c >= 0:
                D[w * wh:(w + 1) * wh, c] = values[:, q]
    return D[:m]


def wcsr_padded_cols(m, k, row_ptr, col_idx, wh, b_col):
    """Padded column count P of the WCSR form (Sec. 2.3) without building it: per window the
    number of distinct columns, rounded up to a multiple of b_col, summed."""
    col = np.asarray(col_idx, dtype=np.int64)
    rows = _csr_rows(row_ptr)
    ukeys = np.unique((rows // wh) * k + col)
    cnt = np.bincount(ukeys // k, minlength=_cdiv(m, wh)).astype(np.int64)
    return int((_cdiv(cnt, b_col) * b_col).sum())


def fill_ratio_wcsr(nnz, P, wh):
    """Stored-value analogue of the BCSR fill ratio: nnz / (wh * padded columns)."""
    return nnz / float(wh * P) if P else 0.0


# --------------------------------------------------------------------------- split plan


def split_plan(window_row_ptr, T):
    """Task decomposition of Sec. 3.3: windows longer than T columns are cut
    into consecutive chunks of T columns; every chunk is one task.

    Returns int32 array [ntasks, 4] with rows (window, q0, count, slot):
    q0 is the chunk's first column relative to the window start, count its
    number of columns, slot the index of the partial-sum tile the task writes
    (running index over all chunks of windows that have more than one chunk,
    in task order) or -1 when the window is a single task that writes C
    directly.  Empty windows produce no task.
    """
    wptr = np.asarray(window_row_ptr, dtype=np.int64)
    length = np.diff(wptr)
    nchunk = _cdiv(length, T)
    win = np.repeat(np.arange(length.shape[0], dtype=np.int64), nchunk)
    firsttask = np.zeros(length.shape[0] + 1, dtype=np.int64)
    firsttask[1:] = np.cumsum(nchunk)
    cidx = np.arange(win.shape[0], dtype=np.int64) - firsttask[win]
    q0 = cidx * T
    count = np.minimum(T, length[win] - q0)
    is_split = nchunk[win] > 1
    slot = np.where(is_split, np.cumsum(is_split) - 1, -1)
    return np.stack([win, q0, count, slot], axis=1).astype(np.int32)


# --------------------------------------------------------------------------- schedules


def bcsr_row_order(block_row_ptr):
    """Order in which block-rows are scheduled: most stored blocks first, ties by index.

    This is the longest-processing-time-first rule applied to the imbalance
    Sec. 3.5 / Sec. 4.2 (opt6) describe for a persistent kernel with a static
    tile order: a block-row's work is proportional to its number of stored blocks.
    """
    lens = np.diff(np.asarray(block_row_ptr, dtype=np.int64))
    return np.argsort(-lens, kind="stable").astype(np.int32)


def default_split_cols(window_row_ptr, n_bins, fixed_cost=32):
    """Sub-task size used when the caller gives none (the paper only says "fixed-size sub-tasks",
    Sec. 3.3): candidates are one bin's share of the padded columns and its half, quarter and
    eighth, each rounded down to a multiple of 64 and clamped to [128, 65536]; for each, the
    windows are cut into chunks of T and dealt longest first to the lightest bin (cost = columns
    + fixed_cost); the largest candidate whose heaviest bin is within 2 % of the best of the four
    is taken -- as few split windows as the balance allows."""
    import heapq
    wptr = np.asarray(window_row_ptr, dtype=np.int64)
    lens = np.diff(wptr)
    P = int(wptr[-1])

    def max_load(T):
        full, rem = lens // T, lens % T
        full = np.where((rem == 0) & (full > 0), full - 1, full)      # the last chunk of a multiple of T is a chunk of T
        rem = np.where((rem == 0) & (lens > 0), T, rem)
        counts = np.concatenate([np.full(int(full.sum()), T, dtype=np.int64), rem[rem > 0]])
        counts = np.sort(counts)[::-1]
        heap = [0] * n_bins
        mx = 0
        for c in counts.tolist():
            l = heapq.heappop(heap) + c + fixed_cost
            heapq.heappush(heap, l)
            mx = max(mx, l)
        return mx

    cands = [int(min(65536, max(128, ((P // n_bins) >> i) // 64 * 64))) for i in range(4)]
    loads = [max_load(T) for T in cands]
    best = min(loads)
    for T, l in zip(cands, loads):
        if l * 100 <= best * 102:
            return T
    return cands[3]


def task_bins(plan, n_bins, fixed_cost=32):
    """Static schedule of the sub-tasks of Sec. 3.3 over n_bins bins: the
    longest-processing-time rule.  cost(task) = its column count + fixed_cost.
    Tasks are taken heaviest first (ties: lower task index first); each goes to
    the bin whose load is smallest at that moment (ties: lowest bin index).
    Inside a bin tasks are listed in ascending task index.

    Returns (bin_ptr int32 [n_bins+1], bin_tasks int32 [ntasks]).
    """
    import heapq
    cost = plan[:, 2].astype(np.int64) + fixed_cost
    order = np.argsort(-plan[:, 2].astype(np.int64), kind="stable")
    heap = [(0, b) for b in range(n_bins)]
    heapq.heapify(heap)
    members = [[] for _ in range(n_bins)]
    for t in order.tolist():
        load, b = heapq.heappop(heap)
        members[b].append(t)
        heapq.heappush(heap, (load + int(cost[t]), b))
    bin_ptr = np.zeros(n_bins + 1, dtype=np.int64)
    bin_ptr[1:] = np.cumsum([len(x) for x in members])
    tasks = [t for x in members for t in sorted(x)]
    return bin_ptr.astype(np.int32), np.asarray(tasks, dtype=np.int32)


def bcsr_tile_schedule(block_row_ptr, n_tt, slab_w, n_ctas, fixed_cost=4, units=None, lens=None,
                       unit_cost=1, initial=None, return_loads=False):
    """Static schedule of BCSR tiles (block-row, token tile) over n_ctas CTAs.

    Addresses the imbalance Sec. 3.5 / Sec. 4.2 (opt6) report for a fixed tile
    order.  Tiles are taken slab by slab (slab_w consecutive token tiles), inside a
    slab in bcsr_row_order (most stored blocks first), inside a block-row by
    ascending token tile; each goes to the CTA whose load is smallest at that
    moment (ties: lowest CTA), load = sum of (stored blocks + fixed_cost) * unit_cost
    on top of the CTA's initial load (0 unless given); loads carry over between
    slabs.  Returns (cta_ptr int32 [n_ctas+1], tiles int32 [n_tiles, 2]) with every
    CTA's tiles in the order it received them (and the CTAs' final loads when
    return_loads).

    ``units`` / ``lens`` replace the block-rows and their lengths by any list of
    units given in schedule order (a subset of the block-rows, or row groups).
    """
    import heapq
    if units is None:
        brp = np.asarray(block_row_ptr, dtype=np.int64)
        all_lens = np.diff(brp)
        units = bcsr_row_order(brp)
        lens = all_lens[units]
    units = [int(u) for u in units]
    lens = [int(x) for x in lens]
    heap = [(0 if initial is None else int(initial[c]), c) for c in range(n_ctas)]
    heapq.heapify(heap)
    lists = [[] for _ in range(n_ctas)]
    for t0 in range(0, n_tt, slab_w):
        t1 = min(n_tt, t0 + slab_w)
        for I, ln in zip(units, lens):
            cost = (ln + fixed_cost) * unit_cost
            for t in range(t0, t1):
                load, c = heapq.heappop(heap)
                lists[c].append((I, t))
                heapq.heappush(heap, (load + cost, c))
    cta_ptr = np.zeros(n_ctas + 1, dtype=np.int64)
    cta_ptr[1:] = np.cumsum([len(x) for x in lists])
    tiles = np.asarray([p for x in lists for p in x], dtype=np.int32).reshape(-1, 2)
    if return_loads:
        loads = np.zeros(n_ctas, dtype=np.int64)
        for load, c in heap:
            loads[c] = load
        return cta_ptr.astype(np.int32), tiles, loads
    return cta_ptr.astype(np.int32), tiles


def bcsr_k_split(block_row_ptr, n_tt, n_ctas, fixed_cost=4, min_cap=8):
    """K-split of outlier block-rows (the static-schedule answer to the imbalance Sec. 3.5 / 3.6
    discuss: a block-row far longer than the rest makes tiles that no assignment can balance).

    cap = max(min_cap, ceil(n_tt * sum over all block-rows of (stored blocks + fixed_cost) /
    (4 * n_ctas))): a quarter of one CTA's mean load.  A block-row with more stored blocks than cap is
    cut into parts = ceil(len / cap) contiguous ranges of its stored blocks, part j = blocks
    [floor(j * len / parts), floor((j + 1) * len / parts)) of the row; every part computes a partial
    C tile and the parts are summed in part order afterwards.

    Returns None when no block-row exceeds cap, else int32 [n_units, 4] rows (block-row, first
    stored block, end stored block, slot): block-rows in bcsr_row_order, parts in order; slot = -1
    for an unsplit row, else the running index of the part counted over the split rows in ascending
    block-row index (parts ascending).
    """
    brp = np.asarray(block_row_ptr, dtype=np.int64)
    lens = np.diff(brp)
    total = int((lens + fixed_cost).sum()) * n_tt
    cap = max(min_cap, -(-total // (4 * n_ctas)))
    if lens.size == 0 or int(lens.max()) <= cap:
        return None
    first_slot = {}
    nslots = 0
    for I in range(lens.shape[0]):
        if lens[I] > cap:
            first_slot[I] = nslots
            nslots += -(-int(lens[I]) // cap)
    units = []
    for I in bcsr_row_order(brp).tolist():
        L = int(lens[I])
        if L <= cap:
            units.append((I, int(brp[I]), int(brp[I + 1]), -1))
        else:
            parts = -(-L // cap)
            for j in range(parts):
                units.append((I, int(brp[I]) + j * L // parts, int(brp[I]) + (j + 1) * L // parts, first_slot[I] + j))
    return np.asarray(units, dtype=np.int32).reshape(-1, 4)


def bcsr_k_split_order(units):
    """Schedule order of the K-split units: most stored blocks first, stable."""
    ln = (units[:, 2] - units[:, 1]).astype(np.int64)
    return np.argsort(-ln, kind="stable").astype(np.int32)


BCSR_GROUP_WORK_LIMIT = 1 << 27


def bcsr_row_groups(block_row_ptr, block_col_idx, b, min_fill_pct):
    """Row groups of the BCSR kernel (a device-side regrouping with no counterpart in the
    paper, whose BCSR blocks are all b x b, Sec. 2.3): R = 128 // b block-rows that store
    blocks in mostly the same block columns are computed together, one 128-row stacked block
    per block column of their union.

    Rule (grouping by similarity): walk bcsr_row_order (most stored blocks first, stable).  A
    block-row that is non-empty and not yet in a group is a seed; its partners are the R - 1 other
    free non-empty block-rows that share the most block columns with it (at least one; ties: the
    one earlier in the order); with fewer than R - 1 such rows the seed forms no group.  The
    candidate (seed and partners, listed in the order) is accepted when 100 * (stored blocks of
    its rows) >= min_fill_pct * R * |union of their block columns|; its rows then leave the free
    set, otherwise all of them stay free (the seed is not tried again as a seed, but may become a
    partner).  The search stops for good once the work it has charged -- per seed, the sum over
    the seed's block columns of the number of block-rows that store that column -- would pass
    BCSR_GROUP_WORK_LIMIT.  Returns (rows int32 [ng, R], ptr int32 [ng+1], col_idx int32 [ns]):
    member rows in the order, and per group the ascending union of block columns.
    """
    brp = np.asarray(block_row_ptr, dtype=np.int64)
    bci = np.asarray(block_col_idx, dtype=np.int64)
    R = 128 // b
    nbr = brp.shape[0] - 1
    order = bcsr_row_order(brp)
    pos = np.empty(nbr, dtype=np.int64)
    pos[order] = np.arange(nbr)
    colsets = [set(bci[brp[I]:brp[I + 1]].tolist()) for I in range(nbr)]
    degree = np.bincount(bci, minlength=int(bci.max()) + 1 if bci.size else 1)
    by_col = {}
    for I in range(nbr):
        for J in colsets[I]:
            by_col.setdefault(J, []).append(I)
    free = [len(colsets[I]) > 0 for I in range(nbr)]
    rows, ptr, cols = [], [0], []
    work = 0
    for s in order.tolist():
        if not free[s]:
            continue
        w = int(sum(degree[J] for J in colsets[s]))
        if work + w > BCSR_GROUP_WORK_LIMIT:
            break
        work += w
        overlap = {}
        for J in colsets[s]:
            for r in by_col[J]:
                if r != s and free[r]:
                    overlap[r] = overlap.get(r, 0) + 1
        if len(overlap) < R - 1:
            continue
        partners = sorted(overlap, key=lambda r: (-overlap[r], pos[r]))[:R - 1]
        members = sorted([s] + partners, key=lambda r: pos[r])
        stored = sum(len(colsets[r]) for r in members)
        union = sorted(set().union(*[colsets[r] for r in members]))
        if 100 * stored >= min_fill_pct * R * len(union):
            for r in members:
                free[r] = False
            rows.append(members)
            cols.extend(union)
            ptr.append(len(cols))
    return (np.asarray(rows, dtype=np.int32).reshape(-1, R), np.asarray(ptr, dtype=np.int32),
            np.asarray(cols, dtype=np.int32))


def padded_width(N, BN):
    """Dense width after padding to a whole number of N-tiles of BN columns, and the share of
    the padded width that is padding (the cost Sec. 4.3 discusses for its N-tile sweep)."""
    padded = -(-N // BN) * BN
    return padded, (padded - N) / N
