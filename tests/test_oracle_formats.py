"""Pins for the format oracle (Sec. 2.3 BCSR / WCSR, Sec. 3.3 split plan).

The numpy definitions in oracle/formats.py are compared with per-element
Python constructions written here from the paper's text, with round trips,
with the array-length and fill-ratio formulas the paper prints, and with
special cases whose answer is known in closed form.
"""
import numpy as np
import pytest

from oracle import formats as F
from paper_2604_17834_b200 import workloads as wl


def _dense(a):
    m, k = a["m"], a["k"]
    D = np.zeros((m, k), dtype=a["vals"].dtype)
    mask = np.zeros((m, k), dtype=bool)
    for i in range(m):
        for p in range(a["row_ptr"][i], a["row_ptr"][i + 1]):
            D[i, a["col_idx"][p]] = a["vals"][p]
            mask[i, a["col_idx"][p]] = True
    return D, mask


def _brute_bcsr(D, mask, b):
    m, k = D.shape
    nbr, nbc = -(-m // b), -(-k // b)
    ptr, idx, blocks = [0], [], []
    for I in range(nbr):
        for J in range(nbc):
            sub = mask[I * b:(I + 1) * b, J * b:(J + 1) * b]
            if sub.any():
                blk = np.zeros((b, b), dtype=D.dtype)
                d = D[I * b:(I + 1) * b, J * b:(J + 1) * b]
                blk[:d.shape[0], :d.shape[1]] = d
                idx.append(J)
                blocks.append(blk)
        ptr.append(len(idx))
    return ptr, idx, blocks


def _brute_wcsr(D, mask, wh, b_col):
    m, k = D.shape
    nwin = -(-m // wh)
    ptr, idx, cols_vals = [0], [], []
    for w in range(nwin):
        rows = range(w * wh, min(m, (w + 1) * wh))
        kept = [c for c in range(k) if any(mask[r, c] for r in rows)]
        for c in kept:
            v = np.zeros(wh, dtype=D.dtype)
            for r in rows:
                v[r - w * wh] = D[r, c]
            idx.append(c)
            cols_vals.append(v)
        while len(idx) % b_col:
            idx.append(-1)
            cols_vals.append(np.zeros(wh, dtype=D.dtype))
        ptr.append(len(idx))
    vals = np.stack(cols_vals, axis=1) if cols_vals else np.zeros((wh, 0), dtype=D.dtype)
    return ptr, idx, vals


CASES = [(37, 29, 0.15), (64, 64, 0.05), (16, 50, 0.5), (70, 130, 0.02)]


@pytest.mark.parametrize("m,k,dens", CASES)
@pytest.mark.parametrize("b", [4, 16, 32])
def test_bcsr_matches_brute_force_and_round_trips(m, k, dens, b):
    a = wl.random_csr(100 + m + b, m, k, dens, "fp16", empty_rows=(0, m - 1))
    D, mask = _dense(a)
    f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
    ptr, idx, blocks = _brute_bcsr(D, mask, b)
    assert f["block_row_ptr"].tolist() == ptr
    assert f["block_col_idx"].tolist() == idx
    assert f["block_row_ptr"].shape[0] == -(-m // b) + 1            # Sec. 2.3 array lengths
    assert f["blocks"].shape == (len(idx), b, b)
    if blocks:
        assert np.array_equal(f["blocks"].view(np.uint16), np.stack(blocks).view(np.uint16))
    back = F.bcsr_to_dense(m, k, b, f["block_row_ptr"], f["block_col_idx"], f["blocks"])
    assert np.array_equal(back.view(np.uint16), D.view(np.uint16))
    # every stored CSR entry is found again: nnz preserved
    assert int(mask.sum()) == a["col_idx"].shape[0]
    nb = -(-m // b) * -(-k // b)
    assert len(idx) == sum(
        mask[I * b:(I + 1) * b, J * b:(J + 1) * b].any()
        for I in range(-(-m // b)) for J in range(-(-k // b)))
    assert len(idx) <= nb
    # the count-only helper agrees with the bitmap brute force
    assert F.bcsr_block_count(m, k, a["row_ptr"], a["col_idx"], b) == len(idx)


def test_bcsr_structural_zero_keeps_block():
    # an explicitly stored 0.0 marks its block (structural reading)
    row_ptr = np.array([0, 1, 1, 1, 1], np.int64)
    f = F.bcsr_from_csr(4, 4, row_ptr, np.array([3], np.int32), np.array([0.0], np.float32), 2)
    assert f["block_row_ptr"].tolist() == [0, 1, 1] and f["block_col_idx"].tolist() == [1]


def test_bcsr_dense_and_block_diagonal_and_fill_ratio():
    m = k = 24
    b = 8
    a = wl.random_csr(1, m, k, 2.0, "tf32")                 # density >= 1 -> fully dense
    f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
    assert f["block_col_idx"].shape[0] == 9
    assert F.fill_ratio_bcsr(m * k, 9, b) == 1.0
    mask = np.eye(3, dtype=bool)
    rp, ci = wl.csr_from_block_mask(mask, b, m, k)
    f = F.bcsr_from_csr(m, k, rp, ci, np.ones(ci.shape[0], np.float32), b)
    assert f["block_col_idx"].tolist() == [0, 1, 2]
    assert f["block_row_ptr"].tolist() == [0, 1, 2, 3]
    # one entry per block: fill ratio = nnz / (nnzb * b * b)
    rp = np.array([0, 1] + [1] * 7 + [2] + [2] * 15, np.int64)
    f = F.bcsr_from_csr(m, k, rp, np.array([0, 9], np.int32), np.ones(2, np.float32), b)
    assert F.fill_ratio_bcsr(2, f["block_col_idx"].shape[0], b) == 2 / (2 * 64)


@pytest.mark.parametrize("m,k,dens", CASES)
@pytest.mark.parametrize("wh,b_col", [(4, 2), (16, 8), (16, 16), (1, 4), (16, 32), (64, 32)])
def test_wcsr_matches_brute_force_and_round_trips(m, k, dens, wh, b_col):
    a = wl.random_csr(200 + m + wh, m, k, dens, "fp16", empty_rows=tuple(range(min(wh, m))))
    D, mask = _dense(a)
    f = F.wcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], wh, b_col)
    ptr, idx, vals = _brute_wcsr(D, mask, wh, b_col)
    assert f["window_row_ptr"].tolist() == ptr
    assert f["window_col_idx"].tolist() == idx
    assert f["values"].shape == (wh, len(idx))               # one 2-D array [b_row, padded cols]
    assert np.array_equal(f["values"].view(np.uint16), vals.view(np.uint16))
    assert f["window_row_ptr"][1] == 0                        # first window emptied above
    lens = np.diff(f["window_row_ptr"])
    assert np.all(lens % b_col == 0)
    pads = f["window_col_idx"] < 0
    assert np.all(f["window_col_idx"][pads] == -1)
    assert not f["values"][:, pads].any()
    for w in range(len(ptr) - 1):
        c = f["window_col_idx"][ptr[w]:ptr[w + 1]]
        c = c[c >= 0]
        assert np.all(np.diff(c) > 0)                         # strictly ascending
    back = F.wcsr_to_dense(m, k, wh, f["window_row_ptr"], f["window_col_idx"], f["values"])
    assert np.array_equal(back.view(np.uint16), D.view(np.uint16))
    # the count-only helper agrees with the per-element construction
    assert F.wcsr_padded_cols(m, k, a["row_ptr"], a["col_idx"], wh, b_col) == len(idx)


def test_wcsr_height_one_is_padded_csr():
    a = wl.random_csr(5, 20, 33, 0.2, "tf32")
    f = F.wcsr_from_csr(20, 33, a["row_ptr"], a["col_idx"], a["vals"], 1, 4)
    for i in range(20):
        lo, hi = a["row_ptr"][i], a["row_ptr"][i + 1]
        q0, q1 = f["window_row_ptr"][i], f["window_row_ptr"][i + 1]
        n = hi - lo
        assert q1 - q0 == -(-n // 4) * 4
        assert np.array_equal(f["window_col_idx"][q0:q0 + n], a["col_idx"][lo:hi])
        assert np.array_equal(f["values"][0, q0:q0 + n], a["vals"][lo:hi])


def test_wcsr_identical_rows_and_diagonal():
    wh, b_col, k = 8, 4, 40
    cols = np.array([1, 5, 6, 20, 39], np.int32)
    rp = np.arange(0, 5 * wh + 1, 5, dtype=np.int64)
    f = F.wcsr_from_csr(wh, k, rp, np.tile(cols, wh), np.ones(5 * wh, np.float32), wh, b_col)
    assert f["window_row_ptr"].tolist() == [0, 8]              # pad(5) = 8
    assert f["window_col_idx"].tolist() == [1, 5, 6, 20, 39, -1, -1, -1]
    n = 24
    f = F.wcsr_from_csr(n, n, np.arange(n + 1, dtype=np.int64), np.arange(n, dtype=np.int32),
                        np.arange(1, n + 1, dtype=np.float32), wh, b_col)
    assert np.all(np.diff(f["window_row_ptr"]) == wh)          # pad(wh) = wh columns per window
    assert np.array_equal(f["values"][np.arange(n) % wh, np.arange(n)], np.arange(1, n + 1))


def _brute_plan(wptr, T):
    tasks, slot = [], 0
    for w in range(len(wptr) - 1):
        L = wptr[w + 1] - wptr[w]
        chunks = [(q0, min(T, L - q0)) for q0 in range(0, L, T)]
        for q0, c in chunks:
            if len(chunks) > 1:
                tasks.append((w, q0, c, slot))
                slot += 1
            else:
                tasks.append((w, q0, c, -1))
    return tasks


@pytest.mark.parametrize("T", [8, 16, 64, 4096])
def test_split_plan(T):
    rng = np.random.default_rng(T)
    lens = rng.choice([0, 8, 16, 24, 64, 72, 200, 1000], size=60)
    wptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    plan = F.split_plan(wptr, T)
    assert plan.dtype == np.int32
    assert [tuple(r) for r in plan.tolist()] == _brute_plan(wptr.tolist(), T)
    assert plan[:, 2].sum() == wptr[-1]                        # chunks tile all padded columns
    assert np.all(plan[:, 2] <= T) and np.all(plan[:, 2] % 8 == 0) and np.all(plan[:, 2] > 0)
    if T >= lens.max():
        assert np.all(plan[:, 3] == -1)                        # nothing split
    # chunks of one window are consecutive, in order, and tile [0, len)
    for w in np.unique(plan[:, 0]):
        rows = plan[plan[:, 0] == w]
        assert rows[0, 1] == 0
        assert np.all(rows[1:, 1] == rows[:-1, 1] + rows[:-1, 2])
        assert rows[-1, 1] + rows[-1, 2] == lens[w]


def _brute_bins(plan, n_bins, fixed_cost=32):
    """The longest-processing-time rule with plain loops: heaviest task first (ties: lower task
    index), each into the bin with the smallest load so far (ties: lowest bin index)."""
    order = sorted(range(len(plan)), key=lambda t: (-int(plan[t][2]), t))
    loads = [0] * n_bins
    members = [[] for _ in range(n_bins)]
    for t in order:
        b = min(range(n_bins), key=lambda j: (loads[j], j))
        members[b].append(t)
        loads[b] += int(plan[t][2]) + fixed_cost
    return members, loads


@pytest.mark.parametrize("seed,n_bins", [(1, 1), (2, 3), (3, 7), (4, 16), (5, 5)])
def test_task_bins_match_brute_force(seed, n_bins):
    rng = np.random.default_rng(seed)
    # many equal lengths on purpose: the tie rules decide most placements
    lens = rng.choice([0, 8, 8, 16, 16, 16, 64, 72, 200, 1000], size=80)
    wptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    plan = F.split_plan(wptr, 64)
    bin_ptr, bin_tasks = F.task_bins(plan, n_bins)
    members, loads = _brute_bins(plan.tolist(), n_bins)
    assert bin_ptr.tolist() == np.concatenate([[0], np.cumsum([len(x) for x in members])]).tolist()
    assert bin_tasks.tolist() == [t for x in members for t in sorted(x)]
    # every task once; the classical bound of the rule: no bin exceeds the mean by more than one task
    assert sorted(bin_tasks.tolist()) == list(range(plan.shape[0]))
    cost = plan[:, 2].astype(np.int64) + 32
    assert max(loads) <= cost.sum() / n_bins + cost.max()


def _brute_split_size(wptr, n_bins, fixed_cost=32):
    """Default sub-task size written out with plain loops only (no call into the oracle's plan or
    bins): the four candidates, each window cut into chunks, chunks dealt heaviest first."""
    lens = [int(wptr[i + 1] - wptr[i]) for i in range(len(wptr) - 1)]
    P = sum(lens)
    cands = [min(65536, max(128, ((P // n_bins) >> i) // 64 * 64)) for i in range(4)]
    worst = []
    for T in cands:
        chunks = []
        for L in lens:
            q = 0
            while q < L:
                chunks.append(min(T, L - q))
                q += T
        chunks.sort(reverse=True)
        loads = [0] * n_bins
        for c in chunks:
            j = min(range(n_bins), key=lambda b: (loads[b], b))
            loads[j] += c + fixed_cost
        worst.append(max(loads))
    best = min(worst)
    for T, l in zip(cands, worst):
        if l * 100 <= best * 102:
            return T
    return cands[3]


@pytest.mark.parametrize("seed,n_bins", [(11, 4), (12, 9), (13, 16)])
def test_default_split_cols_matches_plain_loops(seed, n_bins):
    rng = np.random.default_rng(seed)
    lens = rng.choice([0, 16, 32, 48, 64, 320, 2048, 9000], size=300, p=[.1, .3, .2, .15, .1, .1, .04, .01])
    wptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    assert F.default_split_cols(wptr, n_bins) == _brute_split_size(wptr, n_bins)
    # closed-form cases: one heavy window among light ones balances at a whole share; equal heavy
    # windows, one more than bins, need a smaller size than the share
    wp = np.concatenate(([0], np.cumsum([10000] + [64] * 1000)))
    assert F.default_split_cols(wp, 8) == _brute_split_size(wp, 8) == (74000 // 8) // 64 * 64
    wp = np.concatenate(([0], np.cumsum([4096] * 9)))
    assert F.default_split_cols(wp, 8) == _brute_split_size(wp, 8) < 4608


def _brute_k_split(brp, n_tt, n_ctas, fixed=4, min_cap=8):
    """K-split written with plain loops: cap, parts per long block-row, slots in ascending
    block-row order, units in schedule order of the block-rows."""
    lens = [brp[i + 1] - brp[i] for i in range(len(brp) - 1)]
    total = n_tt * sum(l + fixed for l in lens)
    cap = max(min_cap, (total + 4 * n_ctas - 1) // (4 * n_ctas))
    if not lens or max(lens) <= cap:
        return cap, None
    slot_of, ns = {}, 0
    for i, l in enumerate(lens):
        if l > cap:
            slot_of[i] = ns
            ns += (l + cap - 1) // cap
    order = sorted(range(len(lens)), key=lambda i: (-lens[i], i))
    units = []
    for i in order:
        l = lens[i]
        if l <= cap:
            units.append((i, brp[i], brp[i + 1], -1))
        else:
            parts = (l + cap - 1) // cap
            for j in range(parts):
                units.append((i, brp[i] + j * l // parts, brp[i] + (j + 1) * l // parts, slot_of[i] + j))
    return cap, units


@pytest.mark.parametrize("seed,n_tt,n_ctas", [(1, 4, 16), (2, 1, 3), (3, 16, 148), (4, 2, 40), (5, 8, 148)])
def test_k_split_matches_brute_force_and_tiles_the_rows(seed, n_tt, n_ctas):
    rng = np.random.default_rng(seed)
    lens = rng.choice([0, 0, 1, 2, 3, 5, 9, 17, 64, 64, 128], size=70)
    brp = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cap, want = _brute_k_split(brp.tolist(), n_tt, n_ctas)
    got = F.bcsr_k_split(brp, n_tt, n_ctas)
    if want is None:
        assert got is None
        return
    assert got.dtype == np.int32 and [tuple(r) for r in got.tolist()] == want
    # the parts of a block-row tile its stored blocks in order, none longer than cap, sizes within one of each other
    for I in np.unique(got[:, 0]):
        u = got[got[:, 0] == I]
        assert u[0, 1] == brp[I] and u[-1, 2] == brp[I + 1] and np.all(u[1:, 1] == u[:-1, 2])
        ln = u[:, 2] - u[:, 1]
        assert ln.max() <= cap and ln.max() - ln.min() <= 1
        assert (u.shape[0] == 1) == (u[0, 3] == -1)
        if u.shape[0] > 1:
            assert np.all(np.diff(u[:, 3]) == 1)
    # slots number the parts of split rows in ascending block-row order
    parts = got[got[:, 3] >= 0]
    by_row = parts[np.lexsort((parts[:, 1], parts[:, 0]))]
    assert np.array_equal(by_row[:, 3], np.arange(by_row.shape[0]))
    # no unit longer than a quarter of a CTA's mean load (or the minimum cap)
    total = n_tt * int((np.diff(brp) + 4).sum())
    assert cap == max(8, -(-total // (4 * n_ctas)))
    # schedule order: most stored blocks first, stable
    o = F.bcsr_k_split_order(got)
    ln = (got[:, 2] - got[:, 1])[o]
    assert np.all(np.diff(ln) <= 0)
    for a, b in zip(o[:-1], o[1:]):
        if got[a, 2] - got[a, 1] == got[b, 2] - got[b, 1]:
            assert a < b


def test_k_split_special_cases():
    # equal rows: nothing exceeds a quarter of the mean load unless there are very few of them
    brp = np.arange(0, 65 * 10, 10, dtype=np.int32)
    assert F.bcsr_k_split(brp, 4, 8) is None
    # one row of 100 blocks among 99 single-block rows on 100 CTAs: cap = max(8, ceil(2 * 599 / 400)) = 8 -> 13 parts
    brp = np.concatenate([[0], np.cumsum([100] + [1] * 99)]).astype(np.int32)
    u = F.bcsr_k_split(brp, 2, 100)
    parts = u[u[:, 0] == 0]
    assert parts.shape[0] == 13 and parts[:, 3].tolist() == list(range(13))
    assert (parts[:, 2] - parts[:, 1]).sum() == 100 and np.all(u[u[:, 0] > 0][:, 3] == -1)


def test_generators_are_deterministic_and_shaped():
    a1, a2 = wl.bcsr_tiny(), wl.bcsr_tiny()
    assert np.array_equal(a1["col_idx"], a2["col_idx"]) and np.array_equal(a1["vals"], a2["vals"])
    g = wl.bcsr_llm(m=1024, k=512)
    f = F.bcsr_from_csr(1024, 512, g["row_ptr"], g["col_idx"], g["vals"], 64)
    assert f["block_col_idx"].shape[0] == 128 - int(np.floor(0.9 * 128))
    s = wl.bcsr_sweep(9, m=1024, k=1024, b=32, density=0.2)
    f = F.bcsr_from_csr(1024, 1024, s["row_ptr"], s["col_idx"], s["vals"], 32)
    per_row = np.diff(f["block_row_ptr"])
    assert (per_row == 32).sum() >= 3 and (per_row == 0).sum() >= 6
    r = wl.rmat(scale=10, edge_factor=8)
    assert r["m"] == 1024 and np.all(np.diff(r["row_ptr"]) >= 0)
    keys = np.repeat(np.arange(1024), np.diff(r["row_ptr"])) * 1024 + r["col_idx"]
    assert np.all(np.diff(keys) > 0)                           # sorted, duplicates merged
    w = wl.wcsr_irregular(m=2000)
    keys = np.repeat(np.arange(2000), np.diff(w["row_ptr"])) * 2000 + w["col_idx"]
    assert np.all(np.diff(keys) > 0)
    assert np.diff(w["row_ptr"]).min() >= 1


def test_tile_padding_numbers_of_the_paper():
    """tests/golden/sec4_3_tile_padding.txt: the padded widths and waste percentages Sec. 4.3
    prints for its N-tile sweep (waste relative to the unpadded width, rounded as printed)."""
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "sec4_3_tile_padding.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 5
    for N, BN, padded, pct in ((int(a), int(b), int(c), int(d)) for a, b, c, d in rows):
        got_padded, waste = F.padded_width(N, BN)
        assert got_padded == padded
        assert round(100.0 * waste) == pct


# --------------------------------------------------------------------------- schedules and row groups


def _brute_schedule(units, lens, n_tt, slab_w, n_ctas, fixed, unit_cost, initial):
    """The longest-first dealing rule with a plain argmin instead of a heap."""
    loads = [0] * n_ctas if initial is None else [int(x) for x in initial]
    lists = [[] for _ in range(n_ctas)]
    for t0 in range(0, n_tt, slab_w):
        for I, ln in zip(units, lens):
            for t in range(t0, min(n_tt, t0 + slab_w)):
                c = min(range(n_ctas), key=lambda j: (loads[j], j))
                lists[c].append((int(I), t))
                loads[c] += (int(ln) + fixed) * unit_cost
    return lists, loads


@pytest.mark.parametrize("seed,n_ctas,n_tt,slab_w", [(0, 3, 5, 2), (1, 7, 4, 4), (2, 1, 3, 1), (3, 5, 1, 1)])
def test_tile_schedule_matches_brute_force(seed, n_ctas, n_tt, slab_w):
    rng = np.random.default_rng(seed)
    lens_all = rng.integers(0, 9, size=11)
    brp = np.concatenate(([0], np.cumsum(lens_all)))
    order = F.bcsr_row_order(brp)
    assert np.all(np.diff(lens_all[order]) <= 0)                                   # longest first
    assert all(order[i] < order[i + 1] for i in range(10) if lens_all[order[i]] == lens_all[order[i + 1]])   # stable
    ptr, tiles = F.bcsr_tile_schedule(brp, n_tt, slab_w, n_ctas)
    lists, _ = _brute_schedule(order, lens_all[order], n_tt, slab_w, n_ctas, 4, 1, None)
    assert [tuple(x) for x in tiles.tolist()] == [p for l in lists for p in l]
    assert ptr.tolist() == np.concatenate(([0], np.cumsum([len(l) for l in lists]))).tolist()
    # a subset of the units, weighted costs and a head start per CTA
    units = order[1::2]
    initial = rng.integers(0, 400, size=n_ctas)
    ptr2, tiles2, loads2 = F.bcsr_tile_schedule(None, n_tt, slab_w, n_ctas, fixed_cost=3, units=units, lens=lens_all[units],
                                                unit_cost=17, initial=initial, return_loads=True)
    lists2, bl = _brute_schedule(units, lens_all[units], n_tt, slab_w, n_ctas, 3, 17, initial)
    assert [tuple(x) for x in tiles2.tolist()] == [p for l in lists2 for p in l]
    assert loads2.tolist() == bl
    assert loads2.sum() == initial.sum() + 17 * n_tt * int((lens_all[units] + 3).sum())


def _brute_groups(rows_cols, R, min_fill_pct):
    """rows_cols: list of sets of block columns per block-row.  The similarity rule with plain
    set intersections against every other free block-row (no inverted index)."""
    order = sorted(range(len(rows_cols)), key=lambda i: (-len(rows_cols[i]), i))
    pos = {r: i for i, r in enumerate(order)}
    free = {i for i in range(len(rows_cols)) if rows_cols[i]}
    out = []
    for s in order:
        if s not in free:
            continue
        ov = [(len(rows_cols[s] & rows_cols[r]), r) for r in free if r != s]
        ov = [(n, r) for n, r in ov if n > 0]
        if len(ov) < R - 1:
            continue
        ov.sort(key=lambda x: (-x[0], pos[x[1]]))
        cand = sorted([s] + [r for _, r in ov[:R - 1]], key=lambda r: pos[r])
        union = set().union(*[rows_cols[i] for i in cand])
        stored = sum(len(rows_cols[i]) for i in cand)
        if 100 * stored >= min_fill_pct * R * len(union):
            out.append((cand, sorted(union)))
            free -= set(cand)
    return out


@pytest.mark.parametrize("b,seed,fill", [(16, 0, 30), (32, 1, 45), (64, 2, 75), (16, 3, 1), (32, 4, 100), (64, 5, 50)])
def test_row_groups_match_brute_force(b, seed, fill):
    rng = np.random.default_rng(seed)
    R = 128 // b
    nbr, nbc = 4 * R + 3, 12
    dens = rng.choice([0.0, 0.2, 0.6, 1.0], size=nbr)
    mask = rng.random((nbr, nbc)) < dens[:, None]
    brp = np.concatenate(([0], np.cumsum(mask.sum(axis=1)))).astype(np.int32)
    bci = np.concatenate([np.flatnonzero(mask[i]) for i in range(nbr)]).astype(np.int32)
    rows, ptr, cols = F.bcsr_row_groups(brp, bci, b, fill)
    want = _brute_groups([set(np.flatnonzero(mask[i]).tolist()) for i in range(nbr)], R, fill)
    assert rows.tolist() == [c for c, _ in want]
    assert ptr.tolist() == np.concatenate(([0], np.cumsum([len(u) for _, u in want]))).astype(int).tolist()
    assert cols.tolist() == [j for _, u in want for j in u]
    assert len(set(rows.reshape(-1).tolist())) == rows.size                          # a block-row is in at most one group
    assert all(mask[i].any() for i in rows.reshape(-1))                              # and never empty


def test_row_groups_special_cases():
    b, R = 32, 4
    # identical block-rows: the union is every row's own column set, fill 100 %
    cols = np.array([1, 4, 5, 9], dtype=np.int32)
    brp = np.arange(0, 4 * 9, 4, dtype=np.int32)                                     # 8 block-rows of 4 blocks
    bci = np.tile(cols, 8)
    rows, ptr, gcols = F.bcsr_row_groups(brp, bci, b, 100)
    assert rows.tolist() == [[0, 1, 2, 3], [4, 5, 6, 7]] and ptr.tolist() == [0, 4, 8] and gcols.tolist() == cols.tolist() * 2
    # block-diagonal: no two block-rows share a block column, so nothing is similar to anything
    brp = np.arange(9, dtype=np.int32)
    bci = np.arange(8, dtype=np.int32)
    assert F.bcsr_row_groups(brp, bci, b, 1)[0].shape[0] == 0
    # families scattered over the index range (block-row i belongs to family i % 3, all members of a
    # family store the same columns, all lengths equal): neighbours in the order belong to different
    # families, the groups are the families
    fam = [np.array([0, 1, 2, 3]), np.array([10, 11, 12, 13]), np.array([20, 21, 22, 23])]
    bci = np.concatenate([fam[i % 3] for i in range(12)]).astype(np.int32)
    brp = np.arange(0, 4 * 13, 4, dtype=np.int32)
    rows, ptr, gcols = F.bcsr_row_groups(brp, bci, b, 100)
    assert rows.tolist() == [[0, 3, 6, 9], [1, 4, 7, 10], [2, 5, 8, 11]]
    assert gcols.tolist() == fam[0].tolist() + fam[1].tolist() + fam[2].tolist()
    # partners are the most similar rows, not the next ones in the order: row 0 = {0..7} (longest),
    # rows 1-3 = {0}, rows 4-6 = {0, 1}.  Seed 0 takes rows 4, 5, 6 (overlap 2 beats overlap 1):
    # fill (8 + 6) / (4 * 8) = 44 %.  At 50 % that group is rejected, row 0 stays free, and the
    # seeds 4, 5, 6 each pick row 0 again (overlap 2, earliest in the order): rejected as well
    bci = np.array(list(range(8)) + [0] * 3 + [0, 1] * 3, dtype=np.int32)
    brp = np.array([0, 8, 9, 10, 11, 13, 15, 17], dtype=np.int32)
    rows, ptr, gcols = F.bcsr_row_groups(brp, bci, b, 40)
    assert rows.tolist() == [[0, 4, 5, 6]]
    rows, ptr, gcols = F.bcsr_row_groups(brp, bci, b, 50)
    assert rows.tolist() == []
    # fewer non-empty block-rows than a group needs: nothing to group
    brp = np.array([0, 3, 3, 3, 6, 6, 6, 6, 6], dtype=np.int32)
    bci = np.array([0, 1, 2, 0, 1, 2], dtype=np.int32)
    assert F.bcsr_row_groups(brp, bci, b, 1)[0].shape[0] == 0
