"""CPU tests of the library's host logic through the C ABI (host_only handles):
format construction, split plan and schedules must equal the oracle bit for bit;
malformed input must be rejected with the documented codes; every symbol the
header declares must be exported.  No CUDA call is made here.
"""
import os
import re

import numpy as np
import pytest

from oracle import formats as F
from paper_2604_17834_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import build
    build.build()
    from paper_2604_17834_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(lib):
    import ctypes
    header = open(os.path.join(ROOT, "include", "spmm_b200.h")).read()
    declared = set(re.findall(r"\b(spmm_[a-z0-9_]+)\s*\(", header))
    assert declared == set(lib.EXPORTED_SYMBOLS)
    so = ctypes.CDLL(lib.LIB_PATH)
    for name in declared:
        assert getattr(so, name) is not None
    assert lib.spmm_status_string(0) == "ok"
    assert "wait" in lib.spmm_status_string(lib.SPMM_ERR_DEV_TIMEOUT)


def _bits(a):
    a = np.ascontiguousarray(a)
    return a.view({1: np.uint8, 2: np.uint16, 4: np.uint32}[a.dtype.itemsize])


BCSR_CASES = [
    ("bf16", 512, 512, 64), ("fp16", 300, 410, 16), ("fp16", 257, 129, 32),
    ("bf16", 640, 384, 128), ("fp16", 64, 64, 64), ("tf32", 300, 260, 64), ("tf32", 130, 513, 16),
]


@pytest.mark.parametrize("dtype,m,k,b", BCSR_CASES)
def test_bcsr_format_is_bit_exact(lib, dtype, m, k, b):
    a = wl.random_csr(31 + m, m, k, 0.01, dtype, empty_rows=tuple(range(min(b, m))))
    h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b, host_only=True)
    try:
        f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_ROW_PTR, np.int32), f["block_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"])
        got = lib.spmm_export(h, lib.X_BCSR_BLOCKS, wl.storage_np_dtype(dtype))
        assert np.array_equal(_bits(got), _bits(f["blocks"]).ravel())
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_ROW_ORDER, np.int32), F.bcsr_row_order(f["block_row_ptr"]))
        info = lib.spmm_get_info(h, 256)
        nnzb = f["block_col_idx"].shape[0]
        assert info["n_units"] == nnzb and info["stored_values"] == nnzb * b * b
        assert info["nnz"] == a["col_idx"].shape[0]
        assert info["fill_ratio"] == pytest.approx(F.fill_ratio_bcsr(info["nnz"], nnzb, b))
        assert info["n_empty"] == int((np.diff(f["block_row_ptr"]) == 0).sum()) >= 1
        assert info["flops_stored"] == 2.0 * nnzb * b * b * 256
        rows_touched = min(k, np.unique(f["block_col_idx"]).shape[0] * b)
        assert info["bytes_b_touched"] == rows_touched * 256 * wl.elem_size(dtype)
        assert info["bytes_c"] == m * 256 * 4
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_run(h, 16, 16, 256)
        assert e.value.code == lib.SPMM_ERR_HOST_ONLY
    finally:
        lib.spmm_destroy(h)


def test_bcsr_workload_generators_round_trip(lib):
    a = wl.bcsr_tiny()
    h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64, host_only=True)
    f = F.bcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], 64)
    assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCKS, np.uint16), f["blocks"].ravel())
    assert lib.spmm_get_info(h)["fill_ratio"] == 1.0
    lib.spmm_destroy(h)
    s = wl.bcsr_sweep(77, m=2048, k=2048, b=32, density=0.1)
    h = lib.spmm_bcsr_create_csr(2048, 2048, s["row_ptr"], s["col_idx"], s["vals"], "fp16", 32, host_only=True)
    f = F.bcsr_from_csr(2048, 2048, s["row_ptr"], s["col_idx"], s["vals"], 32)
    order = lib.spmm_export(h, lib.X_BCSR_ROW_ORDER, np.int32)
    assert np.array_equal(order, F.bcsr_row_order(f["block_row_ptr"]))
    lens = np.diff(f["block_row_ptr"])[order]
    assert np.all(np.diff(lens) <= 0) and lens[0] == 64 and lens[-1] == 0
    lib.spmm_destroy(h)


@pytest.mark.parametrize("b,N,n_ctas,k_split", [(64, 4096, 148, 0), (16, 1024, 7, 0), (128, 640, 5, 0), (32, 200, 3, 0),
                                                (64, 4096, 148, 1), (64, 1024, 148, 1), (128, 4096, 148, 1), (16, 4096, 148, 1),
                                                (16, 1024, 7, 1)])
def test_bcsr_tile_schedule_is_bit_exact_and_balanced(lib, b, N, n_ctas, k_split):
    s = wl.bcsr_sweep(55 + b, m=4096, k=2048, b=b, density=0.1)
    h = lib.spmm_bcsr_create_csr(4096, 2048, s["row_ptr"], s["col_idx"], s["vals"], "fp16", b, host_only=True,
                                 n_ctas=n_ctas, stack_min_fill=-1, k_split=k_split)
    try:
        with pytest.raises(lib.SpmmError):
            lib.spmm_export(h, lib.X_BCSR_TILES, np.int32)          # no plan yet
        lib.spmm_bcsr_plan(h, N)
        info = lib.spmm_get_info(h, N)
        assert info["plan_n"] == N and info["plan_token_tile"] in (128, 256, 512)
        bnt = info["plan_token_tile"]
        n_tt = -(-N // bnt)
        f = F.bcsr_from_csr(4096, 2048, s["row_ptr"], s["col_idx"], s["vals"], b)
        brp = f["block_row_ptr"]
        nbr = brp.shape[0] - 1
        got_ptr = lib.spmm_export(h, lib.X_BCSR_TILE_PTR, np.int32)
        got_tiles = lib.spmm_export(h, lib.X_BCSR_TILES, np.int32).reshape(-1, 2)
        got_units = lib.spmm_export(h, lib.X_BCSR_UNITS, np.int32).reshape(-1, 4)
        units = None if k_split <= 0 else F.bcsr_k_split(brp, n_tt, n_ctas)
        if units is None:
            assert got_units.size == 0 and info["n_slots"] == 0
            want_ptr, want_tiles = F.bcsr_tile_schedule(brp, n_tt, info["plan_slab_tiles"], n_ctas)
            assert np.array_equal(got_ptr, want_ptr) and np.array_equal(got_tiles, want_tiles)
            # every (block-row, token tile) exactly once
            keys = got_tiles[:, 0].astype(np.int64) * n_tt + got_tiles[:, 1]
            assert np.array_equal(np.sort(keys), np.arange(nbr * n_tt))
            cost = np.diff(brp)[got_tiles[:, 0]].astype(np.int64) + 4     # stored blocks + the fixed cost per tile
        else:
            # long block-rows cut into parts: the units, their schedule order and the tiles over them
            assert np.array_equal(got_units, units)
            order = F.bcsr_k_split_order(units)
            ulen = (units[:, 2] - units[:, 1]).astype(np.int64)
            want_ptr, want_tiles = F.bcsr_tile_schedule(None, n_tt, info["plan_slab_tiles"], n_ctas, units=order, lens=ulen[order])
            assert np.array_equal(got_ptr, want_ptr) and np.array_equal(got_tiles, want_tiles)
            assert info["n_slots"] == int((units[:, 3] >= 0).sum()) == units[:, 3].max() + 1
            assert info["n_split"] == np.unique(units[units[:, 3] >= 0, 0]).shape[0] and info["n_tasks"] == units.shape[0]
            assert info["workspace_bytes"] == info["n_slots"] * b * N * 4
            # every (stored block, token tile) exactly once, and every empty block-row's tile as well
            seen = np.zeros((int(brp[-1]), n_tt), dtype=np.int32)
            rows_seen = np.zeros((nbr, n_tt), dtype=np.int32)
            for u, t in got_tiles:
                seen[units[u, 1]:units[u, 2], t] += 1
                rows_seen[units[u, 0], t] += 1
            assert np.all(seen == 1) and np.all(rows_seen >= 1)
            cost = ulen[got_tiles[:, 0]] + 4
            assert cost.max() - 4 <= info["split_cols"]            # no tile longer than the cap
        # greedy longest-first bound: no CTA exceeds the lightest by more than the heaviest tile
        loads = np.array([cost[got_ptr[c]:got_ptr[c + 1]].sum() for c in range(n_ctas)])
        assert loads.max() - loads.min() <= cost.max()
        if N % 512 == 0 and b != 128 and nbr * (N // 512) >= 8 * n_ctas:
            assert bnt == 512                                        # widest tile that divides N
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("b,N,n_ctas,fill", [(16, 4096, 148, 0), (32, 1000, 13, 0), (64, 8192, 8, 0), (16, 512, 5, 1),
                                             (32, 4096, 148, 100), (64, 256, 148, 0), (128, 512, 4, 0)])
def test_bcsr_row_groups_and_their_schedules_are_bit_exact(lib, b, N, n_ctas, fill):
    """Row groups (128 / b block-rows computed from 128-row stacked blocks): the grouping, and the two
    tile schedules of a handle that has groups, against the definitions in oracle/formats.py."""
    m, k = 4096, 2048
    s = wl.bcsr_sweep(91 + b, m=m, k=k, b=b, density=0.3)            # 10 % full block-rows, 20 % empty, rest 0.3
    h = lib.spmm_bcsr_create_csr(m, k, s["row_ptr"], s["col_idx"], s["vals"], "fp16", b, host_only=True, n_ctas=n_ctas,
                                 stack_min_fill=fill)
    try:
        f = F.bcsr_from_csr(m, k, s["row_ptr"], s["col_idx"], s["vals"], b)
        brp = f["block_row_ptr"]
        info = lib.spmm_get_info(h, N)
        if b == 128:                                                  # blocks already are 128 rows high
            assert info["n_stacked_rows"] == 0 and lib.spmm_export(h, lib.X_BCSR_STACK_ROWS, np.int32).size == 0
            return
        R = 128 // b
        default = {16: 30, 32: 45, 64: 75}[b]
        rows, ptr, cols = F.bcsr_row_groups(brp, f["block_col_idx"], b, fill or default)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_STACK_ROWS, np.int32).reshape(-1, R), rows)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_STACK_PTR, np.int32), ptr)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_STACK_COL_IDX, np.int32), cols)
        assert info["n_stacked_rows"] == rows.size and info["n_stack_blocks"] == cols.size
        assert rows.shape[0] >= (m // b) // (10 * R)                  # the full block-rows are grouped
        # the plan: groups first (tiles of 256 tokens), the other block-rows dealt with the head start
        # the j-th lightest CTA of the first launch leaves to CTA j of the second
        lib.spmm_bcsr_plan(h, N)
        info = lib.spmm_get_info(h, N)
        ng = rows.shape[0]
        n_tt_g = -(-N // 256)
        got_gtiles = lib.spmm_export(h, lib.X_BCSR_STACK_TILES, np.int32).reshape(-1, 2)
        groups_used = b <= 32 or ng * n_tt_g >= n_ctas
        bnt = info["plan_token_tile"]
        n_tt = -(-N // bnt)
        got_ptr = lib.spmm_export(h, lib.X_BCSR_TILE_PTR, np.int32)
        got_tiles = lib.spmm_export(h, lib.X_BCSR_TILES, np.int32).reshape(-1, 2)
        if not groups_used:
            assert got_gtiles.size == 0
            want_ptr, want_tiles = F.bcsr_tile_schedule(brp, n_tt, info["plan_slab_tiles"], n_ctas)
            assert np.array_equal(got_ptr, want_ptr) and np.array_equal(got_tiles, want_tiles)
            return
        slab_cols = (16 << 20) // (k * 2)
        slab_g = max(1, min(n_tt_g, slab_cols // 256))
        gp, gt, loads = F.bcsr_tile_schedule(None, n_tt_g, slab_g, n_ctas, fixed_cost=8, units=np.arange(ng),
                                             lens=np.diff(ptr), unit_cost=2 * (256 + 128), return_loads=True)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_STACK_TILE_PTR, np.int32), gp)
        assert np.array_equal(got_gtiles, gt)
        order = F.bcsr_row_order(brp)
        rest = order[~np.isin(order, rows.reshape(-1))]
        want_ptr, want_tiles = F.bcsr_tile_schedule(None, n_tt, info["plan_slab_tiles"], n_ctas, units=rest,
                                                    lens=np.diff(brp)[rest], unit_cost=2 * (128 * (bnt // 128) + b),
                                                    initial=np.sort(loads))
        assert np.array_equal(got_ptr, want_ptr) and np.array_equal(got_tiles, want_tiles)
        # together: every (block-row, 128-token group) exactly once
        n128 = -(-N // 128)
        seen = np.zeros((m // b, n128), dtype=np.int32)
        for I, t in got_tiles:
            seen[I, t * (bnt // 128):min(n128, (t + 1) * (bnt // 128))] += 1
        for g, t in got_gtiles:
            for I in rows[g]:
                seen[I, 2 * t:min(n128, 2 * t + 2)] += 1
        assert np.all(seen == 1)
    finally:
        lib.spmm_destroy(h)


WCSR_CASES = [("tf32", 1000, 900, 0.01, 64), ("fp16", 333, 517, 0.05, 32), ("bf16", 160, 4000, 0.2, 128),
              ("fp16", 16, 40, 0.5, 16), ("fp8", 700, 1300, 0.03, 96)]


@pytest.mark.parametrize("wh", [16, 64])
@pytest.mark.parametrize("dtype,m,k,dens,T", WCSR_CASES)
def test_wcsr_format_plan_and_bins_are_bit_exact(lib, dtype, m, k, dens, T, wh):
    a = wl.random_csr(41 + m, m, k, dens, dtype, empty_rows=tuple(range(16, min(32, m))))
    b_col = 32 // wl.elem_size(dtype)
    h = lib.spmm_wcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, wh, split_cols=T,
                                 host_only=True, n_ctas=5)
    try:
        f = F.wcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], wh, b_col)
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32), f["window_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32), f["window_col_idx"])
        got = lib.spmm_export(h, lib.X_WCSR_VALUES, wl.storage_np_dtype(dtype))
        assert np.array_equal(_bits(got), _bits(f["values"]).ravel())
        plan = F.split_plan(f["window_row_ptr"], T)
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_TASKS, np.int32).reshape(-1, 4), plan)
        bin_ptr = lib.spmm_export(h, lib.X_WCSR_BIN_PTR, np.int32)
        bin_tasks = lib.spmm_export(h, lib.X_WCSR_BIN_TASKS, np.int32)
        info = lib.spmm_get_info(h, 128)
        n_bins = info["n_bins"]
        assert n_bins == 5 * (2 if (dtype == "tf32" or wh == 64) else 3)     # one bin per resident CTA
        want_ptr, want_tasks = F.task_bins(plan, n_bins)
        assert np.array_equal(bin_ptr, want_ptr) and np.array_equal(bin_tasks, want_tasks)
        assert sorted(bin_tasks.tolist()) == list(range(plan.shape[0]))      # every task exactly once
        cost = plan[:, 2].astype(np.int64) + 32
        loads = np.array([cost[bin_tasks[bin_ptr[j]:bin_ptr[j + 1]]].sum() for j in range(n_bins)])
        assert loads.max() - loads.min() <= cost.max()                       # LPT balance property
        for j in range(n_bins):
            assert np.all(np.diff(bin_tasks[bin_ptr[j]:bin_ptr[j + 1]]) > 0)
        P = f["window_col_idx"].shape[0]
        assert info["n_units"] == P and info["stored_values"] == wh * P
        assert info["n_tasks"] == plan.shape[0]
        assert info["n_slots"] == int((plan[:, 3] >= 0).sum())
        assert info["n_split"] == np.unique(plan[plan[:, 3] >= 0, 0]).shape[0]
        assert info["n_empty"] == int((np.diff(f["window_row_ptr"]) == 0).sum())
        assert info["distinct_b_rows"] == np.unique(a["col_idx"]).shape[0]
        assert info["workspace_bytes"] == info["n_slots"] * wh * 128 * 4
        assert info["fill_ratio"] == pytest.approx(F.fill_ratio_wcsr(info["nnz"], P, wh))
    finally:
        lib.spmm_destroy(h)


def _split_size_by_plan_and_bins(wptr, n_bins):
    """The default sub-task size recomputed through the (separately pinned) split plan and bins."""
    P = int(wptr[-1])
    cands = [int(min(65536, max(128, ((P // n_bins) >> i) // 64 * 64))) for i in range(4)]
    loads = []
    for T in cands:
        plan = F.split_plan(wptr, T)
        bin_ptr, bin_tasks = F.task_bins(plan, n_bins)
        cost = plan[:, 2].astype(np.int64) + 32
        loads.append(max(int(cost[bin_tasks[bin_ptr[j]:bin_ptr[j + 1]]].sum()) for j in range(n_bins)))
    best = min(loads)
    return next(T for T, l in zip(cands, loads) if l * 100 <= best * 102), cands, loads


def test_default_split_size(lib):
    """No split_cols given: the largest of a bin's share of the columns and its half, quarter and eighth
    whose longest-first assignment ends within 2 % of the best of the four."""
    a = wl.wcsr_irregular(seed=4, m=30000, dtype="fp16")
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, host_only=True, n_ctas=3)
    info = lib.spmm_get_info(h)
    wptr = lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32)
    lib.spmm_destroy(h)
    want, cands, loads = _split_size_by_plan_and_bins(wptr, 9)
    assert info["n_bins"] == 9 and info["split_cols"] == want == F.default_split_cols(wptr, 9)
    assert 128 <= info["split_cols"] <= 65536 and info["split_cols"] % 64 == 0
    # few heavy windows among many light ones: the whole share balances, so nothing smaller is taken
    wp = np.concatenate(([0], np.cumsum([10000] + [64] * 1000)))
    assert F.default_split_cols(wp, 8) == _split_size_by_plan_and_bins(wp, 8)[0] == (74000 // 8) // 64 * 64
    # nine equal heavy windows on eight bins: chunks of a whole share would leave one bin with two of them
    wp = np.concatenate(([0], np.cumsum([4096] * 9)))
    got = F.default_split_cols(wp, 8)
    assert got == _split_size_by_plan_and_bins(wp, 8)[0] and got < 4608
    # clamps
    assert F.default_split_cols(np.array([0, 64, 128]), 8) == 128
    assert F.default_split_cols(np.array([0, 10 ** 8]), 2) == 65536


def test_wcsr_irregular_workload(lib):
    a = wl.wcsr_irregular(seed=3, m=5000, dtype="tf32")
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "tf32", 16, split_cols=256,
                                 host_only=True)
    f = F.wcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], 16, 8)
    assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32), f["window_col_idx"])
    assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_VALUES, np.float32).view(np.uint32),
                          f["values"].ravel().view(np.uint32))
    assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_TASKS, np.int32).reshape(-1, 4),
                          F.split_plan(f["window_row_ptr"], 256))
    lib.spmm_destroy(h)


def test_coo_entry_points_match_csr(lib):
    a = wl.random_csr(5, 200, 300, 0.05, "fp16")
    rows = np.repeat(np.arange(200), np.diff(a["row_ptr"])).astype(np.int32)
    perm = np.random.default_rng(0).permutation(rows.shape[0])
    h1 = lib.spmm_bcsr_create_csr(200, 300, a["row_ptr"], a["col_idx"], a["vals"], "fp16", 32, host_only=True)
    h2 = lib.spmm_bcsr_create_coo(200, 300, rows[perm], a["col_idx"][perm], a["vals"][perm], "fp16", 32, host_only=True)
    for which, dt in ((lib.X_BCSR_BLOCK_ROW_PTR, np.int32), (lib.X_BCSR_BLOCK_COL_IDX, np.int32), (lib.X_BCSR_BLOCKS, np.uint16)):
        assert np.array_equal(lib.spmm_export(h1, which, dt), lib.spmm_export(h2, which, dt))
    lib.spmm_destroy(h1)
    lib.spmm_destroy(h2)
    w1 = lib.spmm_wcsr_create_csr(200, 300, a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, host_only=True)
    w2 = lib.spmm_wcsr_create_coo(200, 300, rows[perm], a["col_idx"][perm], a["vals"][perm], "fp16", 16, host_only=True)
    for which, dt in ((lib.X_WCSR_WINDOW_ROW_PTR, np.int32), (lib.X_WCSR_WINDOW_COL_IDX, np.int32), (lib.X_WCSR_VALUES, np.uint16)):
        assert np.array_equal(lib.spmm_export(w1, which, dt), lib.spmm_export(w2, which, dt))
    lib.spmm_destroy(w1)
    lib.spmm_destroy(w2)


def test_malformed_input_is_rejected(lib):
    rp = np.array([0, 2, 3], np.int64)
    v = np.ones(3, np.float16)

    def code(fn, *args, **kw):
        with pytest.raises(lib.SpmmError) as e:
            fn(*args, **kw)
        return e.value.code

    mk = lib.spmm_bcsr_create_csr
    assert code(mk, 2, 4, rp, np.array([1, 0, 2], np.int32), v, "fp16", 16, host_only=True) == lib.SPMM_ERR_UNSORTED
    assert code(mk, 2, 4, rp, np.array([1, 1, 2], np.int32), v, "fp16", 16, host_only=True) == lib.SPMM_ERR_UNSORTED
    assert code(mk, 2, 4, rp, np.array([0, 4, 2], np.int32), v, "fp16", 16, host_only=True) == lib.SPMM_ERR_OUT_OF_RANGE
    assert code(mk, 2, 4, rp, np.array([-1, 1, 2], np.int32), v, "fp16", 16, host_only=True) == lib.SPMM_ERR_OUT_OF_RANGE
    assert code(mk, 2, 4, np.array([0, 3, 2], np.int64), np.array([0, 1, 2], np.int32), v, "fp16", 16,
                host_only=True) == lib.SPMM_ERR_INVALID_ARG
    assert code(mk, 2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 48, host_only=True) == lib.SPMM_ERR_UNSUPPORTED
    # TF32 BCSR: static schedule only
    assert code(mk, 2, 4, rp, np.array([0, 1, 2], np.int32), np.ones(3, np.float32), "tf32", 16,
                host_only=True, schedule=lib.SCHED_DYNAMIC) == lib.SPMM_ERR_UNSUPPORTED
    mw = lib.spmm_wcsr_create_csr
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 8, host_only=True) == lib.SPMM_ERR_UNSUPPORTED
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 16, split_cols=24,
                host_only=True) == lib.SPMM_ERR_INVALID_ARG
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 16, b_col=8,
                host_only=True) == lib.SPMM_ERR_UNSUPPORTED
    # E4M3 WCSR: fp32 C and the TMA gather only; windows are padded to 32 columns
    v8 = np.full(3, 0x38, np.uint8)
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v8, "fp8", 16, host_only=True,
                c_type=lib.C_SAME_AS_INPUT) == lib.SPMM_ERR_UNSUPPORTED
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v8, "fp8", 16, host_only=True,
                gather=lib.GATHER_LSU) == lib.SPMM_ERR_UNSUPPORTED
    assert code(mw, 2, 4, rp, np.array([0, 1, 2], np.int32), v8, "fp8", 16, host_only=True,
                b_col=16) == lib.SPMM_ERR_UNSUPPORTED
    h8 = mw(2, 4, rp, np.array([0, 1, 2], np.int32), v8, "fp8", 16, host_only=True)
    assert lib.spmm_export(h8, lib.X_WCSR_WINDOW_COL_IDX, np.int32).tolist() == [0, 1, 2] + [-1] * 29
    lib.spmm_destroy(h8)
    # spmm_prepare: spmm_run's rules for N; a host-only WCSR handle has nothing to prepare
    hp = mw(2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 16, host_only=True)
    lib.spmm_prepare(hp, 128)
    assert code(lib.spmm_prepare, hp, 100) == lib.SPMM_ERR_UNSUPPORTED          # rows of 200 bytes
    assert code(lib.spmm_prepare, hp, 0) == lib.SPMM_ERR_INVALID_ARG
    lib.spmm_destroy(hp)
    hp = mk(2, 4, rp, np.array([0, 1, 2], np.int32), v, "fp16", 16, host_only=True)
    lib.spmm_prepare(hp, 128)                                                    # = spmm_bcsr_plan
    assert lib.spmm_get_info(hp, 128)["plan_token_tile"] > 0
    assert code(lib.spmm_prepare, hp, 32) == lib.SPMM_ERR_UNSUPPORTED
    lib.spmm_destroy(hp)
    dup_r, dup_c = np.array([0, 0], np.int32), np.array([1, 1], np.int32)
    assert code(lib.spmm_bcsr_create_coo, 2, 4, dup_r, dup_c, v[:2], "fp16", 16, host_only=True) == lib.SPMM_ERR_UNSORTED
    lib.spmm_destroy(None)                                     # NULL is accepted


def test_empty_matrix(lib):
    rp = np.zeros(33, np.int64)
    h = lib.spmm_wcsr_create_csr(32, 10, rp, np.zeros(0, np.int32), np.zeros(0, np.float32), "tf32", 16, host_only=True)
    info = lib.spmm_get_info(h, 8)
    assert info["n_units"] == 0 and info["n_tasks"] == 0 and info["n_empty"] == 2
    assert lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32).tolist() == [0, 0, 0]
    lib.spmm_destroy(h)
    h = lib.spmm_bcsr_create_csr(32, 10, rp, np.zeros(0, np.int32), np.zeros(0, np.uint16), "bf16", 16, host_only=True)
    assert lib.spmm_get_info(h)["n_units"] == 0
    lib.spmm_destroy(h)


def test_binding_structs_match_the_header(lib, tmp_path):
    """The ctypes mirrors of spmm_opts_t / spmm_info_t have the sizes a C compiler gives the
    header's structs (the header must also compile as plain C)."""
    import ctypes, os, subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include "spmm_b200.h"\n'
                   'int main(void){printf("%zu %zu\\n", sizeof(spmm_opts_t), sizeof(spmm_info_t));return 0;}\n')
    exe = tmp_path / "sizes"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(root, "include"), str(src), "-o", str(exe)], check=True)
    so, si = (int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split())
    assert so == ctypes.sizeof(lib.SpmmOpts) and si == ctypes.sizeof(lib.SpmmInfo)


def test_bcsr_row_major_needs_at_least_64_columns(lib):
    """The documented minimum: a BCSR handle with row-major operands refuses N < 64 (the plan
    call tells without a GPU); N = 64 is planned."""
    a = wl.bcsr_tiny()
    h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64, host_only=True)
    try:
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_bcsr_plan(h, 32)
        assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
        lib.spmm_bcsr_plan(h, 64)
        assert lib.spmm_get_info(h, 64)["plan_n"] == 64
    finally:
        lib.spmm_destroy(h)


def test_wcsr_reuse_classes_of_the_gather_hints(lib):
    """Device-private hint, checked against its rule written out with numpy: B rows ranked by the
    number of windows that gather them (ties: lower index), class 7 for the first 16 Ki, one class
    down per doubling, 0 beyond 1 Mi and for rows gathered once; a group of four padded columns
    takes the highest class among its columns."""
    a = wl.rmat(seed=5, scale=16, edge_factor=12)                     # 65,536 columns, skewed popularity
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, host_only=True)
    try:
        got = lib.spmm_export(h, lib.X_WCSR_GROUP_CLASS, np.uint8)
        wcol = lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32)
    finally:
        lib.spmm_destroy(h)
    refs = np.bincount(wcol[wcol >= 0], minlength=a["k"])
    order = np.argsort(-refs, kind="stable")
    rank = np.empty(a["k"], dtype=np.int64)
    rank[order] = np.arange(a["k"])
    level = np.clip(7 - np.floor(np.log2(np.maximum(rank, 1) / 16384.0) + 1).astype(np.int64), 0, 7)
    level = np.where(rank < 16384, 7, level)
    cls = np.where(refs > 1, level, 0)
    per_col = np.where(wcol >= 0, cls[np.maximum(wcol, 0)], 0).reshape(-1, 4)
    assert got.shape[0] == wcol.shape[0] // 4
    assert np.array_equal(got, per_col.max(axis=1).astype(np.uint8))
    assert got.max() == 7 and (got == 6).any() and (got == 0).any()
