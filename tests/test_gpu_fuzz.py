"""Seeded random sweep over shapes, densities, value types, block / window sizes, dense widths
and creation options: every case is checked element by element against the fp64 oracle, and
format arrays built on the GPU against the ones built on the host.  Shapes are ragged on
purpose (m, k, N not multiples of any tile size unless an option demands it).
"""
import numpy as np
import pytest

from paper_2604_17834_b200 import workloads as wl

from helpers import assert_close, reference, run_gpu_variant, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import binding
    return binding


def _round_up(x, q):
    return -(-x // q) * q


@pytest.mark.parametrize("seed", range(60))
def test_bcsr_random_case(lib, seed):
    import torch
    rng = np.random.default_rng(7000 + seed)
    dtype = ["bf16", "fp16", "fp8"][int(rng.integers(0, 3))]
    b = int([16, 32, 64, 128][int(rng.integers(0, 4))])
    col_major = bool(rng.integers(0, 2)) or dtype == "fp8"
    c16 = bool(rng.integers(0, 2)) and dtype != "fp8"
    dyn = bool(rng.integers(0, 3) == 0) and not (col_major or c16)
    on_gpu = bool(rng.integers(0, 2))
    if dtype == "fp8" and b == 16:
        b = 32
    m, k = int(rng.integers(1, 1500)), int(rng.integers(1, 1500))
    if col_major:
        m, k = _round_up(m, 8), _round_up(k, 16 if dtype == "fp8" else 8)
    es = wl.elem_size(dtype)
    N = int(rng.integers(128 if col_major else 64, 1400))
    if not col_major:
        N = _round_up(N, 16 // es)
    dens = float(10.0 ** rng.uniform(-3.0, -0.7))
    a = wl.random_csr(int(rng.integers(0, 1 << 30)), m, k, dens, dtype, empty_rows=tuple(range(min(b, m // 3))))
    Bs = wl.dense(int(rng.integers(0, 1 << 30)), k, N, ("uniform", -1.0, 1.0), dtype)
    opt = dict(c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32, layout=lib.COLMAJOR if col_major else lib.ROWMAJOR,
               schedule=lib.SCHED_DYNAMIC if dyn else lib.SCHED_STATIC)
    what = "seed %d: %s b=%d m=%d k=%d N=%d dens=%.4f cm=%d c16=%d dyn=%d gpu-built=%d" % (seed, dtype, b, m, k, N, dens, col_major, c16, dyn, on_gpu)
    if on_gpu:
        rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
        ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
        va = to_device(a["vals"])
        h = lib.spmm_bcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, b, **opt)
    else:
        h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b, **opt)
    try:
        C = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16, col_major=col_major)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, what)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("seed", range(24))
def test_bcsr_tf32_random_case(lib, seed):
    """fp32 storage / TF32 arithmetic: block sizes, both operand layouts, both builders, ragged shapes."""
    import torch
    rng = np.random.default_rng(13000 + seed)
    b = int([16, 32, 64, 128][seed % 4])
    col_major = bool(rng.integers(0, 2))
    on_gpu = bool(rng.integers(0, 2))
    m, k = int(rng.integers(1, 1500)), int(rng.integers(1, 1500))
    if col_major:
        m, k = _round_up(m, 8), _round_up(k, 4)
    N = int(rng.integers(128 if col_major else 64, 1400))
    if not col_major:
        N = _round_up(N, 4)
    dens = float(10.0 ** rng.uniform(-3.0, -0.7))
    a = wl.random_csr(int(rng.integers(0, 1 << 30)), m, k, dens, "tf32", empty_rows=tuple(range(min(b, m // 3))))
    Bs = wl.dense(int(rng.integers(0, 1 << 30)), k, N, ("normal", 0.0, 1.0), "tf32")
    opt = dict(layout=lib.COLMAJOR if col_major else lib.ROWMAJOR)
    what = "seed %d: tf32 b=%d m=%d k=%d N=%d dens=%.4f cm=%d gpu-built=%d" % (seed, b, m, k, N, dens, col_major, on_gpu)
    if on_gpu:
        rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
        ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
        va = to_device(a["vals"])
        h = lib.spmm_bcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), "tf32", b, **opt)
    else:
        h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], "tf32", b, **opt)
    try:
        if on_gpu:
            from oracle import formats as F
            f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
            assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"]), what
            assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCKS, np.uint32), f["blocks"].view(np.uint32).ravel()), what
        C = run_gpu_variant(lib, h, Bs, m, N, "tf32", col_major=col_major)
        Cr, S = reference(a, Bs, "tf32")
        assert_close(C, Cr, S, "tf32", what)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("seed", range(40))
def test_bcsr_row_groups_random_case(lib, seed):
    """Row groups forced on (every candidate of 128 / b block-rows that share columns is stacked, however
    few of its sub-blocks are stored) or left to the default threshold, over ragged shapes and all output options."""
    import torch
    rng = np.random.default_rng(11000 + seed)
    dtype = ["bf16", "fp16", "fp8"][seed % 3]
    b = int([16, 32, 64][int(rng.integers(0, 3))])
    col_major = bool(rng.integers(0, 2)) or dtype == "fp8"
    c16 = bool(rng.integers(0, 2)) and dtype != "fp8"
    if dtype == "fp8" and b == 16:
        b = 32
    on_gpu = bool(rng.integers(0, 2))
    fill = int([1, 1, 0, 20][int(rng.integers(0, 4))])
    n_ctas = int([0, 0, 5, 37][int(rng.integers(0, 4))])
    m, k = int(rng.integers(130, 2500)), int(rng.integers(1, 1200))
    if col_major:
        m, k = _round_up(m, 8), _round_up(k, 16 if dtype == "fp8" else 8)
    N = int(rng.integers(128 if col_major else 64, 1100))
    if not col_major:
        N = _round_up(N, 8)
    dens = float(10.0 ** rng.uniform(-2.5, -0.3))
    a = wl.random_csr(int(rng.integers(0, 1 << 30)), m, k, dens, dtype, empty_rows=tuple(range(min(b, m // 3))))
    Bs = wl.dense(int(rng.integers(0, 1 << 30)), k, N, ("uniform", -1.0, 1.0), dtype)
    opt = dict(c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32, layout=lib.COLMAJOR if col_major else lib.ROWMAJOR,
               stack_min_fill=fill, n_ctas=n_ctas)
    what = "seed %d: %s b=%d m=%d k=%d N=%d dens=%.4f cm=%d c16=%d fill=%d ctas=%d gpu-built=%d" % (
        seed, dtype, b, m, k, N, dens, col_major, c16, fill, n_ctas, on_gpu)
    if on_gpu:
        rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
        ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
        va = to_device(a["vals"])
        h = lib.spmm_bcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, b, **opt)
    else:
        h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b, **opt)
    try:
        from oracle import formats as F
        f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
        rows, _, cols = F.bcsr_row_groups(f["block_row_ptr"], f["block_col_idx"], b, fill or {16: 30, 32: 45, 64: 75}[b])
        info = lib.spmm_get_info(h, N)
        assert info["n_stacked_rows"] == rows.size and info["n_stack_blocks"] == cols.size, what
        C = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16, col_major=col_major)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, what)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("seed", range(60))
def test_wcsr_random_case(lib, seed):
    import torch
    rng = np.random.default_rng(9000 + seed)
    dtype = ["tf32", "fp16", "bf16"][int(rng.integers(0, 3))]
    wh = int([16, 16, 64][int(rng.integers(0, 3))])
    c16 = bool(rng.integers(0, 2))
    if seed % 5 == 4:                      # every fifth case: E4M3 values, fp32 C
        dtype, c16 = "fp8", False
    on_gpu = bool(rng.integers(0, 2))
    m, k = int(rng.integers(1, 3000)), int(rng.integers(1, 3000))
    es = wl.elem_size(dtype)
    N = _round_up(int(rng.integers(1, 700)), 16 // es)
    b_col = 32 // es
    T = int(rng.integers(0, 3)) * b_col * int(rng.integers(1, 20))           # 0 = library default
    dens = float(10.0 ** rng.uniform(-3.0, -1.0))
    a = wl.random_csr(int(rng.integers(0, 1 << 30)), m, k, dens, dtype, empty_rows=tuple(range(min(wh, m // 3))))
    Bs = wl.dense(int(rng.integers(0, 1 << 30)), k, N, ("normal", 0.0, 1.0), dtype)
    opt = dict(c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32, split_cols=T)
    what = "seed %d: %s wh=%d m=%d k=%d N=%d dens=%.4f T=%d c16=%d gpu-built=%d" % (seed, dtype, wh, m, k, N, dens, T, c16, on_gpu)
    if on_gpu:
        rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
        ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
        va = to_device(a["vals"])
        h = lib.spmm_wcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, wh, **opt)
    else:
        h = lib.spmm_wcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, wh, **opt)
    try:
        C = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16 and dtype != "tf32")
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, what)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("kind", ["bcsr", "wcsr"])
@pytest.mark.parametrize("on_gpu", [False, True])
@pytest.mark.parametrize("m,k,nnz_rows", [(1, 1, (0,)), (1, 1, ()), (8, 16, ()), (3, 200, (2,)), (200, 3, (0, 199))])
def test_degenerate_shapes(lib, kind, on_gpu, m, k, nnz_rows):
    """One-element, empty and sliver matrices, host- and GPU-built: all of C is written."""
    import torch
    dtype = "fp16"
    dense = np.zeros((m, k), np.float32)
    for r in nnz_rows:
        dense[r, :: max(1, k // 3)] = 1.5
    rows, cols = np.nonzero(dense)
    row_ptr = np.zeros(m + 1, np.int64)
    np.add.at(row_ptr, rows + 1, 1)
    row_ptr = np.cumsum(row_ptr)
    a = dict(m=m, k=k, row_ptr=row_ptr, col_idx=cols.astype(np.int32), vals=wl.to_storage(dense[rows, cols], dtype))
    N = 136
    Bs = wl.dense(4, k, N, ("uniform", -1.0, 1.0), dtype)
    size = 32 if kind == "bcsr" else 16
    if on_gpu:
        rp, ci = torch.from_numpy(a["row_ptr"]).cuda(), torch.from_numpy(a["col_idx"]).cuda()
        va = to_device(a["vals"]) if a["vals"].shape[0] else torch.zeros(8, dtype=torch.int16, device="cuda")
        mk = lib.spmm_bcsr_create_csr_device if kind == "bcsr" else lib.spmm_wcsr_create_csr_device
        h = mk(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, size)
    else:
        mk = lib.spmm_bcsr_create_csr if kind == "bcsr" else lib.spmm_wcsr_create_csr
        h = mk(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, size)
    try:
        C = run_gpu_variant(lib, h, Bs, m, N, dtype)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "%s %dx%d gpu-built=%d" % (kind, m, k, on_gpu))
    finally:
        lib.spmm_destroy(h)
