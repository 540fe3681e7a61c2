"""GPU parity of the output-type and operand-layout variants: C in the input's 16-bit type
(BCSR and WCSR) and column-major operands (BCSR: X = B^T in, Y = C^T out, the layout of the
paper's BCSR kernel, Sec. 3.2, and of a sparse linear layer, Sec. 4.4).  Same oracle, same
bound as the default path: a 16-bit C adds at most 2^-9 |C| <= 2^-9 sum|a b| of rounding.
"""
import numpy as np
import pytest

from paper_2604_17834_b200 import workloads as wl

from helpers import assert_close, reference, run_gpu, run_gpu_variant, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import binding
    return binding


def _bcsr_variant(lib, a, dtype, b, N, c16, col_major, seed=29):
    Bs = wl.dense(seed, a["k"], N, ("uniform", -1.0, 1.0), dtype)
    h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, b,
                                 c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32,
                                 layout=lib.COLMAJOR if col_major else lib.ROWMAJOR)
    try:
        C = run_gpu_variant(lib, h, Bs, a["m"], N, dtype, c16=c16, col_major=col_major)
        Cr, S = reference(a, Bs, dtype)
        worst = assert_close(C, Cr, S, dtype, "bcsr b=%d N=%d c16=%d cm=%d" % (b, N, c16, col_major))
        C2 = run_gpu_variant(lib, h, Bs, a["m"], N, dtype, c16=c16, col_major=col_major)
        assert np.array_equal(C, C2)
        return worst
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("b", [16, 32, 64, 128])
@pytest.mark.parametrize("c16,col_major", [(True, False), (False, True), (True, True)])
def test_bcsr_variants_block_sizes(lib, dtype, b, c16, col_major):
    a = wl.bcsr_sweep(500 + b, m=1024, k=768, b=b, density=0.2, dtype=dtype)
    _bcsr_variant(lib, a, dtype, b, 640, c16, col_major)      # 640 = 512 + 128: several token tiles


@pytest.mark.parametrize("m,k,b,N", [(504, 304, 64, 200), (136, 72, 32, 136), (1000, 1000, 16, 1030),
                                      (264, 640, 128, 333), (64, 64, 64, 128)])
@pytest.mark.parametrize("c16", [False, True])
def test_bcsr_colmajor_ragged_shapes(lib, m, k, b, N, c16):
    """m, k multiples of 8 only; N arbitrary (not a multiple of 128, 64 or even 8); scattered
    entries, empty block-rows."""
    a = wl.random_csr(17 + m, m, k, 0.02, "bf16", empty_rows=tuple(range(min(b, m // 2))))
    _bcsr_variant(lib, a, "bf16", b, N, c16, True)


def test_bcsr_colmajor_matches_rowmajor_bitwise(lib):
    """Same products in the same order: the two layouts differ only in how operands are read and
    results written, so fp32 results are identical."""
    a = wl.bcsr_sweep(77, m=512, k=1024, b=64, density=0.3, dtype="fp16")
    Bs = wl.dense(5, 1024, 512, ("normal", 0.0, 1.0), "fp16")
    h0 = lib.spmm_bcsr_create_csr(512, 1024, a["row_ptr"], a["col_idx"], a["vals"], "fp16", 64)
    h1 = lib.spmm_bcsr_create_csr(512, 1024, a["row_ptr"], a["col_idx"], a["vals"], "fp16", 64, layout=lib.COLMAJOR)
    C0 = run_gpu(lib, h0, Bs, 512, 512)
    C1 = run_gpu_variant(lib, h1, Bs, 512, 512, "fp16", col_major=True)
    lib.spmm_destroy(h0)
    lib.spmm_destroy(h1)
    assert np.array_equal(C0, C1)


def test_bcsr_c16_is_the_rounded_fp32_result(lib):
    a = wl.bcsr_tiny()
    Bs = wl.dense(3, 512, 256, ("uniform", -1.0, 1.0), "bf16")
    h0 = lib.spmm_bcsr_create_csr(512, 512, a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64)
    h1 = lib.spmm_bcsr_create_csr(512, 512, a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64, c_type=lib.C_SAME_AS_INPUT)
    C0 = run_gpu(lib, h0, Bs, 512, 256)
    C1 = run_gpu_variant(lib, h1, Bs, 512, 256, "bf16", c16=True)
    lib.spmm_destroy(h0)
    lib.spmm_destroy(h1)
    import torch
    want = torch.from_numpy(C0).to(torch.bfloat16).float().numpy()     # round to nearest even
    assert np.array_equal(C1, want)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("N", [128, 72, 328])
def test_wcsr_c16(lib, dtype, N):
    a = wl.random_csr(53, 1000, 900, 0.02, dtype, empty_rows=tuple(range(32, 64)))
    Bs = wl.dense(19, 900, N, ("normal", 0.0, 1.0), dtype)
    h = lib.spmm_wcsr_create_csr(1000, 900, a["row_ptr"], a["col_idx"], a["vals"], dtype, 16, split_cols=64,
                                 c_type=lib.C_SAME_AS_INPUT)
    try:
        info = lib.spmm_get_info(h, N)
        assert info["n_split"] > 0 and info["n_empty"] >= 2        # direct, merged and zero-filled rows
        assert info["bytes_c"] == 1000 * N * 2
        C = run_gpu_variant(lib, h, Bs, 1000, N, dtype, c16=True)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "wcsr c16 %s N=%d" % (dtype, N))
        assert np.array_equal(C, run_gpu_variant(lib, h, Bs, 1000, N, dtype, c16=True))
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("dtype", ["tf32", "fp16", "bf16", "fp8"])
@pytest.mark.parametrize("N", [128, 80, 336])
def test_wcsr_window_height_64(lib, dtype, N):
    """The paper's own window height (Sec. 4.1): 64-row windows, MMA N = 64.  Format arrays
    bit-exact against the format oracle, result against the SpMM oracle, split + empty windows."""
    from oracle import formats as F
    a = wl.random_csr(57, 1000, 900, 0.02, dtype, empty_rows=tuple(range(64, 192)))
    Bs = wl.dense(19, 900, N, ("normal", 0.0, 1.0), dtype)
    h = lib.spmm_wcsr_create_csr(1000, 900, a["row_ptr"], a["col_idx"], a["vals"], dtype, 64, split_cols=128)
    try:
        b_col = 32 // wl.elem_size(dtype)
        f = F.wcsr_from_csr(1000, 900, a["row_ptr"], a["col_idx"], a["vals"], 64, b_col)
        bits = {4: np.uint32, 2: np.uint16, 1: np.uint8}[wl.elem_size(dtype)]
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32), f["window_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32), f["window_col_idx"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_VALUES, wl.storage_np_dtype(dtype)).view(bits),
                              f["values"].view(bits).ravel())
        info = lib.spmm_get_info(h, N)
        assert info["block"] == 64 and info["n_split"] > 0 and info["n_empty"] >= 2
        assert info["stored_values"] == 64 * f["window_col_idx"].shape[0]
        assert info["workspace_bytes"] == info["n_slots"] * 64 * N * 4
        plan = F.split_plan(f["window_row_ptr"], 128)
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_TASKS, np.int32).reshape(-1, 4), plan)
        C = run_gpu(lib, h, Bs, 1000, N)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "wcsr wh=64 %s N=%d" % (dtype, N))
        assert np.array_equal(C, run_gpu(lib, h, Bs, 1000, N))
    finally:
        lib.spmm_destroy(h)


def test_wcsr_tf32_same_as_input_is_fp32(lib):
    a = wl.wcsr_irregular(seed=6, m=3000, dtype="tf32")
    Bs = wl.dense(2, a["k"], 128, ("normal", 0.0, 1.0), "tf32")
    h0 = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "tf32", 16)
    h1 = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "tf32", 16, c_type=lib.C_SAME_AS_INPUT)
    C0, C1 = run_gpu(lib, h0, Bs, a["m"], 128), run_gpu(lib, h1, Bs, a["m"], 128)
    lib.spmm_destroy(h0)
    lib.spmm_destroy(h1)
    assert np.array_equal(C0, C1)


@pytest.mark.parametrize("b,N", [(16, 1024), (32, 2048), (64, 640), (128, 1032), (64, 4096)])
def test_bcsr_dynamic_schedule_matches_static_bitwise(lib, b, N):
    """Tiles handed out at run time through Cluster Launch Control (more tiles than SMs, so
    running CTAs do take over tiles of CTAs that never start): every tile is computed exactly
    once and exactly as in the static plan, whichever CTA runs it."""
    a = wl.bcsr_sweep(700 + b, m=2048, k=1024, b=b, density=0.15, dtype="fp16")
    Bs = wl.dense(31, a["k"], N, ("uniform", -1.0, 1.0), "fp16")
    args = (a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", b)
    h0 = lib.spmm_bcsr_create_csr(*args)
    h1 = lib.spmm_bcsr_create_csr(*args, schedule=lib.SCHED_DYNAMIC)
    try:
        C0 = run_gpu(lib, h0, Bs, a["m"], N)
        C1 = run_gpu(lib, h1, Bs, a["m"], N)
        assert np.array_equal(C0, C1)
        assert np.array_equal(C1, run_gpu(lib, h1, Bs, a["m"], N))
        Cr, S = reference(a, Bs, "fp16")
        assert_close(C1, Cr, S, "fp16", "bcsr dynamic b=%d N=%d" % (b, N))
        # the dynamic plan is one list: every (block-row, token tile) once, slab by slab, longest first
        tp = lib.spmm_export(h1, lib.X_BCSR_TILE_PTR, np.int32)
        tiles = lib.spmm_export(h1, lib.X_BCSR_TILES, np.int32).reshape(-1, 2)
        info = lib.spmm_get_info(h1, N)
        n_tt = -(-N // info["plan_token_tile"])
        assert tp.tolist() == [0, tiles.shape[0]] and tiles.shape[0] == (2048 // b) * n_tt
        from oracle import formats as F
        f = F.bcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], b)
        want_ptr, want_tiles = F.bcsr_tile_schedule(f["block_row_ptr"], n_tt, info["plan_slab_tiles"], 1)
        assert np.array_equal(tiles, want_tiles)
    finally:
        lib.spmm_destroy(h0)
        lib.spmm_destroy(h1)


@pytest.mark.parametrize("b", [32, 64, 128])
@pytest.mark.parametrize("N", [640, 333, 128])
def test_bcsr_fp8_e4m3_colmajor(lib, b, N):
    """8-bit E4M3 inputs (the next step Sec. 5 names), K-major operands: X [N][k] and the stored
    blocks as E4M3, fp32 accumulation and output.  Products of two E4M3 values are exact in
    fp32, so the 16-bit bound applies unchanged."""
    a = wl.bcsr_sweep(900 + b, m=1024, k=768, b=b, density=0.2, dtype="fp8")
    Bs = wl.dense(37, a["k"], N, ("uniform", -1.0, 1.0), "fp8")
    h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp8", b, layout=lib.COLMAJOR)
    try:
        from oracle import formats as F
        f = F.bcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], b)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"])
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCKS, np.uint8), f["blocks"].ravel())
        C = run_gpu_variant(lib, h, Bs, a["m"], N, "fp8", col_major=True)
        Cr, S = reference(a, Bs, "fp8")
        assert_close(C, Cr, S, "fp8", "bcsr fp8 b=%d N=%d" % (b, N))
        assert np.array_equal(C, run_gpu_variant(lib, h, Bs, a["m"], N, "fp8", col_major=True))
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("dtype,b,m,k", [("fp16", 64, 1024, 768), ("bf16", 16, 1000, 1000), ("fp16", 32, 130, 70),
                                          ("bf16", 128, 257, 640), ("fp16", 16, 4096, 70000)])
def test_bcsr_built_on_the_gpu_is_bit_exact(lib, dtype, b, m, k):
    """Format construction as GPU kernels from a CSR matrix in device memory: every exported
    array equals the format oracle's, and the handle runs like a host-built one."""
    import torch
    from oracle import formats as F
    a = wl.random_csr(23 + m, m, k, 0.02 if k < 5000 else 0.0005, dtype, empty_rows=tuple(range(min(b, m // 2))))
    rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
    ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
    va = to_device(a["vals"])
    h = lib.spmm_bcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, b)
    try:
        f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_ROW_PTR, np.int32), f["block_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"])
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCKS, np.uint16), f["blocks"].view(np.uint16).ravel())
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_ROW_ORDER, np.int32), F.bcsr_row_order(f["block_row_ptr"]))
        info = lib.spmm_get_info(h, 128)
        assert info["nnz"] == a["col_idx"].shape[0] and info["n_units"] == f["block_col_idx"].shape[0]
        assert info["n_empty"] == int((np.diff(f["block_row_ptr"]) == 0).sum())
        N = 200
        Bs = wl.dense(3, k, N, ("uniform", -1.0, 1.0), dtype)
        C = run_gpu(lib, h, Bs, m, N)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "bcsr built on the GPU b=%d" % b)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("dtype,wh,m,k,dens", [("tf32", 16, 1000, 900, 0.02), ("fp16", 16, 333, 517, 0.05),
                                                ("bf16", 64, 1000, 4000, 0.01), ("fp16", 16, 5000, 70000, 0.0005),
                                                ("tf32", 64, 130, 70, 0.2), ("fp8", 16, 1000, 900, 0.02),
                                                ("fp8", 64, 400, 2000, 0.01)])
def test_wcsr_built_on_the_gpu_is_bit_exact(lib, dtype, wh, m, k, dens):
    """Window condensation and value packing as GPU kernels (sort / unique of (window, column)
    keys): every exported array equals the format oracle's, plan and bins included, and the
    handle runs like a host-built one."""
    import torch
    from oracle import formats as F
    a = wl.random_csr(29 + m, m, k, dens, dtype, empty_rows=tuple(range(wh, min(3 * wh, m))))
    rp = torch.from_numpy(a["row_ptr"].astype(np.int64)).cuda()
    ci = torch.from_numpy(a["col_idx"].astype(np.int32)).cuda()
    va = to_device(a["vals"])
    h = lib.spmm_wcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), va.data_ptr(), dtype, wh, split_cols=64)
    h0 = lib.spmm_wcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, wh, split_cols=64)
    try:
        b_col = 32 // wl.elem_size(dtype)
        f = F.wcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], wh, b_col)
        bits = {4: np.uint32, 2: np.uint16, 1: np.uint8}[wl.elem_size(dtype)]
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32), f["window_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32), f["window_col_idx"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_VALUES, wl.storage_np_dtype(dtype)).view(bits),
                              f["values"].view(bits).ravel())
        for which in (lib.X_WCSR_TASKS, lib.X_WCSR_BIN_PTR, lib.X_WCSR_BIN_TASKS):
            assert np.array_equal(lib.spmm_export(h, which, np.int32), lib.spmm_export(h0, which, np.int32))
        # the gather hints (reuse class per four padded columns): same bytes from both builders
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_GROUP_CLASS, np.uint8), lib.spmm_export(h0, lib.X_WCSR_GROUP_CLASS, np.uint8))
        i1, i0 = lib.spmm_get_info(h, 128), lib.spmm_get_info(h0, 128)
        assert i1 == i0
        N = 144
        Bs = wl.dense(3, k, N, ("normal", 0.0, 1.0), dtype)
        C = run_gpu(lib, h, Bs, m, N)
        assert np.array_equal(C, run_gpu(lib, h0, Bs, m, N))
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "wcsr built on the GPU wh=%d" % wh)
    finally:
        lib.spmm_destroy(h)
        lib.spmm_destroy(h0)


def test_bcsr_gpu_builder_rejects_malformed_csr(lib):
    import torch
    vals = to_device(wl.to_storage(np.ones(4), "fp16"))
    cases = [(np.array([0, 2, 4]), np.array([1, 0, 2, 3]), lib.SPMM_ERR_UNSORTED),         # descending columns
             (np.array([0, 2, 4]), np.array([0, 0, 2, 3]), lib.SPMM_ERR_UNSORTED),         # duplicate
             (np.array([0, 2, 4]), np.array([0, 1, 2, 9]), lib.SPMM_ERR_OUT_OF_RANGE),     # column >= k
             (np.array([0, 3, 2]), np.array([0, 1, 2, 3]), lib.SPMM_ERR_INVALID_ARG),      # row_ptr not monotone
             (np.array([1, 2, 4]), np.array([0, 1, 2, 3]), lib.SPMM_ERR_INVALID_ARG)]      # row_ptr[0] != 0
    for rp, ci, code in cases:
        rpd = torch.from_numpy(rp.astype(np.int64)).cuda()
        cid = torch.from_numpy(ci.astype(np.int32)).cuda()
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_bcsr_create_csr_device(2, 8, rpd.data_ptr(), cid.data_ptr(), vals.data_ptr(), "fp16", 16)
        assert e.value.code == code
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_wcsr_create_csr_device(2, 8, rpd.data_ptr(), cid.data_ptr(), vals.data_ptr(), "fp16", 16)
        assert e.value.code == code


def test_variant_argument_errors(lib):
    a = wl.bcsr_tiny()
    args = (512, 512, a["row_ptr"], a["col_idx"], a["vals"], "bf16")
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_wcsr_create_csr(*args, 16, layout=lib.COLMAJOR)            # BCSR only
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_bcsr_create_csr(*args, 64, c_type=7)
    assert e.value.code == lib.SPMM_ERR_INVALID_ARG
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_bcsr_create_csr(*args, 64, schedule=lib.SCHED_DYNAMIC, c_type=lib.C_SAME_AS_INPUT)   # fp32 row-major only
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_wcsr_create_csr(*args, 16, schedule=lib.SCHED_DYNAMIC)
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    a8 = wl.bcsr_sweep(5, m=256, k=256, b=32, density=0.3, dtype="fp8")
    for kw in (dict(c_type=lib.C_SAME_AS_INPUT), dict(layout=lib.COLMAJOR, c_type=lib.C_SAME_AS_INPUT),
               dict(schedule=lib.SCHED_DYNAMIC)):                                  # E4M3: fp32 C, static schedule only
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_bcsr_create_csr(256, 256, a8["row_ptr"], a8["col_idx"], a8["vals"], "fp8", 32, **kw)
        assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_bcsr_create_csr(256, 256, a8["row_ptr"], a8["col_idx"], a8["vals"], "fp8", 16, layout=lib.COLMAJOR)
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    b = wl.random_csr(3, 100, 64, 0.1, "bf16")                             # m = 100: not a multiple of 8
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_bcsr_create_csr(100, 64, b["row_ptr"], b["col_idx"], b["vals"], "bf16", 32, layout=lib.COLMAJOR)
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    import torch
    h = lib.spmm_bcsr_create_csr(*args, 64, layout=lib.COLMAJOR)
    buf = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_run(h, buf.data_ptr(), buf.data_ptr(), 64)                 # fewer than 128 tokens
    assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    lib.spmm_destroy(h)


# --------------------------------------------------------------------------- row groups (stacked 128-row blocks)


def _grouped_matrix(seed, m, k, b, dtype):
    """Block pattern with what the grouping looks for: a band of dense block-rows, block-rows
    that share most of their columns, sparse ones and empty ones, in scattered positions."""
    rng = np.random.default_rng(seed)
    nbr, nbc = -(-m // b), -(-k // b)
    kind = rng.choice(4, size=nbr, p=[0.3, 0.3, 0.25, 0.15])
    shared = rng.random(nbc) < 0.5
    mask = np.zeros((nbr, nbc), dtype=bool)
    for i in range(nbr):
        if kind[i] == 0:
            mask[i] = True
        elif kind[i] == 1:
            mask[i] = shared & (rng.random(nbc) < 0.9)
        elif kind[i] == 2:
            mask[i] = rng.random(nbc) < 0.08
    D = np.zeros((nbr * b, nbc * b), dtype=np.float32)
    for i, j in zip(*np.nonzero(mask)):
        blk = rng.uniform(-1.0, 1.0, size=(b, b)).astype(np.float32)
        blk[rng.random((b, b)) < 0.3] = 0.0                           # blocks are not full either
        D[i * b:(i + 1) * b, j * b:(j + 1) * b] = blk
    D = D[:m, :k]
    rows, cols = np.nonzero(D)
    row_ptr = np.concatenate(([0], np.cumsum(np.bincount(rows, minlength=m)))).astype(np.int64)
    return dict(m=m, k=k, row_ptr=row_ptr, col_idx=cols.astype(np.int32), vals=wl.to_storage(D[rows, cols], dtype))


@pytest.mark.parametrize("b,dtype,m,k,N,c16,cm,fill", [
    (16, "fp16", 1024, 640, 384, False, False, 0),
    (16, "bf16", 1000, 520, 328, True, False, 0),        # ragged m, k and N
    (32, "fp16", 1024, 768, 256, False, True, 0),
    (32, "bf16", 1096, 512, 200, True, True, 0),         # N below one 256-token tile, Y rows of 1096 elements
    (64, "fp16", 2048, 512, 1184, False, False, 0),      # (b = 64 groups are used when they make a tile per CTA: 24 CTAs)
    (64, "bf16", 2048, 512, 1184, True, True, 0),
    (16, "fp16", 512, 512, 128, False, False, 1),        # forced: groups of sparse rows, mostly absent sub-blocks
    (32, "fp16", 640, 384, 512, False, False, 1),
    (64, "fp16", 4096, 256, 608, False, False, 1),
    (32, "fp8", 1024, 768, 328, False, True, 0),         # E4M3: column-major operands, fp32 Y
    (64, "fp8", 2048, 512, 1184, False, True, 0),
    (32, "fp8", 640, 384, 512, False, True, 1),
])
def test_bcsr_row_groups_match_the_oracle(lib, b, dtype, m, k, N, c16, cm, fill):
    from oracle import formats as F
    a = _grouped_matrix(7 * b + N, m, k, b, dtype)
    Bs = wl.dense(300 + b, k, N, ("uniform", -1.0, 1.0), dtype)
    Cr, S = reference(a, Bs, dtype)
    outs = {}
    for mode in (fill, -1):
        h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b,
                                     c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32,
                                     layout=lib.COLMAJOR if cm else lib.ROWMAJOR, stack_min_fill=mode,
                                     n_ctas=24 if b == 64 else 0)
        try:
            info = lib.spmm_get_info(h, N)
            if mode >= 0:
                assert info["n_stacked_rows"] >= 128 // b, "the test matrix must produce row groups"
            else:
                assert info["n_stacked_rows"] == 0
            got = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16, col_major=cm)
            assert_close(got, Cr, S, dtype, "b=%d %s groups %s" % (b, dtype, "on" if mode >= 0 else "off"))
            if mode >= 0:
                used = lib.spmm_export(h, lib.X_BCSR_STACK_TILES, np.int32).size > 0
                assert used, "the plan must use the row groups in this case"
                # the exported format stays the canonical one
                f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
                assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"])
                again = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16, col_major=cm)
                assert np.array_equal(got, again), "run-to-run difference"
            outs[mode] = got
        finally:
            lib.spmm_destroy(h)
    # absent sub-blocks add exact zeros: the grouped and the plain launch agree to the last bit
    assert np.array_equal(outs[fill], outs[-1])


def test_bcsr_row_groups_from_the_gpu_builder(lib):
    """Same handle from a device-resident CSR: the stacked values are built from the blocks the GPU builder wrote."""
    import torch
    b, dtype, m, k, N = 16, "fp16", 768, 512, 256
    a = _grouped_matrix(5, m, k, b, dtype)
    Bs = wl.dense(77, k, N, ("uniform", -1.0, 1.0), dtype)
    Cr, S = reference(a, Bs, dtype)
    rp, ci, v = to_device(a["row_ptr"]), to_device(a["col_idx"]), to_device(a["vals"])
    h = lib.spmm_bcsr_create_csr_device(m, k, rp.data_ptr(), ci.data_ptr(), v.data_ptr(), dtype, b,
                                        stream=torch.cuda.current_stream().cuda_stream)
    try:
        assert lib.spmm_get_info(h, N)["n_stacked_rows"] > 0
        got = run_gpu_variant(lib, h, Bs, m, N, dtype)
        assert_close(got, Cr, S, dtype, "gpu-built, row groups")
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("b,dtype", [(16, "fp16"), (32, "bf16")])
def test_bcsr_row_groups_find_scattered_families(lib, b, dtype):
    """Block-rows of one family are far apart in the index range and in the length order: the
    groups must still be (mostly) families, i.e. far fewer stacked blocks than R neighbours' union
    would need, and the product must match the oracle."""
    from oracle import formats as F
    m, k, N = 2048, 2048, 384
    a = wl.bcsr_families(55 + b, m=m, k=k, b=b, density=0.15, n_families=8, drop=0.1, dtype=dtype)
    Bs = wl.dense(56 + b, k, N, ("uniform", -1.0, 1.0), dtype)
    Cr, S = reference(a, Bs, dtype)
    f = F.bcsr_from_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], b)
    rows, ptr, cols = F.bcsr_row_groups(f["block_row_ptr"], f["block_col_idx"], b, {16: 30, 32: 45}[b])
    R = 128 // b
    stored = np.diff(f["block_row_ptr"].astype(np.int64))[rows].sum()
    assert rows.shape[0] >= (m // b) // R * 3 // 4, "most block-rows must end up in a group"
    # (a group of one family is ~90 % full; the leftovers of every family mix; unrelated rows at this
    # density would give ~20 %)
    assert stored >= 0.65 * R * cols.size, "groups must be made of rows of one family"
    h = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b)
    try:
        info = lib.spmm_get_info(h, N)
        assert info["n_stacked_rows"] == rows.size and info["n_stack_blocks"] == cols.size
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_STACK_ROWS, np.int32).reshape(-1, R), rows)
        got = run_gpu_variant(lib, h, Bs, m, N, dtype)
        assert_close(got, Cr, S, dtype, "families b=%d" % b)
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("kind", ["bcsr", "bcsr_ksplit", "wcsr"])
def test_prepare_leaves_nothing_to_allocate_for_the_run(lib, kind):
    """After spmm_prepare(h, N) the first spmm_run at that width changes neither the free device
    memory nor the workspace the handle reports (one throw-away handle of the same kind runs first,
    so that the kernel variant's code is already loaded)."""
    import torch
    dtype, N = "fp16", 512
    st = torch.cuda.current_stream().cuda_stream

    def make():
        if kind == "wcsr":
            a = wl.wcsr_irregular(seed=91, m=6000, dtype=dtype)
            return a, lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 16, split_cols=64)
        a = wl.bcsr_sweep(93, m=2048, k=2048, b=64, density=0.05, dtype=dtype)
        return a, lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 64,
                                           k_split=1 if kind == "bcsr_ksplit" else 0)

    a, h0 = make()
    Bs = wl.dense(94, a["k"], N, ("normal", 0.0, 1.0), dtype)
    Bd = to_device(Bs)
    C = torch.empty((a["m"], N), dtype=torch.float32, device="cuda")
    lib.spmm_run(h0, Bd.data_ptr(), C.data_ptr(), N, st)                 # loads the kernels
    torch.cuda.synchronize()
    want = C.cpu().numpy().copy()
    lib.spmm_destroy(h0)
    _, h = make()
    try:
        lib.spmm_prepare(h, N)
        info = lib.spmm_get_info(h, N)
        if kind != "bcsr":
            assert info["workspace_bytes"] > 0, "the case must need a workspace"
        C.fill_(float("nan"))
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        lib.spmm_run(h, Bd.data_ptr(), C.data_ptr(), N, st)
        free1 = torch.cuda.mem_get_info()[0]
        torch.cuda.synchronize()
        lib.spmm_check(h)
        assert free1 == free0
        assert lib.spmm_get_info(h, N)["workspace_bytes"] == info["workspace_bytes"]
        assert np.array_equal(C.cpu().numpy(), want)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C.cpu().numpy(), Cr, S, dtype, "prepared run, " + kind)
    finally:
        lib.spmm_destroy(h)


# --------------------------------------------------------------------------- the paper's own gather (load/store units)


@pytest.mark.parametrize("dtype,m,k,N,T", [("tf32", 3000, 2500, 128, 0), ("tf32", 1000, 900, 328, 64), ("fp16", 4000, 3000, 256, 0),
                                           ("bf16", 777, 1300, 72, 32), ("fp16", 2048, 2048, 1000, 128)])
def test_wcsr_lsu_gather_matches_the_oracle_and_the_tma_gather(lib, dtype, m, k, N, T):
    """opts.gather = GATHER_LSU: B rows copied by the producer warps with 16-byte cp.async (the
    cooperative 128-bit gather of Sec. 3.2) to the swizzled positions the MMA reads.  Same MMAs in the
    same order as the default TMA gather, so the two results agree to the last bit."""
    a = wl.wcsr_irregular(seed=500 + N, m=m, k=k, dtype=dtype, max_len=700)
    Bs = wl.dense(501, k, N, ("normal", 0.0, 1.0), dtype)
    Cr, S = reference(a, Bs, dtype)
    outs = []
    for gather in (lib.GATHER_LSU, lib.GATHER_TMA):
        h = lib.spmm_wcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, 16, split_cols=T, gather=gather)
        try:
            info = lib.spmm_get_info(h, N)
            if T:
                assert info["n_split"] > 0, "the case must exercise split windows"
            C = run_gpu(lib, h, Bs, m, N)
            assert_close(C, Cr, S, dtype, "wcsr %s gather=%d" % (dtype, gather))
            assert np.array_equal(C, run_gpu(lib, h, Bs, m, N))
            outs.append(C)
        finally:
            lib.spmm_destroy(h)
    assert np.array_equal(outs[0], outs[1])


def test_wcsr_lsu_gather_argument_errors(lib):
    a = wl.wcsr_irregular(seed=9, m=256, k=256, dtype="fp16")
    for kw, wh in ((dict(gather=lib.GATHER_LSU), 64), (dict(gather=lib.GATHER_LSU, c_type=lib.C_SAME_AS_INPUT), 16)):
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_wcsr_create_csr(256, 256, a["row_ptr"], a["col_idx"], a["vals"], "fp16", wh, **kw)
        assert e.value.code == lib.SPMM_ERR_UNSUPPORTED
    with pytest.raises(lib.SpmmError) as e:
        lib.spmm_wcsr_create_csr(256, 256, a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, gather=7)
    assert e.value.code == lib.SPMM_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype,b,m,k,N", [("fp16", 64, 2048, 4096, 1024), ("bf16", 128, 1000, 4096, 1000),
                                           ("tf32", 64, 1536, 2048, 520), ("fp16", 32, 2048, 2048, 768)])
def test_bcsr_k_split_of_long_block_rows(lib, dtype, b, m, k, N):
    """A few full block-rows among short ones: the plan cuts them into parts whose partial tiles a
    second kernel adds in order.  Same oracle bound as the uncut plan, run-to-run identical bits, and
    (parts only regroup the fp32 sum) agreement with the uncut result to fp32 rounding."""
    a = wl.bcsr_sweep(700 + b, m=m, k=k, b=b, density=0.05, dtype=dtype)
    Bs = wl.dense(41, k, N, ("normal", 0.0, 1.0), dtype)
    h1 = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b, stack_min_fill=-1, k_split=1)
    h0 = lib.spmm_bcsr_create_csr(m, k, a["row_ptr"], a["col_idx"], a["vals"], dtype, b, stack_min_fill=-1)
    try:
        C1 = run_gpu(lib, h1, Bs, m, N)
        info = lib.spmm_get_info(h1, N)
        assert info["n_slots"] > 0 and info["n_split"] > 0 and info["workspace_bytes"] == info["n_slots"] * b * N * 4
        units = lib.spmm_export(h1, lib.X_BCSR_UNITS, np.int32).reshape(-1, 4)
        assert (units[:, 2] - units[:, 1]).max() <= info["split_cols"]
        C0 = run_gpu(lib, h0, Bs, m, N)
        assert lib.spmm_get_info(h0, N)["n_slots"] == 0
        Cr, S = reference(a, Bs, dtype)
        assert_close(C1, Cr, S, dtype, "bcsr with K-split %s b=%d" % (dtype, b))
        assert_close(C0, Cr, S, dtype, "bcsr without K-split %s b=%d" % (dtype, b))
        assert np.array_equal(C1, run_gpu(lib, h1, Bs, m, N))            # fixed summation order
        assert np.max(np.abs(C1 - C0)) <= 1e-4 * max(1.0, float(S.max()))
    finally:
        lib.spmm_destroy(h0)
        lib.spmm_destroy(h1)


@pytest.mark.parametrize("b,N", [(32, 640), (64, 1024), (128, 400), (64, 128)])
def test_bcsr_fp8_e4m3_rowmajor(lib, b, N):
    """E4M3 inputs with the default row-major operands (B [k][N] as the token-major tensor-core
    operand of 1-byte elements): oracle bound, and the same bits as the column-major path (same
    products, same order)."""
    a = wl.bcsr_sweep(950 + b, m=1024, k=768, b=b, density=0.2, dtype="fp8")
    Bs = wl.dense(43, a["k"], N, ("uniform", -1.0, 1.0), "fp8")
    h0 = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp8", b)
    h1 = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp8", b, layout=lib.COLMAJOR,
                                  stack_min_fill=-1)
    try:
        C0 = run_gpu_variant(lib, h0, Bs, a["m"], N, "fp8")
        Cr, S = reference(a, Bs, "fp8")
        assert_close(C0, Cr, S, "fp8", "bcsr fp8 row-major b=%d N=%d" % (b, N))
        assert np.array_equal(C0, run_gpu_variant(lib, h0, Bs, a["m"], N, "fp8"))
        C1 = run_gpu_variant(lib, h1, Bs, a["m"], N, "fp8", col_major=True)
        assert np.array_equal(C0, C1)
    finally:
        lib.spmm_destroy(h0)
        lib.spmm_destroy(h1)
