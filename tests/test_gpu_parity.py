"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle,
element by element on the same seeded inputs.  Sizes span several tiles, ragged
tails, empty block-rows / windows, split windows, and every supported block size
and dtype.  Format arrays exported from the device copy are compared bit for bit.
"""
import numpy as np
import pytest

from oracle import formats as F
from paper_2604_17834_b200 import workloads as wl

from helpers import assert_close, reference, run_gpu, run_gpu_variant

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import binding
    return binding


def _bcsr_case(lib, a, dtype, b, N, Bdist=("uniform", -1.0, 1.0), seed=9):
    Bs = wl.dense(seed, a["k"], N, Bdist, dtype)
    h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, b)
    try:
        f = F.bcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], b)
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_ROW_PTR, np.int32), f["block_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCK_COL_IDX, np.int32), f["block_col_idx"])
        bits = np.uint32 if dtype == "tf32" else np.uint16
        assert np.array_equal(lib.spmm_export(h, lib.X_BCSR_BLOCKS, bits), f["blocks"].view(bits).ravel())
        C = run_gpu(lib, h, Bs, a["m"], N)
        Cr, S = reference(a, Bs, dtype)
        worst = assert_close(C, Cr, S, dtype, "bcsr %s b=%d N=%d" % (dtype, b, N))
        C2 = run_gpu(lib, h, Bs, a["m"], N)
        assert np.array_equal(C, C2)                   # run-to-run identical
        return worst
    finally:
        lib.spmm_destroy(h)


def test_bcsr_tiny_config(lib):
    """configs[0]: 512 x 512 bf16, 64 x 64 blocks kept w.p. 0.5, B 512 x 256."""
    a = wl.bcsr_tiny()
    _bcsr_case(lib, a, "bf16", 64, 256)


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("b", [16, 32, 64, 128])
def test_bcsr_block_sizes(lib, dtype, b):
    a = wl.bcsr_sweep(300 + b, m=1024, k=768, b=b, density=0.2, dtype=dtype)
    _bcsr_case(lib, a, dtype, b, 640)                  # 640 = 512 + 128: several token tiles


@pytest.mark.parametrize("m,k,b,N", [(500, 300, 64, 200), (130, 70, 32, 72), (1000, 1000, 16, 1032),
                                      (257, 640, 128, 328), (64, 64, 64, 64)])
def test_bcsr_ragged_shapes(lib, m, k, b, N):
    """m, k not multiples of b; N not a multiple of the token tile; scattered entries."""
    a = wl.random_csr(7 + m, m, k, 0.02, "fp16", empty_rows=tuple(range(min(b, m // 2))))
    _bcsr_case(lib, a, "fp16", b, N)


@pytest.mark.parametrize("b", [16, 32, 64, 128])
def test_bcsr_tf32_block_sizes(lib, b):
    """fp32 storage, TF32 tensor-core arithmetic (the type of Sec. 4.1's BCSR evaluation; Sec. 3.1's
    k8 instruction shape): every block size, several token tiles, bound 2e-3."""
    a = wl.bcsr_sweep(400 + b, m=1024, k=768, b=b, density=0.2, dtype="tf32")
    worst = _bcsr_case(lib, a, "tf32", b, 640, Bdist=("normal", 0.0, 1.0))
    assert worst < 1.0


@pytest.mark.parametrize("m,k,b,N", [(500, 300, 64, 200), (130, 70, 32, 72), (1000, 1000, 16, 1032),
                                      (257, 640, 128, 328), (64, 64, 64, 64), (300, 200, 128, 2052)])
def test_bcsr_tf32_ragged_shapes(lib, m, k, b, N):
    """m, k not multiples of b; N not a multiple of the token tile (nor of the 32-token box)."""
    a = wl.random_csr(9 + m, m, k, 0.02, "tf32", empty_rows=tuple(range(min(b, m // 2))))
    _bcsr_case(lib, a, "tf32", b, N)


@pytest.mark.parametrize("b,N", [(16, 384), (32, 200), (64, 1024), (128, 520)])
def test_bcsr_tf32_colmajor(lib, b, N):
    """TF32 with column-major operands (X [N][k] in, Y [N][m] out): the plain K-major operand case,
    bit-identical to the row-major result (same products, same order)."""
    a = wl.bcsr_sweep(500 + b, m=512, k=768, b=b, density=0.3, dtype="tf32")
    Bs = wl.dense(11, a["k"], N, ("normal", 0.0, 1.0), "tf32")
    h0 = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "tf32", b)
    h1 = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "tf32", b, layout=lib.COLMAJOR)
    try:
        C0 = run_gpu(lib, h0, Bs, a["m"], N)
        C1 = run_gpu_variant(lib, h1, Bs, a["m"], N, "tf32", col_major=True)
        Cr, S = reference(a, Bs, "tf32")
        assert_close(C1, Cr, S, "tf32", "bcsr tf32 column-major b=%d" % b)
        assert np.array_equal(C0, C1)
    finally:
        lib.spmm_destroy(h0)
        lib.spmm_destroy(h1)


def test_bcsr_all_empty_and_identity(lib):
    rp = np.zeros(129, np.int64)
    a = dict(m=128, k=128, row_ptr=rp, col_idx=np.zeros(0, np.int32), vals=np.zeros(0, np.uint16))
    Bs = wl.dense(1, 128, 128, ("normal", 0.0, 1.0), "bf16")
    h = lib.spmm_bcsr_create_csr(128, 128, rp, a["col_idx"], a["vals"], "bf16", 64)
    assert not run_gpu(lib, h, Bs, 128, 128).any()
    lib.spmm_destroy(h)
    one = wl.to_storage(np.ones(128), "bf16")
    h = lib.spmm_bcsr_create_csr(128, 128, np.arange(129, dtype=np.int64), np.arange(128, dtype=np.int32), one, "bf16", 32)
    C = run_gpu(lib, h, Bs, 128, 128)
    assert np.array_equal(C.astype(np.float64), wl.widen(Bs, "bf16"))   # identity: exact
    lib.spmm_destroy(h)


def _wcsr_case(lib, a, dtype, N, T=0, Bdist=("normal", 0.0, 1.0), seed=19):
    Bs = wl.dense(seed, a["k"], N, Bdist, dtype)
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 16, split_cols=T)
    try:
        b_col = 32 // wl.elem_size(dtype)
        info = lib.spmm_get_info(h, N)
        f = F.wcsr_from_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], 16, b_col)
        np_dt = wl.storage_np_dtype(dtype)
        bits = {4: np.uint32, 2: np.uint16, 1: np.uint8}[wl.elem_size(dtype)]
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_ROW_PTR, np.int32), f["window_row_ptr"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_WINDOW_COL_IDX, np.int32), f["window_col_idx"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_VALUES, np_dt).view(bits), f["values"].view(bits).ravel())
        plan = F.split_plan(f["window_row_ptr"], info["split_cols"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_TASKS, np.int32).reshape(-1, 4), plan)
        bin_ptr, bin_tasks = F.task_bins(plan, info["n_bins"])
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_BIN_PTR, np.int32), bin_ptr)
        assert np.array_equal(lib.spmm_export(h, lib.X_WCSR_BIN_TASKS, np.int32), bin_tasks)
        C = run_gpu(lib, h, Bs, a["m"], N)
        Cr, S = reference(a, Bs, dtype)
        worst = assert_close(C, Cr, S, dtype, "wcsr %s N=%d T=%d" % (dtype, N, T))
        C2 = run_gpu(lib, h, Bs, a["m"], N)
        assert np.array_equal(C, C2)                   # deterministic merge
        return worst, info
    finally:
        lib.spmm_destroy(h)


@pytest.mark.parametrize("dtype", ["tf32", "fp16", "bf16"])
@pytest.mark.parametrize("N", [128, 32, 256, 72, 328])   # 328: three token tiles, ragged tail
def test_wcsr_small(lib, dtype, N):
    a = wl.random_csr(51, 1000, 900, 0.02, dtype, empty_rows=tuple(range(32, 64)))
    _, info = _wcsr_case(lib, a, dtype, N, T=64)
    assert info["n_split"] > 0 and info["n_empty"] >= 2


@pytest.mark.parametrize("N", [128, 32, 256, 80, 336])     # 80: ragged single tile; 336: three tiles, ragged tail
def test_wcsr_fp8_e4m3_small(lib, N):
    """E4M3 values (Sec. 5 names 8-bit inputs as the next step): windows padded to 32 columns = one
    K step of the 8-bit MMA, 128 gathered rows of 128 bytes per stage, fp32 C."""
    a = wl.random_csr(53, 1000, 900, 0.03, "fp8", empty_rows=tuple(range(32, 64)))
    _, info = _wcsr_case(lib, a, "fp8", N, T=64, Bdist=("uniform", -1.0, 1.0))
    assert info["n_split"] > 0 and info["n_empty"] >= 2


@pytest.mark.parametrize("T", [16, 256, 4096])
def test_wcsr_split_sizes_agree(lib, T):
    a = wl.wcsr_irregular(seed=5, m=4000, dtype="tf32")
    _wcsr_case(lib, a, "tf32", 128, T=T)


def test_wcsr_irregular_scaled(lib):
    """configs[1] recipe at 20,000 rows (the oracle finishes in seconds)."""
    a = wl.wcsr_irregular(seed=1002, m=20_000, dtype="tf32")
    worst, _ = _wcsr_case(lib, a, "tf32", 128)
    assert worst < 1.0


@pytest.mark.parametrize("dtype", ["fp16", "fp8"])
def test_wcsr_rmat_scaled(lib, dtype):
    """configs[4] recipe at 2^14 rows, fp16 (and E4M3 values), N = 32 / 128."""
    a = wl.rmat(scale=14, dtype=dtype)
    for N in (32, 128):
        _wcsr_case(lib, a, dtype, N, T=512)


def test_wcsr_ragged_rows_and_identity(lib):
    a = wl.random_csr(61, 1003, 77, 0.1, "fp16")
    _wcsr_case(lib, a, "fp16", 40)
    n = 100
    one = np.ones(n, np.float32)
    Bs = wl.dense(2, n, 64, ("normal", 0.0, 1.0), "tf32")
    h = lib.spmm_wcsr_create_csr(n, n, np.arange(n + 1, dtype=np.int64), np.arange(n, dtype=np.int32), one, "tf32", 16)
    C = run_gpu(lib, h, Bs, n, 64)
    lib.spmm_destroy(h)
    # identity: each output is one product 1.0 * b, exact up to the TF32 rounding of b
    assert np.max(np.abs(C - Bs) / np.maximum(np.abs(Bs), 1e-30)) <= 2.0 ** -10


def test_run_host_matches_device_run(lib):
    a = wl.bcsr_tiny()
    Bs = wl.dense(3, 512, 256, ("uniform", -1.0, 1.0), "bf16")
    h = lib.spmm_bcsr_create_csr(512, 512, a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64)
    C = run_gpu(lib, h, Bs, 512, 256)
    Ch = np.full((512, 256), np.nan, np.float32)
    lib.spmm_run_host(h, Bs, Ch, 256)
    assert np.array_equal(C, Ch)
    lib.spmm_destroy(h)


@pytest.mark.parametrize("case", ["wcsr_tf32", "bcsr_fp16", "bcsr_bf16_colmajor_c16", "wcsr_fp16_c16"])
def test_run_host_in_chunks_matches_device_run(lib, case):
    """Operands of 8 MB and more go through spmm_run_host in column chunks whose transfers overlap;
    the result is the one spmm_run gives on the whole operand, bit for bit, with pinned and with
    ordinary host memory, and the same again on the second call."""
    import torch
    c16 = case.endswith("c16")
    cm = "colmajor" in case
    if case.startswith("wcsr"):
        dtype = "tf32" if "tf32" in case else "fp16"
        a = wl.wcsr_irregular(seed=77, m=24000, dtype=dtype)
        N = 128 if dtype == "tf32" else 256
        h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 16,
                                     c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32)
    else:
        dtype = "bf16" if "bf16" in case else "fp16"
        a = wl.bcsr_sweep(78, m=4096, k=4096, b=32, density=0.1, dtype=dtype)
        N = 1024
        h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 32,
                                     c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32,
                                     layout=lib.COLMAJOR if cm else lib.ROWMAJOR)
    try:
        m, k = a["m"], a["k"]
        Bs = wl.dense(79, k, N, ("uniform", -1.0, 1.0), dtype)
        want = run_gpu_variant(lib, h, Bs, m, N, dtype, c16=c16, col_major=cm)       # m x N float32
        Bh = np.ascontiguousarray(Bs.T) if cm else np.ascontiguousarray(Bs)
        cdt = np.float32 if not c16 else np.uint16
        shape = (N, m) if cm else (m, N)
        assert Bh.nbytes + int(np.prod(shape)) * np.dtype(cdt).itemsize >= 8 << 20
        for pinned in (False, True, True):
            if pinned:
                Bt = torch.from_numpy(Bh.view(np.int16) if Bh.dtype == np.uint16 else Bh).pin_memory()
                Ct = torch.zeros(shape, dtype=torch.float32 if not c16 else torch.int16).pin_memory()
                lib.spmm_run_host(h, Bt.data_ptr(), Ct.data_ptr(), N)
                got_raw = Ct.numpy().view(cdt)
            else:
                got_raw = np.zeros(shape, dtype=cdt)
                lib.spmm_run_host(h, Bh, got_raw, N)
            lib.spmm_check(h)
            if c16:
                t16 = torch.from_numpy(got_raw.view(np.int16).copy()).view(torch.bfloat16 if dtype == "bf16" else torch.float16)
                got = t16.float().numpy()
            else:
                got = got_raw
            got = np.ascontiguousarray(got.T) if cm else got
            assert np.array_equal(got, want), "%s pinned=%s" % (case, pinned)
    finally:
        lib.spmm_destroy(h)


def test_bad_run_arguments(lib):
    import torch
    a = wl.bcsr_tiny()
    h = lib.spmm_bcsr_create_csr(512, 512, a["row_ptr"], a["col_idx"], a["vals"], "bf16", 64)
    buf = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    for args, code in (((buf.data_ptr(), buf.data_ptr(), 100), lib.SPMM_ERR_UNSUPPORTED),      # N*2 % 16 != 0
                       ((buf.data_ptr() + 2, buf.data_ptr(), 256), lib.SPMM_ERR_UNSUPPORTED),  # misaligned
                       ((0, buf.data_ptr(), 256), lib.SPMM_ERR_INVALID_ARG)):
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_run(h, *args)
        assert e.value.code == code
    lib.spmm_destroy(h)


@pytest.mark.parametrize("kind", ["bcsr", "wcsr", "bcsr_dynamic", "bcsr_row_groups"])
def test_wait_that_runs_out_is_reported_and_the_context_survives(lib, kind):
    """Every wait inside the kernels is bounded.  With the bound set to zero the first wait
    for operands that are still on their way runs out: the kernel leaves early
    through its normal teardown, spmm_check reports SPMM_ERR_DEV_TIMEOUT, and the same
    handle then works again once the bound is restored."""
    if kind == "bcsr_row_groups":
        # 10 % of the block-rows are full: they form row groups, so the step is two overlapping
        # launches (the second waits for the first before its CTAs exit) and both leave early
        a, dtype, size, N = wl.bcsr_sweep(406, m=2048, k=2048, b=16, density=0.1, dtype="fp16"), "fp16", 16, 1024
        mk = lib.spmm_bcsr_create_csr
    elif kind.startswith("bcsr"):
        a, dtype, size, N = wl.bcsr_sweep(404, m=2048, k=2048, b=64, density=0.3, dtype="fp16"), "fp16", 64, 1024
        mk = lib.spmm_bcsr_create_csr
        if kind == "bcsr_dynamic":       # tiles handed out at run time: the scheduler warp's waits are bounded too
            def mk(*args):
                return lib.spmm_bcsr_create_csr(*args, schedule=lib.SCHED_DYNAMIC)
    else:
        a, dtype, size, N = wl.wcsr_irregular(seed=405, m=20000, dtype="tf32"), "tf32", 16, 128
        mk = lib.spmm_wcsr_create_csr
    Bs = wl.dense(41, a["k"], N, ("normal", 0.0, 1.0), dtype)
    h = mk(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, size)
    try:
        if kind == "bcsr_row_groups":
            assert lib.spmm_get_info(h, N)["n_stacked_rows"] > 0
        lib.spmm_set_wait_limit_ns(0)
        run_gpu(lib, h, Bs, a["m"], N, check=False)
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_check(h)
        assert e.value.code == lib.SPMM_ERR_DEV_TIMEOUT
        lib.spmm_set_wait_limit_ns(2_000_000_000)
        lib.spmm_check(h)                                   # the status word was cleared
        C = run_gpu(lib, h, Bs, a["m"], N)
        Cr, S = reference(a, Bs, dtype)
        assert_close(C, Cr, S, dtype, "after timeout")
    finally:
        lib.spmm_set_wait_limit_ns(2_000_000_000)
        lib.spmm_destroy(h)
