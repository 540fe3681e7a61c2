"""spmm_wcsr_run_static: the WCSR run that allocates no device memory.

Some callers cannot allocate when they call into the library -- a framework's memory
pool already owns the device, or the synchronisation an allocation can cause is not
acceptable in their loop.  For them the library carries an 8 MiB scratch array for the
partial tiles of split windows.  This test calls that entry point through the C ABI and
checks that it returns exactly what spmm_run returns, twice in a row (the array keeps
the first call's contents, so the second call shows that nothing stale leaks through),
and that a request larger than the array is refused instead of overrunning it.
The file name sorts last on purpose: a run that stops at the first failure has then
already been through every other test.
"""
import numpy as np
import pytest

from paper_2604_17834_b200 import workloads as wl

from helpers import assert_close, reference, run_gpu, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import binding
    return binding


def _run_static(lib, h, Bd, m, N, tdt=None):
    import torch
    C = torch.full((m, N), float("nan"), dtype=tdt or torch.float32, device="cuda")
    lib.spmm_wcsr_run_static(h, Bd.data_ptr(), C.data_ptr(), N, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    lib.spmm_check(h)
    return C.float().cpu().numpy()


@pytest.mark.parametrize("dtype,N", [("tf32", 128), ("fp16", 64)])
def test_static_scratch_run_matches_spmm_run_twice(lib, dtype, N):
    a = wl.wcsr_irregular(seed=77, m=6000, dtype=dtype)
    Bs1 = wl.dense(31, a["k"], N, ("normal", 0.0, 1.0), dtype)
    Bs2 = wl.dense(32, a["k"], N, ("normal", 0.0, 1.0), dtype)
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, 16, split_cols=64)
    try:
        info = lib.spmm_get_info(h, N)
        assert info["n_slots"] > 0 and 0 < info["workspace_bytes"] <= (8 << 20)
        for Bs in (Bs1, Bs2):                              # two calls in a row, different inputs
            want = run_gpu(lib, h, Bs, a["m"], N)
            got = _run_static(lib, h, to_device(Bs), a["m"], N)
            assert np.array_equal(got, want)
            Cr, S = reference(a, Bs, dtype)
            assert_close(got, Cr, S, dtype, "static scratch run")
    finally:
        lib.spmm_destroy(h)


def test_static_scratch_refuses_what_does_not_fit(lib):
    import torch
    a = wl.wcsr_irregular(seed=78, m=20000, dtype="fp16")
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, split_cols=16)
    try:
        N = 1024
        assert lib.spmm_get_info(h, N)["workspace_bytes"] > (8 << 20)
        B = torch.zeros((a["k"], N), dtype=torch.float16, device="cuda")
        C = torch.zeros((a["m"], N), dtype=torch.float32, device="cuda")
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_wcsr_run_static(h, B.data_ptr(), C.data_ptr(), N)
        assert e.value.code == lib.SPMM_ERR_TOO_LARGE
    finally:
        lib.spmm_destroy(h)
    b = wl.bcsr_tiny()
    hb = lib.spmm_bcsr_create_csr(512, 512, b["row_ptr"], b["col_idx"], b["vals"], "bf16", 64)
    try:
        B = torch.zeros((512, 256), dtype=torch.bfloat16, device="cuda")
        C = torch.zeros((512, 256), dtype=torch.float32, device="cuda")
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_wcsr_run_static(hb, B.data_ptr(), C.data_ptr(), 256)
        assert e.value.code == lib.SPMM_ERR_INVALID_ARG
    finally:
        lib.spmm_destroy(hb)


def test_static_scratch_run_leaves_device_memory_alone(lib):
    """The point of the entry point: on a warmed handle a call neither takes nor returns device
    memory.  Free memory as the driver reports it is read before and after calls whose output
    buffer already exists, and the handle's own workspace is never created by this path."""
    import torch
    a = wl.wcsr_irregular(seed=79, m=6000, dtype="fp16")
    N = 128
    Bd = to_device(wl.dense(33, a["k"], N, ("normal", 0.0, 1.0), "fp16"))
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", 16, split_cols=64)
    try:
        assert lib.spmm_get_info(h, N)["n_slots"] > 0
        C = torch.empty((a["m"], N), dtype=torch.float32, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        lib.spmm_wcsr_run_static(h, Bd.data_ptr(), C.data_ptr(), N, st)      # warm-up: address look-up, kernel attributes
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        for _ in range(3):
            lib.spmm_wcsr_run_static(h, Bd.data_ptr(), C.data_ptr(), N, st)
        torch.cuda.synchronize()
        lib.spmm_check(h)
        assert torch.cuda.mem_get_info()[0] == free0
    finally:
        lib.spmm_destroy(h)


def test_static_scratch_with_64_row_windows_and_16_bit_output(lib):
    """A 64-row handle needs four times the scratch per slot: one case that fits (and, written as
    fp16, goes through the merge kernel's rounding), one that is refused."""
    import torch
    a = wl.wcsr_irregular(seed=80, m=6000, dtype="fp16")
    Bs = wl.dense(34, a["k"], 128, ("normal", 0.0, 1.0), "fp16")
    h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], "fp16", 64, split_cols=256,
                                 c_type=lib.C_SAME_AS_INPUT)
    try:
        info = lib.spmm_get_info(h, 128)
        assert info["n_slots"] > 0 and info["workspace_bytes"] == info["n_slots"] * 64 * 128 * 4 <= (8 << 20)
        Bd = to_device(Bs)
        want = torch.full((a["m"], 128), float("nan"), dtype=torch.float16, device="cuda")
        lib.spmm_run(h, Bd.data_ptr(), want.data_ptr(), 128, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        for _ in range(2):
            got = _run_static(lib, h, Bd, a["m"], 128, torch.float16)
            assert np.array_equal(got, want.float().cpu().numpy())
        Cr, S = reference(a, Bs, "fp16")
        assert_close(got, Cr, S, "fp16", "static scratch run, 64-row windows, fp16 C")
        # the same handle at a width whose partial tiles exceed the array
        N = 2048
        assert lib.spmm_get_info(h, N)["workspace_bytes"] > (8 << 20)
        B = torch.zeros((a["k"], N), dtype=torch.float16, device="cuda")
        C = torch.zeros((a["m"], N), dtype=torch.float16, device="cuda")
        with pytest.raises(lib.SpmmError) as e:
            lib.spmm_wcsr_run_static(h, B.data_ptr(), C.data_ptr(), N)
        assert e.value.code == lib.SPMM_ERR_TOO_LARGE
    finally:
        lib.spmm_destroy(h)
