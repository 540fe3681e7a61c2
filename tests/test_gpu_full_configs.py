"""GPU parity at the full sizes of the five benchmark configurations, launched exactly as
bench.py launches them (spmm_run on device-resident operands).

Where the oracle cannot afford every output, all rows are checked on a seeded subset of
columns: the columns of C are independent of one another (C[:, j] depends on B[:, j] only,
pinned in tests/test_oracle_spmm.py), and the subset covers the first, an interior and the
last position of a token tile, a tile boundary, the ragged end of N, and at least one column
of every 128-column group, hence of every token tile the launch computes.
"""
import numpy as np
import pytest

from paper_2604_17834_b200 import workloads as wl

from helpers import assert_close, reference, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2604_17834_b200 import binding
    return binding


def _sample_cols(N, seed):
    """Fixed positions (tile edges, the ragged end) plus one seeded column inside EVERY group of
    128 columns: whatever the kernel's token tile (128, 256 or 512 columns) and L2 slab, each
    tile of the launch holds at least one column the oracle checks."""
    fixed = [0, 1, 31, 32, 63, 64, 127, 128, 129, 255, 256, 511, 512, 513, N // 2, N - 129, N - 128, N - 65, N - 2, N - 1]
    rng = np.random.default_rng(seed)
    groups = np.arange(0, N, 128, dtype=np.int64)
    per_group = np.minimum(groups + rng.integers(0, 128, size=groups.shape[0]), N - 1)
    cols = set(c for c in fixed if 0 <= c < N) | set(per_group.tolist())
    return np.array(sorted(cols), dtype=np.int64)


def _run_and_check(lib, kind, a, dtype, size, N, Bs, cols=None, what="", c16=False, col_major=False):
    """Bs is the k x N operand.  c16: C in the input's 16-bit type; col_major: the device gets
    X = B^T (N x k) and returns Y = C^T (N x m)."""
    import torch
    mk = lib.spmm_bcsr_create_csr if kind == "bcsr" else lib.spmm_wcsr_create_csr
    h = mk(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], dtype, size,
           c_type=lib.C_SAME_AS_INPUT if c16 else lib.C_FP32, layout=lib.COLMAJOR if col_major else lib.ROWMAJOR)
    try:
        Bd = to_device(Bs)
        if col_major:
            Bd = Bd.t().contiguous()
        cdt = torch.float32 if not c16 else (torch.bfloat16 if dtype == "bf16" else torch.float16)
        shape = (N, a["m"]) if col_major else (a["m"], N)
        C = torch.full(shape, float("nan"), dtype=cdt, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        lib.spmm_run(h, Bd.data_ptr(), C.data_ptr(), N, st)
        torch.cuda.synchronize()
        lib.spmm_check(h)
        assert not bool(torch.isnan(C).any()), "%s: unwritten outputs" % what
        if cols is None:
            got = (C.t() if col_major else C).float().cpu().numpy()
            Cr, S = reference(a, Bs, dtype)
        else:
            ci = torch.from_numpy(cols).cuda()
            got = (C[ci, :].t() if col_major else C[:, ci]).float().cpu().numpy()
            Cr, S = reference(a, Bs, dtype, cols=cols)
        worst = assert_close(got, Cr, S, dtype, what)
        # second launch: same bits
        C2 = torch.empty_like(C)
        lib.spmm_run(h, Bd.data_ptr(), C2.data_ptr(), N, st)
        torch.cuda.synchronize()
        assert bool(torch.equal(C, C2)), "%s: run-to-run difference" % what
        return worst
    finally:
        lib.spmm_destroy(h)


def test_config1_wcsr_irregular_full(lib):
    """configs[1]: 100,000 x 100,000 TF32, N = 128 -- every output element."""
    a = wl.wcsr_irregular()
    Bs = wl.dense(1102, a["k"], 128, ("normal", 0.0, 1.0), "tf32")
    worst = _run_and_check(lib, "wcsr", a, "tf32", 16, 128, Bs, what="configs[1]")
    assert worst < 1.0


def test_config1_second_reading_zipf_1_8_full(lib):
    """configs[1] quotes a mean row length of 12, which Zipf(2) clipped at 5000 cannot give
    (its mean is near 6); an exponent of 1.8 does.  Same check on that second reading."""
    a = wl.wcsr_irregular(seed=1012, alpha=1.8)
    mean_len = float(a["row_ptr"][-1]) / a["m"]
    assert 10.0 < mean_len < 16.0
    Bs = wl.dense(1112, a["k"], 128, ("normal", 0.0, 1.0), "tf32")
    worst = _run_and_check(lib, "wcsr", a, "tf32", 16, 128, Bs, what="configs[1] zipf(1.8)")
    assert worst < 1.0


@pytest.mark.parametrize("shape", ["gate", "down"])
def test_config2_bcsr_llm_full(lib, shape):
    """configs[2]: 18944 x 3584 (gate) and 3584 x 18944 (down), 64 x 64 blocks, N = 65536."""
    a = wl.bcsr_llm() if shape == "gate" else wl.bcsr_llm(seed=1013, m=3584, k=18944)
    N = 65536
    Bs = wl.dense(1103, a["k"], N, ("normal", 0.0, 1.0), "bf16")
    _run_and_check(lib, "bcsr", a, "bf16", 64, N, Bs, cols=_sample_cols(N, 3), what="configs[2] " + shape)


@pytest.mark.parametrize("shape,c16,col_major", [("gate", True, False), ("gate", False, True), ("gate", True, True),
                                                  ("down", True, True)])
def test_config2_bcsr_llm_variants_full(lib, shape, c16, col_major):
    """configs[2] with C in bf16 and / or column-major operands (the linear-layer shape of
    Sec. 4.4: X [65536][k] in, Y [65536][m] out), as bench.py launches them."""
    a = wl.bcsr_llm() if shape == "gate" else wl.bcsr_llm(seed=1013, m=3584, k=18944)
    N = 65536
    Bs = wl.dense(1103, a["k"], N, ("normal", 0.0, 1.0), "bf16")
    _run_and_check(lib, "bcsr", a, "bf16", 64, N, Bs, cols=_sample_cols(N, 3), c16=c16, col_major=col_major,
                   what="configs[2] %s c16=%d cm=%d" % (shape, c16, col_major))


def test_config2_bcsr_llm_fp8_full(lib):
    """configs[2] gate shape with E4M3 weights and activations (column-major operands, fp32 Y)."""
    a = wl.bcsr_llm(dtype="fp8", std=0.5)
    N = 65536
    Bs = wl.dense(1103, a["k"], N, ("normal", 0.0, 1.0), "fp8", chunk_rows=256)
    _run_and_check(lib, "bcsr", a, "fp8", 64, N, Bs, cols=_sample_cols(N, 3), col_major=True, what="configs[2] gate fp8")


@pytest.mark.parametrize("b,d,skewed", [(16, 0.1, True), (32, 0.2, True), (64, 0.1, True), (128, 0.05, True),
                                         (64, 0.05, False), (16, 0.01, False), (128, 0.5, True)])
def test_config3_bcsr_sweep_full(lib, b, d, skewed):
    """configs[3]: 8192 x 8192 fp16, N = 4096, skewed block-row lengths and flat low densities."""
    a = wl.bcsr_sweep(1004 + b + int(d * 1000), b=b, density=d, skewed=skewed)
    N = 4096
    Bs = wl.dense(1104, a["k"], N, ("uniform", -1.0, 1.0), "fp16")
    _run_and_check(lib, "bcsr", a, "fp16", b, N, Bs, cols=_sample_cols(N, b), what="configs[3] b=%d d=%g" % (b, d))


@pytest.fixture(scope="module")
def rmat_full():
    return wl.rmat()


@pytest.mark.parametrize("N", [32, 128, 256])
def test_config4_wcsr_rmat_full(lib, rmat_full, N):
    """configs[4]: R-MAT 2^21 x 2^21, ~32.4 M nnz, fp16, N = 32 / 128 / 256."""
    a = rmat_full
    Bs = wl.dense(1105 + N, a["k"], N, ("normal", 0.0, 1.0), "fp16")
    # a third of the sampled positions, and in any case one column of every 128-column token tile
    cols = np.unique(np.concatenate([_sample_cols(N, N)[::3], np.arange(5, N, 128)])) if N > 32 else np.arange(0, 32, 3)
    _run_and_check(lib, "wcsr", a, "fp16", 16, N, Bs, cols=cols, what="configs[4] N=%d" % N)


def test_config4_wcsr_rmat_fp16_output_full(lib, rmat_full):
    """configs[4] at N = 128 with C written as fp16."""
    a = rmat_full
    Bs = wl.dense(1105 + 128, a["k"], 128, ("normal", 0.0, 1.0), "fp16")
    _run_and_check(lib, "wcsr", a, "fp16", 16, 128, Bs, cols=_sample_cols(128, 128)[::3], c16=True, what="configs[4] N=128 fp16 C")
