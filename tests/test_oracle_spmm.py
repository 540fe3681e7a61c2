"""Pins for the fp64 SpMM oracle (Sec. 2.3: C = A x B with sparse A, dense B).

None of these re-type the oracle's loop: each compares it with something the
mathematics fixes independently (a dense triple loop over the expanded
matrix, identity / permutation behaviour, a closed form, exact integer
linearity, column independence).
"""
import numpy as np
import pytest

from oracle import spmm_ref
from paper_2604_17834_b200 import workloads as wl


def _dense_from_csr(m, k, row_ptr, col_idx, vals64):
    A = np.zeros((m, k), dtype=np.float64)
    for i in range(m):
        for p in range(row_ptr[i], row_ptr[i + 1]):
            A[i, col_idx[p]] = vals64[p]
    return A


def _brute(A, B):
    m, k = A.shape
    n = B.shape[1]
    C = np.zeros((m, n))
    S = np.zeros((m, n))
    for i in range(m):
        for j in range(n):
            acc = 0.0
            sab = 0.0
            for p in range(k):
                t = A[i, p] * B[p, j]
                acc += t
                sab += abs(t)
            C[i, j] = acc
            S[i, j] = sab
    return C, S


@pytest.mark.parametrize("dtype", wl.DTYPES)
@pytest.mark.parametrize("shape", [(7, 5, 3), (33, 40, 17), (64, 64, 8)])
def test_matches_dense_triple_loop(dtype, shape):
    m, k, n = shape
    a = wl.random_csr(11 + m, m, k, 0.3, dtype, empty_rows=(1,))
    Bs = wl.dense(5 + n, k, n, ("normal", 0.0, 1.0), dtype)
    v64, B64 = wl.widen(a["vals"], dtype), wl.widen(Bs, dtype)
    C, S = spmm_ref(a["row_ptr"], a["col_idx"], v64, B64)
    Cb, Sb = _brute(_dense_from_csr(m, k, a["row_ptr"], a["col_idx"], v64), B64)
    # same products, different summation order (zeros interleaved): agree to fp64 rounding
    assert np.max(np.abs(C - Cb)) <= 1e-13 * max(1.0, Sb.max())
    assert np.max(np.abs(S - Sb)) <= 1e-13 * max(1.0, Sb.max())
    assert np.all(C[1] == 0.0) and np.all(S[1] == 0.0)      # empty row -> zero row


def test_identity_returns_B_bit_for_bit():
    k, n = 50, 9
    B = wl.widen(wl.dense(3, k, n, ("normal", 0.0, 1.0), "bf16"), "bf16")
    row_ptr = np.arange(k + 1, dtype=np.int64)
    C, S = spmm_ref(row_ptr, np.arange(k, dtype=np.int32), np.ones(k), B)
    assert np.array_equal(C, B)
    assert np.array_equal(S, np.abs(B))


def test_permutation_permutes_rows():
    k, n = 41, 6
    rng = np.random.default_rng(0)
    perm = rng.permutation(k).astype(np.int32)
    B = rng.standard_normal((k, n))
    C, _ = spmm_ref(np.arange(k + 1, dtype=np.int64), perm, np.ones(k), B)
    assert np.array_equal(C, B[perm])


def test_all_ones_gives_row_counts():
    a = wl.random_csr(21, 30, 25, 0.4, "fp16", empty_rows=(0, 29))
    ones = np.ones(a["col_idx"].shape[0])
    C, S = spmm_ref(a["row_ptr"], a["col_idx"], ones, np.ones((25, 4)))
    want = np.diff(a["row_ptr"]).astype(np.float64)[:, None] * np.ones((1, 4))
    assert np.array_equal(C, want) and np.array_equal(S, want)


def test_linearity_is_exact_on_integers():
    rng = np.random.default_rng(4)
    a = wl.random_csr(22, 20, 31, 0.3, "tf32")
    vals = rng.integers(-8, 9, size=a["col_idx"].shape[0]).astype(np.float64)
    B1 = rng.integers(-16, 17, size=(31, 5)).astype(np.float64)
    B2 = rng.integers(-16, 17, size=(31, 5)).astype(np.float64)
    C1, _ = spmm_ref(a["row_ptr"], a["col_idx"], vals, B1)
    C2, _ = spmm_ref(a["row_ptr"], a["col_idx"], vals, B2)
    C12, _ = spmm_ref(a["row_ptr"], a["col_idx"], vals, B1 + B2)
    assert np.array_equal(C12, C1 + C2)
    Cm, _ = spmm_ref(a["row_ptr"], a["col_idx"], -3.0 * vals, B1)
    assert np.array_equal(Cm, -3.0 * C1)


def test_sign_and_transpose_sensitivity():
    # A = [[0, 2], [0, 0]], B = [[1, 10], [100, 1000]]: C[0] = 2 * B[1]; a transposed
    # operand or swapped index would give a different, easily told apart, result.
    row_ptr = np.array([0, 1, 1], dtype=np.int64)
    C, S = spmm_ref(row_ptr, np.array([1], np.int32), np.array([-2.0]),
                    np.array([[1.0, 10.0], [100.0, 1000.0]]))
    assert np.array_equal(C, np.array([[-200.0, -2000.0], [0.0, 0.0]]))
    assert np.array_equal(S, np.array([[200.0, 2000.0], [0.0, 0.0]]))


def test_columns_are_independent_and_row_ranges_compose():
    a = wl.random_csr(23, 40, 37, 0.2, "fp16")
    v = wl.widen(a["vals"], "fp16")
    B = wl.widen(wl.dense(8, 37, 12, ("uniform", -1.0, 1.0), "fp16"), "fp16")
    C, S = spmm_ref(a["row_ptr"], a["col_idx"], v, B)
    sel = [0, 5, 11]
    Cs, Ss = spmm_ref(a["row_ptr"], a["col_idx"], v, B[:, sel])
    assert np.array_equal(Cs, C[:, sel]) and np.array_equal(Ss, S[:, sel])
    Ca, _ = spmm_ref(a["row_ptr"], a["col_idx"], v, B, rows=(0, 13))
    Cb, _ = spmm_ref(a["row_ptr"], a["col_idx"], v, B, rows=(13, 40))
    assert np.array_equal(Ca + Cb, C)
    assert np.all(Ca[13:] == 0.0)


def test_matches_scipy_on_a_medium_matrix():
    import scipy.sparse as sp
    a = wl.wcsr_irregular(seed=7, m=3000, alpha=2.0, dtype="tf32")
    v = wl.widen(a["vals"], "tf32")
    B = np.random.default_rng(1).standard_normal((a["k"], 16))
    C, S = spmm_ref(a["row_ptr"], a["col_idx"], v, B)
    M = sp.csr_matrix((v, a["col_idx"], a["row_ptr"]), shape=(a["m"], a["k"]))
    assert np.max(np.abs(C - M @ B)) <= 1e-12 * S.max()


def test_rejects_out_of_range_column():
    with pytest.raises(ValueError):
        spmm_ref(np.array([0, 1], np.int64), np.array([3], np.int32), np.ones(1), np.ones((3, 2)))


def test_e4m3_storage_matches_an_independent_conversion():
    """The E4M3 quantiser of the input generators (nearest, ties to even) against torch's
    float8_e4m3fn cast, and its decoder against torch's widening, on values inside the finite
    range; saturation and the sign of zero separately."""
    import torch
    rng = np.random.default_rng(12)
    x = np.concatenate([rng.standard_normal(50000).astype(np.float32) * 3.0,
                        rng.standard_normal(50000).astype(np.float32) * 0.01,
                        np.array([0.0, 448.0, -448.0, 2.0 ** -9, 2.0 ** -10, 1.0625, 1.1875, 0.4375 + 2.0 ** -5], np.float32)])
    code = wl.to_storage(x, "fp8")
    t = torch.from_numpy(x).to(torch.float8_e4m3fn)
    assert np.array_equal(code, t.view(torch.uint8).numpy())
    assert np.array_equal(wl.widen(code, "fp8"), t.float().numpy().astype(np.float64))
    assert wl.widen(wl.to_storage(np.array([1e6, -1e6], np.float32), "fp8"), "fp8").tolist() == [448.0, -448.0]
    z = wl.to_storage(np.array([-0.0], np.float32), "fp8")
    assert z[0] == 0x80 and np.signbit(wl.widen(z, "fp8"))[0]


def test_bf16_and_fp16_storage_match_independent_conversions():
    """The 16-bit quantisers of the input generators (round to nearest, ties to even) and their
    exact widening against torch's casts: normal values, ties, subnormals of bf16, large values."""
    import torch
    rng = np.random.default_rng(13)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 2.0,
                        rng.standard_normal(20000).astype(np.float32) * 1e-3,
                        rng.standard_normal(2000).astype(np.float32) * 1e-40,       # subnormal in bf16 and fp32
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -3.0e38, 65504.0, 2.0 ** -24], np.float32)])
    t = torch.from_numpy(x)
    b = wl.to_storage(x, "bf16")
    assert b.dtype == np.uint16
    assert np.array_equal(b, t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(wl.widen(b, "bf16"), t.to(torch.bfloat16).to(torch.float64).numpy())
    xh = x[np.abs(x) < 60000.0]
    h = wl.to_storage(xh, "fp16")
    th = torch.from_numpy(xh).to(torch.float16)
    assert np.array_equal(h.view(np.uint16), th.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(wl.widen(h, "fp16"), th.to(torch.float64).numpy())
    # the tie cases by hand: 1 + 2^-8 is halfway between two bf16 values -> the even one (1.0);
    # 1 + 3 * 2^-8 is halfway as well -> the even one above (1 + 2^-6)
    assert wl.widen(wl.to_storage(np.array([1.00390625, 1.01171875], np.float32), "bf16"), "bf16").tolist() == [1.0, 1.015625]
