"""Shared pieces of the GPU parity tests: run the CUDA path through the C ABI and
compare it element by element with the fp64 oracle under the stated bound

    |C_gpu - C_ref| <= tau * sum_k |a_ik b_kj| + 1e-6,

tau = 8e-3 for bf16 / fp16 (and E4M3) inputs, 2e-3 for the TF32 path (fp32 accumulation).
"""
import numpy as np

from oracle import spmm_ref
from paper_2604_17834_b200 import workloads as wl

TAU = {"bf16": 8e-3, "fp16": 8e-3, "tf32": 2e-3, "fp8": 8e-3}


def to_device(arr):
    """numpy storage array -> torch CUDA tensor holding the same bytes."""
    import torch
    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


GUARD = 8192          # elements of canary on either side of C
CANARY = 24576.0      # exact in fp32, fp16 and bf16


def guarded_c(shape, tdt, fill):
    """C inside a larger allocation whose margins hold a canary value: a store that lands outside C
    (a tile clipped wrongly, a row index off by one block) shows up in check_guards.
    -> (whole buffer, view of C with the requested shape)."""
    import torch
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), CANARY, dtype=tdt, device="cuda")
    C = buf[GUARD:GUARD + n].view(*shape)
    C.fill_(fill)
    return buf, C


def check_guards(buf, what=""):
    import torch
    lo, hi = buf[:GUARD].float(), buf[-GUARD:].float()
    assert bool(torch.all(lo == CANARY)) and bool(torch.all(hi == CANARY)), "%s: a store landed outside C" % what


def run_gpu(lib, h, B_storage, m, N, fill=float("nan"), check=True):
    """One spmm_run on device buffers; C is pre-filled with NaN so unwritten elements show, and
    sits between two canary margins so that stores outside it show as well."""
    import torch
    Bd = to_device(B_storage)
    buf, C = guarded_c((m, N), torch.float32, fill)
    lib.spmm_run(h, Bd.data_ptr(), C.data_ptr(), N, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    if check:
        lib.spmm_check(h)
    check_guards(buf, "spmm_run")
    return C.cpu().numpy()


def run_gpu_variant(lib, h, B_storage, m, N, dtype, c16=False, col_major=False, check=True):
    """spmm_run for a handle created with c_type / layout options.  B_storage is always the
    k x N operand; with col_major the device gets X = B^T (N x k) and returns Y = C^T (N x m).
    The result comes back as an m x N float32 array either way."""
    import torch
    Bs = np.ascontiguousarray(B_storage.T) if col_major else B_storage
    Bd = to_device(Bs)
    tdt = torch.float32 if not c16 else (torch.bfloat16 if dtype == "bf16" else torch.float16)
    shape = (N, m) if col_major else (m, N)
    buf, C = guarded_c(shape, tdt, float("nan"))
    lib.spmm_run(h, Bd.data_ptr(), C.data_ptr(), N, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    if check:
        lib.spmm_check(h)
    check_guards(buf, "spmm_run")
    out = C.float().cpu().numpy()
    return np.ascontiguousarray(out.T) if col_major else out


def reference(a, B_storage, dtype, cols=None, rows=None):
    v64 = wl.widen(a["vals"], dtype)
    B64 = wl.widen(B_storage if cols is None else B_storage[:, cols], dtype)
    return spmm_ref(a["row_ptr"], a["col_idx"], v64, B64, rows=rows)


def assert_close(C_gpu, C_ref, S, dtype, what=""):
    assert C_gpu.shape == C_ref.shape
    assert np.all(np.isfinite(C_gpu)), "%s: %d non-finite / unwritten outputs" % (what, int((~np.isfinite(C_gpu)).sum()))
    err = np.abs(C_gpu.astype(np.float64) - C_ref)
    bound = TAU[dtype] * S + 1e-6
    bad = err > bound
    if bad.any():
        i, j = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError("%s: %d of %d outside the bound; worst at (%d,%d): gpu %.6g ref %.6g err %.3g bound %.3g"
                             % (what, int(bad.sum()), err.size, i, j, C_gpu[i, j], C_ref[i, j], err[i, j], bound[i, j]))
    return float(np.max(err / bound))
