"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random inputs and converts them to their storage
dtype.  It holds none of the method's arithmetic (no format construction, no
multiplication) and is the one module that both the CPU oracle's tests and
the CUDA path's tests / benchmark may use.  It imports neither of them.

All draws use ``numpy.random.default_rng(seed)`` (PCG64) and happen in the
order written in each function, so a (function, arguments, seed) triple names
one input exactly.

Stand-ins (the paper's own data is not available here):
  * ``wcsr_irregular`` / ``rmat`` stand in for the SuiteSparse selection of
    Sec. 4.1 (power-law row lengths, a diagonal band that mimics the
    locality left by the reordering the paper applies, graph adjacency).
  * ``bcsr_llm`` stands in for the block-pruned Qwen2.5-7B FFN weights of
    Sec. 4.4 (shapes 18944 x 3584 and 3584 x 18944, 64 x 64 blocks).
  * ``bcsr_tiny`` / ``bcsr_sweep`` are block-sparse matrices with dense kept
    blocks (the block sparsity of Sec. 1 / Sec. 2.3).

Storage dtypes: "bf16" travels as uint16 bit patterns (numpy has no
bfloat16), "fp16" as numpy.float16, "tf32" as numpy.float32 (fp32 storage,
TF32 tensor-core arithmetic), "fp8" as uint8 bit patterns of E4M3 (1 sign,
4 exponent bits with bias 7, 3 mantissa bits; no infinities, largest finite
value 448; the all-ones exponent-and-mantissa code is NaN and never drawn).
"""
from __future__ import annotations

import numpy as np

DTYPES = ("bf16", "fp16", "tf32", "fp8")


# --------------------------------------------------------------------------- dtype helpers


def to_storage(x, dtype):
    """Round an fp32/fp64 array to the storage dtype (round-to-nearest-even)."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "tf32":
        return x32
    if dtype == "fp16":
        return x32.astype(np.float16)
    if dtype == "bf16":
        u = x32.view(np.uint32)
        rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
        return (rounded >> np.uint32(16)).astype(np.uint16)
    if dtype == "fp8":
        # nearest E4M3 value, ties to the even code, saturating at +-448
        mag = _e4m3_magnitudes()                              # codes 0..126, ascending
        ax = np.minimum(np.abs(x32.astype(np.float64)), mag[-1])
        hi = np.clip(np.searchsorted(mag, ax, side="left"), 1, mag.shape[0] - 1)
        lo = hi - 1
        dlo, dhi = ax - mag[lo], mag[hi] - ax
        code = np.where(dlo < dhi, lo, np.where(dhi < dlo, hi, np.where(lo % 2 == 0, lo, hi)))
        return (code.astype(np.uint8) | (np.signbit(x32).astype(np.uint8) << np.uint8(7))).astype(np.uint8)
    raise ValueError(dtype)


def _e4m3_magnitudes():
    """Values of the E4M3 codes 0 .. 126 (sign bit clear, NaN code 127 left out)."""
    code = np.arange(127)
    e, m = code >> 3, code & 7
    return np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7.0))


def widen(s, dtype):
    """Exact widening of a storage array to float64."""
    s = np.asarray(s)
    if dtype == "bf16":
        return (s.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if dtype == "fp8":
        mag = np.append(_e4m3_magnitudes(), np.nan)
        return np.where(s >> 7 == 1, -1.0, 1.0) * mag[s & 0x7F]
    return s.astype(np.float64)


def elem_size(dtype):
    return {"tf32": 4, "fp8": 1}.get(dtype, 2)


def storage_np_dtype(dtype):
    return {"bf16": np.uint16, "fp16": np.float16, "tf32": np.float32, "fp8": np.uint8}[dtype]


def dense(seed, rows, cols, dist, dtype, chunk_rows=4096):
    """Dense [rows, cols] operand in storage dtype.

    dist = ("uniform", lo, hi) or ("normal", mean, std).  Drawn row-chunk by
    row-chunk (chunk_rows rows at a time, fp32 draws) from one generator.
    """
    rng = np.random.default_rng(seed)
    out = np.empty((rows, cols), dtype=storage_np_dtype(dtype))
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        if dist[0] == "uniform":
            x = rng.random((r1 - r0, cols), dtype=np.float32) * np.float32(dist[2] - dist[1]) + np.float32(dist[1])
        elif dist[0] == "normal":
            x = rng.standard_normal((r1 - r0, cols), dtype=np.float32) * np.float32(dist[2]) + np.float32(dist[1])
        else:
            raise ValueError(dist)
        out[r0:r1] = to_storage(x, dtype)
    return out


def _draw_vals(rng, n, dist, dtype):
    if dist[0] == "uniform":
        x = rng.random(n, dtype=np.float32) * np.float32(dist[2] - dist[1]) + np.float32(dist[1])
    elif dist[0] == "normal":
        x = rng.standard_normal(n, dtype=np.float32) * np.float32(dist[2]) + np.float32(dist[1])
    elif dist[0] == "uniform_open0":       # (0, 1]
        x = np.float32(1.0) - rng.random(n, dtype=np.float32)
    else:
        raise ValueError(dist)
    return to_storage(x, dtype)


# --------------------------------------------------------------------------- block-sparse matrices


def csr_from_block_mask(mask, b, m, k):
    """CSR index arrays of a matrix whose kept b x b blocks (mask[I, J]) are dense.

    Entries outside m x k (ragged edge) are dropped.  Returns (row_ptr int64,
    col_idx int32).
    """
    nbr, nbc = mask.shape
    cols_parts = []
    row_len = np.zeros(m, dtype=np.int64)
    ar = np.arange(b, dtype=np.int64)
    for I in range(nbr):
        J = np.nonzero(mask[I])[0].astype(np.int64)
        r0, r1 = I * b, min(m, (I + 1) * b)
        if r1 <= r0:
            continue
        cols_row = (J[:, None] * b + ar[None, :]).ravel()
        cols_row = cols_row[cols_row < k]
        row_len[r0:r1] = cols_row.shape[0]
        if cols_row.shape[0]:
            cols_parts.append(np.tile(cols_row, r1 - r0))
    row_ptr = np.zeros(m + 1, dtype=np.int64)
    row_ptr[1:] = np.cumsum(row_len)
    col_idx = np.concatenate(cols_parts).astype(np.int32) if cols_parts else np.zeros(0, np.int32)
    return row_ptr, col_idx


def bcsr_tiny(seed=1001, m=512, k=512, b=64, keep=0.5, dtype="bf16"):
    """Block grid with each block kept with probability ``keep``; kept blocks dense U[-1,1].

    Draw order: block mask (row-major), then values in CSR order.
    """
    rng = np.random.default_rng(seed)
    nbr, nbc = -(-m // b), -(-k // b)
    mask = rng.random((nbr, nbc)) < keep
    row_ptr, col_idx = csr_from_block_mask(mask, b, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], ("uniform", -1.0, 1.0), dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals, block=b)


def bcsr_llm(seed=1003, m=18944, k=3584, b=64, sparsity=0.9, dtype="bf16", std=0.02):
    """Block-pruned weight matrix: exactly floor(sparsity * #blocks) blocks removed.

    Draw order: permutation of all blocks (kept = the first #blocks - floor(sparsity * #blocks)
    entries of the permutation), then values N(0, std) in CSR order.
    """
    rng = np.random.default_rng(seed)
    nbr, nbc = -(-m // b), -(-k // b)
    nblocks = nbr * nbc
    nkeep = nblocks - int(np.floor(sparsity * nblocks))
    perm = rng.permutation(nblocks)
    mask = np.zeros(nblocks, dtype=bool)
    mask[perm[:nkeep]] = True
    mask = mask.reshape(nbr, nbc)
    row_ptr, col_idx = csr_from_block_mask(mask, b, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], ("normal", 0.0, std), dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals, block=b)


def bcsr_sweep(seed, m=8192, k=8192, b=64, density=0.1, skewed=True, dtype="fp16"):
    """Block-sparse matrix with skewed block-row lengths.

    skewed: a seeded permutation of the block-rows picks the first 10 % as
    full, the next 20 % as empty, and every block of the rest is kept with
    probability ``density``.  Not skewed: every block kept with probability
    ``density``.  Kept blocks are dense U[-1,1].
    Draw order: block-row permutation (skewed only), Bernoulli mask (row-major,
    all block-rows), values in CSR order.
    """
    rng = np.random.default_rng(seed)
    nbr, nbc = -(-m // b), -(-k // b)
    if skewed:
        perm = rng.permutation(nbr)
        nfull, nempty = int(round(0.1 * nbr)), int(round(0.2 * nbr))
    mask = rng.random((nbr, nbc)) < density
    if skewed:
        mask[perm[:nfull]] = True
        mask[perm[nfull:nfull + nempty]] = False
    row_ptr, col_idx = csr_from_block_mask(mask, b, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], ("uniform", -1.0, 1.0), dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals, block=b)


def bcsr_families(seed, m=8192, k=8192, b=16, density=0.1, n_families=32, drop=0.1, dtype="fp16"):
    """Block-sparse matrix whose block-rows come in families scattered over the row range (the
    pattern structured pruning leaves when channels that are pruned together are not adjacent).

    Every family has a Bernoulli(density) mask over the block columns; every block-row is
    assigned a family uniformly at random, takes that family's mask and drops each kept block
    with probability ``drop``.  Kept blocks are dense U[-1,1].
    Draw order: family masks (row-major), family of every block-row, drop mask (row-major, all
    blocks), values in CSR order.
    """
    rng = np.random.default_rng(seed)
    nbr, nbc = -(-m // b), -(-k // b)
    fam_mask = rng.random((n_families, nbc)) < density
    fam = rng.integers(0, n_families, size=nbr)
    mask = fam_mask[fam] & (rng.random((nbr, nbc)) >= drop)
    row_ptr, col_idx = csr_from_block_mask(mask, b, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], ("uniform", -1.0, 1.0), dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals, block=b)


# --------------------------------------------------------------------------- irregular matrices


def _csr_from_keys(keys, m, k):
    """Sorted unique (row * k + col) keys -> (row_ptr int64, col_idx int32)."""
    rows = keys // k
    row_ptr = np.zeros(m + 1, dtype=np.int64)
    row_ptr[1:] = np.cumsum(np.bincount(rows, minlength=m))
    return row_ptr, (keys % k).astype(np.int32)


def wcsr_irregular(seed=1002, m=100_000, k=None, alpha=2.0, max_len=5000, band=256,
                   dtype="tf32"):
    """Power-law row lengths, half the entries uniform and half in a diagonal band.

    Draw order: row lengths min(zipf(alpha), max_len); per entry a coin
    (uniform column vs. band); uniform columns; band offsets in [-band, band]
    (clipped to the matrix); duplicates inside a row merged; values N(0,1) in
    CSR order after merging.
    """
    k = m if k is None else k
    rng = np.random.default_rng(seed)
    length = np.minimum(rng.zipf(alpha, size=m), max_len).astype(np.int64)
    rows = np.repeat(np.arange(m, dtype=np.int64), length)
    n = rows.shape[0]
    coin = rng.random(n) < 0.5
    ucol = rng.integers(0, k, size=n, dtype=np.int64)
    off = rng.integers(-band, band + 1, size=n, dtype=np.int64)
    bcol = np.clip(rows * k // m + off, 0, k - 1)
    col = np.where(coin, ucol, bcol)
    keys = np.unique(rows * k + col)
    row_ptr, col_idx = _csr_from_keys(keys, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], ("normal", 0.0, 1.0), dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals)


def rmat(seed=1005, scale=21, edge_factor=16, probs=(0.57, 0.19, 0.19, 0.05), dtype="fp16",
         chunk=1 << 22):
    """R-MAT adjacency matrix, 2^scale rows and columns, edge_factor * 2^scale edge draws.

    Draw order: edges in chunks of ``chunk``; inside a chunk one uniform draw
    per edge per level, most significant bit first (quadrants in the order
    (0,0), (0,1), (1,0), (1,1) with the given probabilities); duplicates
    merged (directed, not symmetrised); values U(0,1] in CSR order after
    merging.
    """
    rng = np.random.default_rng(seed)
    n = 1 << scale
    nedges = edge_factor * n
    a, b_, c, _ = probs
    t1, t2, t3 = a, a + b_, a + b_ + c
    parts = []
    for e0 in range(0, nedges, chunk):
        ne = min(chunk, nedges - e0)
        r = np.zeros(ne, dtype=np.int64)
        cc = np.zeros(ne, dtype=np.int64)
        for _lvl in range(scale):
            u = rng.random(ne, dtype=np.float32)
            rbit = (u >= t2)
            cbit = ((u >= t1) & (u < t2)) | (u >= t3)
            r = (r << 1) | rbit
            cc = (cc << 1) | cbit
        parts.append(np.unique(r * n + cc))
    keys = np.unique(np.concatenate(parts))
    row_ptr, col_idx = _csr_from_keys(keys, n, n)
    vals = _draw_vals(rng, col_idx.shape[0], ("uniform_open0",), dtype)
    return dict(m=n, k=n, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals)


def random_csr(seed, m, k, density, dtype, dist=("uniform", -1.0, 1.0), empty_rows=()):
    """Small unstructured matrix for tests: every entry kept with probability ``density``."""
    rng = np.random.default_rng(seed)
    mask = rng.random((m, k)) < density
    for r in empty_rows:
        mask[r] = False
    rows, cols = np.nonzero(mask)
    keys = rows.astype(np.int64) * k + cols.astype(np.int64)
    row_ptr, col_idx = _csr_from_keys(keys, m, k)
    vals = _draw_vals(rng, col_idx.shape[0], dist, dtype)
    return dict(m=m, k=k, dtype=dtype, row_ptr=row_ptr, col_idx=col_idx, vals=vals)
