"""Seeded synthetic inputs for the SpMM path  C = alpha*A*B + beta*C.

This module only *draws inputs*: CSR structure, values, dense operands and the
scalars.  It holds none of the method's arithmetic (no products, no sums of
products, no format conversion, no structure analysis) and is the one piece of
code that both the CPU oracle's tests and the CUDA path's tests / bench use.

Five generators follow the five benchmark workloads:

  g1_tiny_uniform   Poisson(8) row lengths, distinct uniform columns
  g2_stencil        5-point 2-D Laplacian, natural ordering
  g3_gcn_rmat       symmetrised R-MAT graph + I, D^-1/2 (A+I) D^-1/2 values
  g4_block          fully dense 16x16 blocks at random block positions
  g5_skewed         rank-size (Zipf 1.2) row lengths, distinct uniform columns

Every generator takes size parameters so that tests can run scaled-down cases
with the same structure, and a `seed`.  The default seed of config `i` is
0x5D170000 + i.  bf16 data are produced by rounding the fp32 draws to nearest
even once, here; both consumers receive the same uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

SEED_BASE = 0x5D170000
SD_F32 = 0
SD_BF16 = 1


@dataclass
class Workload:
    name: str
    M: int
    K: int
    N: int
    rowptr: np.ndarray          # int32 [M+1]
    colind: np.ndarray          # int32 [nnz], ascending inside a row
    vals: np.ndarray            # float32 [nnz]  or uint16 [nnz] (bf16 bits)
    B: np.ndarray               # float32 [K, N] or uint16 [K, N] (bf16 bits)
    C0: np.ndarray | None       # float32 [M, N] initial C (None when beta == 0)
    alpha: float = 1.0
    beta: float = 0.0
    dtype: int = SD_F32
    meta: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])

    def compulsory_bytes(self) -> int:
        """Bytes of the compulsory-traffic model: A (values, indices, rowptr)
        read once, B read once, C written once, C read once when beta != 0."""
        es = 4 if self.dtype == SD_F32 else 2
        b = self.nnz * (es + 4) + 4 * (self.M + 1)
        b += self.K * self.N * es
        b += 4 * self.M * self.N * (2 if self.beta != 0.0 else 1)
        return b

    def flops(self) -> int:
        return 2 * self.nnz * self.N


# --------------------------------------------------------------------------
# helpers (random draws and bit casts only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_f32(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(size=shape, dtype=np.float32)


def _uniform_pm1_f32(rng: np.random.Generator, n: int) -> np.ndarray:
    return (rng.random(size=n, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)).astype(np.float32)


def _rowptr_from_lengths(lengths: np.ndarray) -> np.ndarray:
    rp = np.zeros(lengths.size + 1, dtype=np.int64)
    np.cumsum(lengths, out=rp[1:])
    if rp[-1] >= 2**31:
        raise ValueError("nnz does not fit int32")
    return rp.astype(np.int32)


def distinct_sorted_columns(rng: np.random.Generator, lengths: np.ndarray, K: int) -> np.ndarray:
    """For each row i draw lengths[i] distinct columns uniformly from [0, K),
    ascending inside the row.  Duplicates are re-drawn until none is left, which
    is sequential sampling without replacement."""
    lengths = np.asarray(lengths, dtype=np.int64)
    if np.any(lengths > K):
        raise ValueError("row longer than K")
    M = lengths.size
    nnz = int(lengths.sum())
    rows = np.repeat(np.arange(M, dtype=np.int64), lengths)
    key = rows * np.int64(K) + rng.integers(0, K, size=nnz, dtype=np.int64)
    del rows
    key.sort(kind="stable")
    # rows that still hold a duplicate are re-drawn as a (small) sub-problem
    while True:
        dup = np.flatnonzero(key[1:] == key[:-1]) + 1
        if dup.size == 0:
            break
        bad_rows = np.unique(key[dup] // K)
        rp = np.zeros(M + 1, dtype=np.int64)
        np.cumsum(lengths, out=rp[1:])
        for r in bad_rows:
            lo, hi = int(rp[r]), int(rp[r + 1])
            if hi - lo == K:   # a full row holds every column: nothing to draw
                key[lo:hi] = np.arange(K, dtype=np.int64) + r * K
                continue
            seg = key[lo:hi] - r * K
            while True:
                u = np.unique(seg)
                if u.size == seg.size:
                    break
                extra = rng.integers(0, K, size=seg.size - u.size, dtype=np.int64)
                seg = np.concatenate([u, extra])
            key[lo:hi] = np.sort(seg) + r * K
    return (key % K).astype(np.int32)


# --------------------------------------------------------------------------
# config 1: tiny uniform
# --------------------------------------------------------------------------
def g1_tiny_uniform(M: int = 2048, K: int = 2048, N: int = 32, mean_len: float = 8.0,
                    seed: int = SEED_BASE + 1, dtype: int = SD_F32) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    lengths = np.clip(rng.poisson(mean_len, size=M), 0, K).astype(np.int64)
    rowptr = _rowptr_from_lengths(lengths)
    colind = distinct_sorted_columns(rng, lengths, K)
    vals = _uniform_pm1_f32(rng, colind.size)
    B = _normal_f32(rng, (K, N))
    w = Workload("tiny_uniform", M, K, N, rowptr, colind, vals, B, None, 1.0, 0.0, SD_F32,
                 {"generator": "G1", "seed": seed})
    return _maybe_bf16(w, dtype)


# --------------------------------------------------------------------------
# config 2: 5-point Laplacian on an n x n grid
# --------------------------------------------------------------------------
def g2_stencil(n: int = 1024, N: int = 64, seed: int = SEED_BASE + 2,
               alpha: float = 1.0, beta: float = 0.5, dtype: int = SD_F32) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    M = n * n
    idx = np.arange(M, dtype=np.int64)
    x = idx % n
    y = idx // n
    # candidate neighbours in ascending column order: i-n, i-1, i, i+1, i+n
    cand_col = np.stack([idx - n, idx - 1, idx, idx + 1, idx + n], axis=1)
    cand_ok = np.stack([y > 0, x > 0, np.ones(M, bool), x < n - 1, y < n - 1], axis=1)
    cand_val = np.broadcast_to(np.array([-1, -1, 4, -1, -1], dtype=np.float32), (M, 5))
    lengths = cand_ok.sum(axis=1)
    rowptr = _rowptr_from_lengths(lengths)
    colind = cand_col[cand_ok].astype(np.int32)
    vals = np.ascontiguousarray(cand_val[cand_ok], dtype=np.float32)
    B = _normal_f32(rng, (M, N))
    C0 = _normal_f32(rng, (M, N)) if beta != 0.0 else None
    w = Workload("stencil", M, M, N, rowptr, colind, vals, B, C0, alpha, beta, SD_F32,
                 {"generator": "G2", "seed": seed, "grid": n})
    return _maybe_bf16(w, dtype)


# --------------------------------------------------------------------------
# config 3: GCN aggregation on an R-MAT graph
# --------------------------------------------------------------------------
def g3_gcn_rmat(scale: int = 20, edge_factor: int = 16, N: int = 128,
                a: float = 0.57, b: float = 0.19, c: float = 0.19,
                seed: int = SEED_BASE + 3, dtype: int = SD_F32) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    n = 1 << scale
    ne = edge_factor * n
    src = np.zeros(ne, dtype=np.int64)
    dst = np.zeros(ne, dtype=np.int64)
    for _level in range(scale):
        u = rng.random(size=ne)
        sbit = u >= (a + b)                               # quadrants c, d: lower half
        dbit = ((u >= a) & (u < a + b)) | (u >= a + b + c)  # quadrants b, d: right half
        src = (src << 1) | sbit
        dst = (dst << 1) | dbit
    keep = src != dst                                     # generated self-loops dropped
    src, dst = src[keep], dst[keep]
    diag = np.arange(n, dtype=np.int64)
    key = np.concatenate([src * n + dst, dst * n + src, diag * n + diag])
    del src, dst
    key.sort()                                            # symmetrised, + I ...
    key = key[np.concatenate([[True], key[1:] != key[:-1]])]   # ... deduplicated
    rows = key // n
    colind = (key % n).astype(np.int32)
    deg = np.bincount(rows, minlength=n).astype(np.int64)  # row count of A + I
    rowptr = _rowptr_from_lengths(deg)
    # values of D^-1/2 (A+I) D^-1/2: an input recipe (double, rounded once to fp32)
    dinv = 1.0 / np.sqrt(deg.astype(np.float64))
    vals = (dinv[rows] * dinv[colind]).astype(np.float32)
    B = _normal_f32(rng, (n, N))
    w = Workload("gcn_rmat", n, n, N, rowptr, colind, vals, B, None, 1.0, 0.0, SD_F32,
                 {"generator": "G3", "seed": seed, "scale": scale, "edge_factor": edge_factor,
                  "degree": deg})
    return _maybe_bf16(w, dtype)


# --------------------------------------------------------------------------
# config 4: fully dense 16x16 blocks at random block positions
# --------------------------------------------------------------------------
def g4_block(Mb: int = 4096, Kb: int = 4096, N: int = 256, nblocks: int | None = None,
             frac: float = 0.002, seed: int = SEED_BASE + 4, dtype: int = SD_F32) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    if nblocks is None:
        nblocks = int(round(frac * Mb * Kb))
    pos = np.sort(rng.choice(Mb * Kb, size=nblocks, replace=False).astype(np.int64))
    bi = pos // Kb
    bj = pos % Kb
    blockvals = _normal_f32(rng, (nblocks, 16, 16))       # [block][r][c]
    per_brow = np.bincount(bi, minlength=Mb).astype(np.int64)
    browptr = np.zeros(Mb + 1, dtype=np.int64)
    np.cumsum(per_brow, out=browptr[1:])
    M, K = 16 * Mb, 16 * Kb
    lengths = np.repeat(per_brow * 16, 16)
    rowptr = _rowptr_from_lengths(lengths)
    # CSR order: row 16*I+r holds, for its blocks in ascending J, columns 16J..16J+15
    colind = np.empty(nblocks * 256, dtype=np.int32)
    vals = np.empty(nblocks * 256, dtype=np.float32)
    blk_of = np.arange(nblocks, dtype=np.int64)
    rank_in_brow = blk_of - browptr[bi]                   # position of the block in its block-row
    c16 = np.arange(16, dtype=np.int64)
    for r in range(16):
        base = rowptr[16 * bi + r].astype(np.int64) + rank_in_brow * 16   # [nblocks]
        dstidx = (base[:, None] + c16[None, :]).ravel()
        colind[dstidx] = (bj[:, None] * 16 + c16[None, :]).ravel().astype(np.int32)
        vals[dstidx] = blockvals[:, r, :].ravel()
    B = _normal_f32(rng, (K, N))
    w = Workload("block16", M, K, N, rowptr, colind, vals, B, None, 1.0, 0.0, SD_F32,
                 {"generator": "G4", "seed": seed, "nblocks": nblocks, "block_row": bi,
                  "block_col": bj, "block_vals": blockvals})
    return _maybe_bf16(w, dtype)


def thin_blocks(w: Workload, fill: float, seed: int = SEED_BASE + 44) -> Workload:
    """The block workload with every stored entry kept with probability `fill` (partly filled 16x16 blocks; the
    occupied blocks stay the same unless a block loses all of its entries).  Values and B are those of `w`."""
    if fill >= 1.0:
        return w
    rng = np.random.Generator(np.random.PCG64(seed))
    keep = rng.random(w.nnz) < fill
    rows = np.repeat(np.arange(w.M, dtype=np.int64), np.diff(w.rowptr))
    lengths = np.bincount(rows[keep], minlength=w.M).astype(np.int64)
    return Workload(f"{w.name}_fill{fill:g}", w.M, w.K, w.N, _rowptr_from_lengths(lengths), w.colind[keep], w.vals[keep],
                    w.B, None, w.alpha, w.beta, w.dtype, {"generator": "G4 thinned", "fill": fill, "seed": seed})


# --------------------------------------------------------------------------
# config 5: skewed rank-size row lengths
# --------------------------------------------------------------------------
def g5_skewed(M: int = 4_194_304, N: int = 32, scale_c: float = 2.4e7, exponent: float = 1.2,
              cap: int = 200_000, seed: int = SEED_BASE + 5, dtype: int = SD_F32) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    K = M
    rank = np.arange(1, M + 1, dtype=np.float64)
    lengths_by_rank = np.clip(np.floor(scale_c * rank ** (-exponent)), 1, min(cap, K)).astype(np.int64)
    perm = rng.permutation(M)
    lengths = np.empty(M, dtype=np.int64)
    lengths[perm] = lengths_by_rank
    rowptr = _rowptr_from_lengths(lengths)
    colind = distinct_sorted_columns(rng, lengths, K)
    vals = _uniform_pm1_f32(rng, colind.size)
    B = _normal_f32(rng, (K, N))
    w = Workload("skewed", M, K, N, rowptr, colind, vals, B, None, 1.0, 0.0, SD_F32,
                 {"generator": "G5", "seed": seed, "cap": cap, "scale_c": scale_c})
    return _maybe_bf16(w, dtype)


# --------------------------------------------------------------------------
# generic random CSR for edge-case tests
# --------------------------------------------------------------------------
def random_csr(M: int, K: int, N: int, lengths, seed: int, dtype: int = SD_F32,
               alpha: float = 1.0, beta: float = 0.0, positive: bool = False) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    lengths = np.asarray(lengths, dtype=np.int64)
    rowptr = _rowptr_from_lengths(lengths)
    colind = distinct_sorted_columns(rng, lengths, K)
    vals = _uniform_pm1_f32(rng, colind.size)
    B = _normal_f32(rng, (K, N))
    if positive:
        vals = np.abs(vals) + np.float32(0.01)
        B = np.abs(B) + np.float32(0.01)
    C0 = _normal_f32(rng, (M, N)) if beta != 0.0 else None
    w = Workload("random_csr", M, K, N, rowptr, colind, vals, B, C0, alpha, beta, SD_F32,
                 {"seed": seed})
    return _maybe_bf16(w, dtype)


def _maybe_bf16(w: Workload, dtype: int) -> Workload:
    if dtype == SD_F32:
        return w
    w.vals = f32_to_bf16_bits(w.vals)
    w.B = f32_to_bf16_bits(w.B).reshape(w.B.shape)
    w.dtype = SD_BF16
    return w


# Full-size configurations, by index in the benchmark list (0-based).
def config(i: int, dtype: int = SD_F32, **kw) -> Workload:
    if i == 0:
        return g1_tiny_uniform(dtype=dtype, **kw)
    if i == 1:
        return g2_stencil(dtype=dtype, **kw)
    if i == 2:
        return g3_gcn_rmat(dtype=dtype, **kw)
    if i == 3:
        return g4_block(dtype=dtype, **kw)
    if i == 4:
        return g5_skewed(dtype=dtype, **kw)
    raise ValueError("config index 0..4")
