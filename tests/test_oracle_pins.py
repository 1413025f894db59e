"""Pins of the CPU oracle against things other than itself: brute force on tiny
inputs, closed forms, invariants, hand-worked cases, and the figures the paper
prints.  CPU only."""
import math
import os

import numpy as np
import pytest

import oracle
import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    d = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            d[k] = float(v)
    return d


def densify(w):
    A = np.zeros((w.M, w.K), dtype=np.float64)
    v = w.vals if w.dtype == W.SD_F32 else W.bf16_bits_to_f32(w.vals)
    for i in range(w.M):
        for p in range(w.rowptr[i], w.rowptr[i + 1]):
            A[i, w.colind[p]] += float(v[p])
    return A


def dense_f64(w, X):
    return (X if w.dtype == W.SD_F32 else W.bf16_bits_to_f32(X)).astype(np.float64)


def brute_gemm(A, B):
    """Dense triple loop in Python floats (IEEE double)."""
    M, K = A.shape
    N = B.shape[1]
    out = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            s = 0.0
            for k in range(K):
                if A[i, k] != 0.0:
                    s += float(A[i, k]) * float(B[k, j])
            out[i][j] = s
    return np.array(out, dtype=np.float64).reshape(M, N)


# ------------------------------------------------------------------ O1
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
@pytest.mark.parametrize("N", [1, 3, 4, 32])
def test_o1_brute_force_tiny(dtype, N):
    rng = np.random.default_rng(7 + N)
    M, K = 37, 29
    lengths = rng.integers(0, 9, size=M)
    lengths[5] = 0
    lengths[11] = K
    for alpha in (0.0, 1.0, -0.5):
        for beta in (0.0, 1.0, -0.5):
            w = W.random_csr(M, K, N, lengths, seed=100 + N, dtype=dtype, alpha=alpha, beta=beta)
            # ld > N: pad B and C with sentinel columns
            Bp = np.full((K, N + 3), 7, dtype=w.B.dtype)
            Bp[:, :N] = w.B
            Cin = None
            if beta != 0.0:
                Cin = np.full((M, N + 2), np.float32(99.0))
                Cin[:, :N] = w.C0
            Cref, S = oracle.spmm(w.rowptr, w.colind, w.vals, Bp[:, :N], N,
                                  Cin[:, :N] if Cin is not None else None, alpha, beta)
            A = densify(w)
            Bd = dense_f64(w, w.B)
            want = np.float64(np.float32(alpha)) * brute_gemm(A, Bd)
            if beta != 0.0:
                want = want + np.float64(np.float32(beta)) * w.C0.astype(np.float64)
            np.testing.assert_allclose(Cref, want, rtol=1e-14, atol=1e-300)
            np.testing.assert_allclose(S, brute_gemm(np.abs(A), np.abs(Bd)), rtol=1e-14, atol=1e-300)


def test_o1_hand_worked_3x3():
    # A = [[2,0,1],[0,0,0],[0,-3,4]],  B = [[1,2],[3,4],[5,6]]
    rowptr = np.array([0, 2, 2, 4], np.int32)
    colind = np.array([0, 2, 1, 2], np.int32)
    vals = np.array([2, 1, -3, 4], np.float32)
    B = np.array([[1, 2], [3, 4], [5, 6]], np.float32)
    Cin = np.array([[10, 20], [30, 40], [50, 60]], np.float32)
    # A*B = [[2*1+1*5, 2*2+1*6], [0,0], [-9+20, -12+24]] = [[7,10],[0,0],[11,12]]
    Cref, S = oracle.spmm(rowptr, colind, vals, B, 2)
    assert Cref.tolist() == [[7.0, 10.0], [0.0, 0.0], [11.0, 12.0]]
    assert S.tolist() == [[7.0, 10.0], [0.0, 0.0], [29.0, 36.0]]
    # alpha = 2, beta = -1:  2*AB - Cin
    Cref, _ = oracle.spmm(rowptr, colind, vals, B, 2, Cin, 2.0, -1.0)
    assert Cref.tolist() == [[4.0, 0.0], [-30.0, -40.0], [-28.0, -36.0]]
    # N = 1 is SpMV with x = first column
    Cref, _ = oracle.spmm(rowptr, colind, vals, np.ascontiguousarray(B[:, :1]), 1)
    assert Cref.ravel().tolist() == [7.0, 0.0, 11.0]


def test_o1_hand_worked_4x5():
    # A (4x5): row0: (0,1)=1 (0,4)=2 ; row1: (1,0)=-1 ; row2: empty ; row3: (3,1)=0.5 (3,2)=0.25 (3,3)=-2
    rowptr = np.array([0, 2, 3, 3, 6], np.int32)
    colind = np.array([1, 4, 0, 1, 2, 3], np.int32)
    vals = np.array([1, 2, -1, 0.5, 0.25, -2], np.float32)
    B = np.array([[1, 0, 2], [0, 1, 4], [8, 8, 8], [1, 2, 3], [10, 20, 30]], np.float32)
    # row0 = B[1] + 2 B[4] = [20, 41, 64]; row1 = -B[0] = [-1, 0, -2]; row2 = 0
    # row3 = .5 B[1] + .25 B[2] - 2 B[3] = [0+2-2, .5+2-4, 2+2-6] = [0, -1.5, -2]
    Cref, S = oracle.spmm(rowptr, colind, vals, B, 3)
    assert Cref.tolist() == [[20.0, 41.0, 64.0], [-1.0, 0.0, -2.0], [0.0, 0.0, 0.0], [0.0, -1.5, -2.0]]
    assert S[3].tolist() == [4.0, 6.5, 10.0]
    # beta == 0 must not read C: poison it
    poison = np.full((4, 3), np.nan, np.float32)
    Cref2, _ = oracle.spmm(rowptr, colind, vals, B, 3, poison, 1.0, 0.0)
    assert np.array_equal(Cref, Cref2)


def test_o1_identity_and_permutation():
    rng = np.random.default_rng(3)
    n, N = 50, 5
    B = rng.standard_normal((n, N)).astype(np.float32)
    Cin = rng.standard_normal((n, N)).astype(np.float32)
    rowptr = np.arange(n + 1, dtype=np.int32)
    ones = np.ones(n, np.float32)
    ident = np.arange(n, dtype=np.int32)
    Cref, _ = oracle.spmm(rowptr, ident, ones, B, N, Cin, 0.75, -2.0)
    want = np.float64(0.75) * B.astype(np.float64) + np.float64(-2.0) * Cin.astype(np.float64)
    assert np.array_equal(Cref, want)
    perm = rng.permutation(n).astype(np.int32)
    Cref, _ = oracle.spmm(rowptr, perm, ones, B, N)
    assert np.array_equal(Cref, B[perm].astype(np.float64))


def test_o1_row_sums_col_sums_linearity():
    w = W.g1_tiny_uniform(M=300, K=257, N=8, seed=11)
    v64 = w.vals.astype(np.float64)
    # B = ones  =>  every column of C is the row sum of A
    ones = np.ones((w.K, 4), np.float32)
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, ones, 4)
    rows = np.repeat(np.arange(w.M), np.diff(w.rowptr))
    rs = np.zeros(w.M)
    np.add.at(rs, rows, v64)
    np.testing.assert_allclose(Cref, np.repeat(rs[:, None], 4, 1), rtol=1e-13, atol=1e-13)
    # 1^T (A B) = (1^T A) B
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, w.B, w.N)
    cs = np.zeros(w.K)
    np.add.at(cs, w.colind, v64)
    np.testing.assert_allclose(Cref.sum(0), cs @ w.B.astype(np.float64), rtol=1e-11, atol=1e-11)
    # width consistency: columns are independent
    left, _ = oracle.spmm(w.rowptr, w.colind, w.vals, np.ascontiguousarray(w.B[:, :3]), 3)
    one, _ = oracle.spmm(w.rowptr, w.colind, w.vals, np.ascontiguousarray(w.B[:, :1]), 1)
    assert np.array_equal(left, Cref[:, :3])
    assert np.array_equal(one, Cref[:, :1])
    # strided view of a wider B gives the same answer
    viewed, _ = oracle.spmm(w.rowptr, w.colind, w.vals, w.B[:, :5], 5)
    assert np.array_equal(viewed, Cref[:, :5])
    # spmm_rows returns the same rows
    pick = np.array([0, 7, 299, 150], np.int64)
    sub, _ = oracle.spmm_rows(pick, w.rowptr, w.colind, w.vals, w.B, w.N)
    assert np.array_equal(sub, Cref[pick])


def test_o1_check_flags_errors():
    w = W.g1_tiny_uniform(M=64, K=64, N=8, seed=5)
    Cref, S = oracle.spmm(w.rowptr, w.colind, w.vals, w.B, w.N)
    good = Cref.astype(np.float32)
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, good)
    assert r["ok"] and r["max_ratio"] < 1.0
    bad = good.copy()
    i = int(np.argmax(np.diff(w.rowptr) > 0))
    bad[i, 3] += np.float32(1e-3) * max(1.0, abs(bad[i, 3]))
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, bad)
    assert not r["ok"] and r["violations"] == 1 and r["worst"] == (i, 3)
    bad = good.copy()
    bad[1, 1] = np.nan
    assert oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, bad)["nonfinite"] == 1


# ------------------------------------------------------------------ workload closed forms
def test_stencil_closed_forms_small_and_eigenmodes():
    n = 48
    w = W.g2_stencil(n=n, N=4, beta=0.0)
    assert w.nnz == 5 * n * n - 4 * n
    r = np.diff(w.rowptr)
    assert (r == 3).sum() == 4 and (r == 4).sum() == 4 * (n - 2) and (r == 5).sum() == (n - 2) ** 2
    # A*1: 0 interior, 1 edge, 2 corner; total 4n
    ones = np.ones((w.K, 1), np.float32)
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, ones, 1)
    assert Cref.sum() == 4 * n
    assert sorted(np.unique(Cref).tolist()) == [0.0, 1.0, 2.0]
    # discrete sine modes are eigenvectors (textbook): lambda = 4 - 2cos(p pi/(n+1)) - 2cos(q pi/(n+1))
    idx = np.arange(n * n)
    x, y = idx % n, idx // n
    modes = [(1, 1), (2, 5), (7, 3), (n, n)]
    B = np.stack([np.sin(p * math.pi * (x + 1) / (n + 1)) * np.sin(q * math.pi * (y + 1) / (n + 1))
                  for p, q in modes], axis=1).astype(np.float32)
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, B, 4)
    lam = np.array([4 - 2 * math.cos(p * math.pi / (n + 1)) - 2 * math.cos(q * math.pi / (n + 1))
                    for p, q in modes])
    np.testing.assert_allclose(Cref, B.astype(np.float64) * lam[None, :], atol=2e-6)


def test_stencil_full_size_counts():
    n = 1024
    w = W.g2_stencil(n=n, N=1, beta=0.0)
    assert w.nnz == 5_238_784 == 5 * n * n - 4 * n
    r = np.diff(w.rowptr)
    assert (r == 3).sum() == 4 and (r == 4).sum() == 4088 and (r == 5).sum() == 1_044_484
    info = oracle.summary(w.rowptr, w.colind, w.M, w.K, 64)
    # occupied 16x16 blocks: diagonal + left/right neighbours + up/down neighbours
    nb = n // 16
    assert info.nnzb16 == n * nb + 2 * (nb - 1) * n + 2 * (n - 1) * nb
    assert info.diag == n * n and info.unsorted_rows == 0 and info.max_r == 5
    assert info.max_span == 2 * n + 1


def test_gcn_normalised_adjacency_invariants():
    w = W.g3_gcn_rmat(scale=10, edge_factor=8, N=2, seed=99)
    d = w.meta["degree"].astype(np.float64)
    assert np.array_equal(np.diff(w.rowptr), w.meta["degree"])
    sq = np.sqrt(d)
    B = np.stack([sq, -2 * sq], 1).astype(np.float32)
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, B, 2)
    # A_hat sqrt(d) = sqrt(d): eigenvalue 1 (up to fp32 rounding of the inputs)
    np.testing.assert_allclose(Cref, B.astype(np.float64), rtol=2e-6)
    # symmetry: x^T (A y) = y^T (A x)
    rng = np.random.default_rng(0)
    X = rng.standard_normal((w.M, 2)).astype(np.float32)
    AX, _ = oracle.spmm(w.rowptr, w.colind, w.vals, X, 2)
    x, y = X[:, 0].astype(np.float64), X[:, 1].astype(np.float64)
    assert abs(x @ AX[:, 1] - y @ AX[:, 0]) < 1e-9 * (np.abs(x) @ np.abs(AX[:, 1]) + 1)


@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_block_workload_strip_gemm_and_bsr(dtype):
    w = W.g4_block(Mb=24, Kb=40, N=8, nblocks=60, seed=21, dtype=dtype)
    bi, bj, bv = w.meta["block_row"], w.meta["block_col"], w.meta["block_vals"]
    if dtype == W.SD_BF16:
        bv = W.bf16_bits_to_f32(W.f32_to_bf16_bits(bv).reshape(bv.shape))
    Bd = dense_f64(w, w.B)
    Cref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, w.B, w.N)
    for I in range(24):
        want = np.zeros((16, w.N))
        for b in np.flatnonzero(bi == I):
            want += bv[b].astype(np.float64) @ Bd[16 * bj[b]:16 * bj[b] + 16]
        np.testing.assert_allclose(Cref[16 * I:16 * I + 16], want, rtol=1e-12, atol=1e-12)
    browptr, bcol, bval = oracle.bsr16(w.rowptr, w.colind, w.vals, w.M, w.K)
    assert browptr[-1] == 60
    assert np.array_equal(np.diff(browptr), np.bincount(bi, minlength=24))
    assert np.array_equal(bcol, bj.astype(np.int32))
    gen_vals = w.meta["block_vals"]
    gen_vals = W.f32_to_bf16_bits(gen_vals).reshape(gen_vals.shape) if dtype == W.SD_BF16 else gen_vals
    assert np.array_equal(bval, gen_vals)
    info = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    assert info.nnzb16 == 60 and oracle.rho_bsr16(info) == 1.0
    assert info.blk_hist[8] == 60 and info.nnz_dense_blocks == w.nnz
    assert oracle.decide(info) != oracle.BSR_TC     # 8 columns: not a width of the tensor-core kernel
    info.N = 64
    assert oracle.decide(info) == oracle.BSR_TC


# ------------------------------------------------------------------ O2
def test_o2_against_python_sets_and_round_trip():
    rng = np.random.default_rng(17)
    M, K = 70, 45       # neither a multiple of 16
    lengths = rng.integers(0, 12, size=M)
    w = W.random_csr(M, K, 1, lengths, seed=33)
    browptr, bcol, bval = oracle.bsr16(w.rowptr, w.colind, w.vals, M, K)
    blocks = {}
    for i in range(M):
        for p in range(w.rowptr[i], w.rowptr[i + 1]):
            blocks.setdefault((i >> 4, w.colind[p] >> 4), {})[(i & 15, w.colind[p] & 15)] = w.vals[p]
    keys = sorted(blocks)
    assert len(keys) == browptr[-1]
    k = 0
    for I in range((M + 15) // 16):
        mine = [key for key in keys if key[0] == I]
        assert browptr[I + 1] - browptr[I] == len(mine)
        for (_, J) in mine:
            assert bcol[k] == J
            dense = np.zeros((16, 16), np.float32)
            for (r, c), v in blocks[(I, J)].items():
                dense[r, c] = v
            assert np.array_equal(bval[k], dense)
            k += 1
    # round trip BSR -> CSR through the structure mask returns the input
    back = []
    for I in range((M + 15) // 16):
        for r in range(16):
            i = 16 * I + r
            if i >= M:
                break
            for b in range(browptr[I], browptr[I + 1]):
                for c in range(16):
                    if (r, c) in blocks[(I, int(bcol[b]))]:
                        back.append((i, 16 * int(bcol[b]) + c, bval[b, r, c]))
    got_rows = np.repeat(np.arange(M), np.diff(w.rowptr))
    assert [(int(a), int(b), float(c)) for a, b, c in back] == \
        [(int(a), int(b), float(c)) for a, b, c in zip(got_rows, w.colind, w.vals)]


def test_o2_stored_zero_counts_as_structure():
    rowptr = np.array([0, 1, 2], np.int32)
    colind = np.array([3, 40], np.int32)
    vals = np.array([0.0, 5.0], np.float32)
    browptr, bcol, bval = oracle.bsr16(rowptr, colind, vals, 2, 48)
    assert browptr.tolist() == [0, 2] and bcol.tolist() == [0, 2]
    assert bval[1, 1, 8] == 5.0 and not bval[0].any()


# ------------------------------------------------------------------ O3
def test_o3_against_brute_force():
    rng = np.random.default_rng(5)
    M, K = 90, 300
    lengths = rng.integers(0, 40, size=M)
    lengths[3] = 280
    lengths[4] = 0
    w = W.random_csr(M, K, 1, lengths, seed=44)
    info = oracle.summary(w.rowptr, w.colind, M, K, 7)
    assert (info.M, info.K, info.N, info.nnz) == (M, K, 7, w.nnz)
    hist = [0] * 32
    for r in lengths:
        hist[0 if r == 0 else int(math.floor(math.log2(r))) + 1] += 1
    assert list(info.row_hist) == hist
    assert info.sum_r2 == int((lengths.astype(np.int64) ** 2).sum())
    assert info.max_r == 280 and info.empty_rows == int((lengths == 0).sum())
    assert info.long_rows == 1 and info.nnz_long_rows == 280
    span = gap = diag = 0
    mspan = 0
    blocks = {}
    for i in range(M):
        cols = w.colind[w.rowptr[i]:w.rowptr[i + 1]]
        if cols.size:
            s = int(cols.max() - cols.min() + 1)
            span += s
            mspan = max(mspan, s)
            gap += int(np.diff(cols).sum())      # sum of gaps between sorted consecutive indices
            diag += int((cols == i).sum())
        for c in cols:
            blocks[(i >> 4, c >> 4)] = blocks.get((i >> 4, c >> 4), 0) + 1
    assert (info.sum_span, info.max_span, info.sum_gap, info.diag) == (span, mspan, gap, diag)
    assert info.unsorted_rows == 0
    assert info.nnzb16 == len(blocks)
    bh = [0] * 9
    for c in blocks.values():
        bh[min(int(math.floor(math.log2(c))), 8)] += 1
    assert list(info.blk_hist) == bh
    assert info.nnz_dense_blocks == sum(c for c in blocks.values() if c >= 128)


def test_o3_unsorted_and_duplicate_rows_are_counted():
    rowptr = np.array([0, 3, 5, 7], np.int32)
    colind = np.array([0, 2, 1, 4, 4, 1, 9], np.int32)   # row0 unsorted, row1 duplicate, row2 fine
    info = oracle.summary(rowptr, colind, 3, 10, 1)
    assert info.unsorted_rows == 2
    assert oracle.decide(info) != oracle.BSR_TC


def test_paper_worked_example_sec3_3():
    g = read_golden("sec3_3_shen_e40r0100.txt")
    info = oracle.Info()
    info.M = info.K = int(g["m"])
    info.nnz = int(g["nnz"])
    info.max_r = int(g["max_row_length"])
    info.nnzb16 = int(g["nnzb16"])
    assert round(oracle.rho_ell(info), 1) == g["rho_ell_approx"]
    assert round(oracle.rho_bsr16(info), 1) == g["rho_bsr16_approx"]
    assert round(info.nnz / info.nnzb16, 1) == g["nnz_per_occupied_tile_approx"]
    assert round(100 * oracle.tile_coverage16(info), 1) == g["occupied_tile_fraction_percent_approx"]
    assert oracle.csr_bytes(info, 4) == int(g["csr_bytes_fp32_int32"])


def test_paper_planning_record_nemeth26():
    g = read_golden("appE_nemeth26_working_set.txt")
    info = oracle.Info()
    info.M = info.K = int(g["rows"])
    info.N = int(g["dense_width"])
    info.nnz = int(g["rows"] * g["mean_row_length"])
    _, m_t = oracle.working_set_bytes(oracle.csr_bytes(info, 4), info, 4)
    assert abs(m_t / 2**20 - g["csr_working_set_mib"]) < 0.01


# ------------------------------------------------------------------ O4
def test_o4_merge_coords_match_closed_form():
    rng = np.random.default_rng(2)
    for trial in range(6):
        S = int(rng.integers(1, 200))
        lengths = rng.integers(0, 6, size=S)
        if trial % 2:
            lengths[rng.integers(0, S)] = 500
        ptr = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        for items in (1, 7, 64):
            got = oracle.merge_coords(ptr, items)
            total = S + int(ptr[-1])
            ntiles = (total + items - 1) // items
            assert got.size == ntiles + 1
            # end of segment r is item number ptr[r+1] + r of the merged list
            pos = ptr[1:].astype(np.int64) + np.arange(S)
            want = [int(np.searchsorted(pos, min(t * items, total), side="left")) for t in range(ntiles + 1)]
            assert got.tolist() == want
            assert got[0] == 0 and got[-1] == S


def test_o4_block_rule_thresholds_by_width_and_value_type():
    # the block form is taken while 256 * nnzb <= rho_max * nnz; rho_max by dense width and value type
    # (integer arithmetic: the boundary itself is inside)
    table = {(oracle.F32, 64): (9, 8), (oracle.F32, 96): (9, 8), (oracle.F32, 128): (2, 1), (oracle.F32, 256): (3, 1), (oracle.F32, 1024): (3, 1),
             (oracle.BF16, 64): (3, 1), (oracle.BF16, 128): (7, 1), (oracle.BF16, 192): (7, 1), (oracle.BF16, 256): (10, 1)}
    w = W.g4_block(Mb=16, Kb=16, N=4, nblocks=30)
    base = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    for (dt, N), (num, den) in table.items():
        nnzb = 1000
        edge = (den * 256 * nnzb + num - 1) // num          # smallest nnz that still qualifies
        for nnz, want in ((edge, True), (edge - 1, False)):
            info = oracle.Info.from_buffer_copy(base)
            info.N, info.nnzb16, info.nnz = N, nnzb, nnz
            info.sum_r2 = 0          # keep the row-length part of the rule out of the picture
            info.max_r = 1
            assert (oracle.decide(info, dt) == oracle.BSR_TC) == want, (dt, N, nnz)
    # widths that are not whole 128-byte column groups never take the block form, however dense the blocks
    for dt, N in ((oracle.F32, 1), (oracle.F32, 4), (oracle.F32, 16), (oracle.F32, 32), (oracle.F32, 48), (oracle.F32, 100),
                  (oracle.BF16, 32), (oracle.BF16, 96), (oracle.BF16, 255)):
        info = oracle.Info.from_buffer_copy(base)
        info.N = N
        assert info.nnz == 256 * info.nnzb16 and oracle.decide(info, dt) != oracle.BSR_TC, (dt, N)


def test_o4_uniform_rows_stay_row_split_at_every_width_and_length():
    for L, N in ((5, 1), (31, 1), (32, 1), (32, 4), (200, 1), (200, 8), (8, 2)):
        M = 64
        rowptr = np.arange(0, M * L + 1, L, dtype=np.int32)
        colind = np.tile(np.arange(L, dtype=np.int32) * 3, M)    # uniform rows: no skew, blocks sparse
        info = oracle.summary(rowptr, colind, M, 3 * L + 8, N)
        assert oracle.decide(info) == oracle.ROWSPLIT, (L, N)


def test_o4_family_rule_on_the_five_shapes():
    w = W.g1_tiny_uniform()
    assert oracle.decide(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)) == oracle.ROWSPLIT
    w = W.g2_stencil(n=64, N=4)
    assert oracle.decide(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)) == oracle.ROWSPLIT
    w = W.g3_gcn_rmat(scale=12, N=4)
    assert oracle.decide(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)) == oracle.MERGE
    w = W.g4_block(Mb=32, Kb=32, N=64, nblocks=40)
    assert oracle.decide(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)) == oracle.BSR_TC
    w = W.g5_skewed(M=1 << 14, N=4, scale_c=2.4e7 / 256, cap=800)
    assert oracle.decide(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)) == oracle.MERGE


def test_skewed_generator_counts():
    # lengths are a deterministic rank-size law; only their assignment to rows is random
    M = 1 << 12
    w = W.g5_skewed(M=M, N=1, scale_c=5000.0, cap=300)
    r = np.sort(np.diff(w.rowptr))[::-1]
    rank = np.arange(1, M + 1, dtype=np.float64)
    want = np.clip(np.floor(5000.0 * rank ** -1.2), 1, 300).astype(np.int64)
    assert np.array_equal(r, want)
    for i in range(0, M, 97):
        cols = w.colind[w.rowptr[i]:w.rowptr[i + 1]]
        assert np.all(np.diff(cols) > 0) and cols.min() >= 0 and cols.max() < M


def test_o4_window_segments_against_python_sets():
    rng = np.random.default_rng(9)
    M, K = 60, 101
    lengths = rng.integers(0, 9, size=M)
    lengths[7] = 0
    lengths[20] = 90
    wl = W.random_csr(M, K, 1, lengths, seed=3)
    short_len = 5
    seg_ptr, seg_row, perm, bounds = oracle.window_segments(wl.rowptr, wl.colind, M, K, 4, short_len)
    wcols = -(-K // 4)
    # brute force: dictionary (window, row) -> positions
    groups = {}
    for i in range(M):
        for p in range(wl.rowptr[i], wl.rowptr[i + 1]):
            groups.setdefault((wl.colind[p] // wcols, i), []).append(p)
    empties = [i for i in range(M) if lengths[i] == 0]
    # expected order: by (window, class), long first; inside window 0's short class the empty
    # rows come before the other rows; rows ascending inside a class
    want = []
    for win in range(4):
        runs = sorted((row, ps) for (w2, row), ps in groups.items() if w2 == win)
        want += [(win, row, ps) for row, ps in runs if len(ps) > short_len]
        if win == 0:
            want += [(0, row, []) for row in empties]
        want += [(win, row, ps) for row, ps in runs if 2 <= len(ps) <= short_len]
        want += [(win, row, ps) for row, ps in runs if len(ps) == 1]
    assert len(seg_row) == len(want) == bounds[-1]
    q = 0
    for s, (win, row, ps) in enumerate(want):
        assert seg_ptr[s] == q
        assert (int(seg_row[s]) & 0x7FFFFFFF) == row
        if ps:
            first_w = wl.colind[wl.rowptr[row]] // wcols
            assert bool(int(seg_row[s]) & 0x80000000) == (first_w != win)
        assert perm[q:q + len(ps)].tolist() == ps
        q += len(ps)
    assert seg_ptr[-1] == q == wl.nnz
    assert sorted(perm.tolist()) == list(range(wl.nnz))
    pos = 0
    for win in range(4):
        nlong = sum(1 for x in want if x[0] == win and len(x[2]) > short_len)
        nsingle = sum(1 for x in want if x[0] == win and len(x[2]) == 1)
        nall = sum(1 for x in want if x[0] == win)
        assert bounds[3 * win] == pos and bounds[3 * win + 1] == pos + nlong
        assert bounds[3 * win + 2] == pos + nall - nsingle
        pos += nall


def test_o4_window_rule():
    info = oracle.Info()
    info.M = info.K = 4_194_304
    info.N = 32
    info.nnz = 59_839_586
    assert oracle.decide_windows(info, oracle.F32, 126 * 2**20) == 8     # 512 MiB of B, 75.6 MiB budget
    info.nnz = 16 * info.M
    assert oracle.decide_windows(info, oracle.F32, 126 * 2**20) == 1     # long rows on average
    info.nnz = 59_839_586
    info.unsorted_rows = 1
    assert oracle.decide_windows(info, oracle.F32, 126 * 2**20) == 1
    info.unsorted_rows = 0
    info.K = 100_000
    assert oracle.decide_windows(info, oracle.F32, 126 * 2**20) == 1     # B fits


def test_o4_class_split_rule_by_dense_width():
    info = oracle.Info()
    info.M = info.K = 1 << 20
    info.nnz = 32 << 20
    for dt, N, want in ((oracle.F32, 8, False), (oracle.F32, 15, False), (oracle.F32, 16, True), (oracle.F32, 24, True),
                        (oracle.F32, 32, True), (oracle.F32, 33, True), (oracle.F32, 64, True), (oracle.F32, 65, False),
                        (oracle.F32, 128, False), (oracle.BF16, 7, False), (oracle.BF16, 8, True), (oracle.BF16, 16, True), (oracle.BF16, 32, True),
                        (oracle.BF16, 33, False), (oracle.BF16, 64, False)):
        info.N = N
        assert oracle.decide_class_split(info, dt) == want, (dt, N)
    info.N = 32
    info.unsorted_rows = 1
    assert not oracle.decide_class_split(info, oracle.F32)      # needs ascending columns
    info.unsorted_rows = 0
    info.nnz = 0
    assert not oracle.decide_class_split(info, oracle.F32)


# ------------------------------------------------------------------ O5
def _features_of(w, value_bytes=4):
    info = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    return info, oracle.features(w.rowptr, w.colind, w.M, w.K, info, value_bytes)


def test_o5_quartiles_are_nearest_rank():
    # hand case: 1..8 -> the 2nd, 4th and 6th smallest
    assert [oracle.quartile(np.arange(8, 0, -1), q) for q in (1, 2, 3)] == [2, 4, 6]
    assert [oracle.quartile([7], q) for q in (1, 2, 3)] == [7, 7, 7]
    assert oracle.quartile([], 2) == 0
    # the library's inverted-CDF percentile is the same definition
    rng = np.random.default_rng(5)
    for n in (2, 3, 4, 5, 7, 100, 1001):
        v = rng.integers(0, 50, n).astype(np.int32)
        for q in (1, 2, 3):
            assert oracle.quartile(v, q) == int(np.percentile(v, 25 * q, method="inverted_cdf")), (n, q)


def test_o5_sell_slots_special_cases_and_hand_example():
    lengths = np.array([3, 1, 0, 5, 2], np.int64)
    rowptr = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    # slices {3,1}, {0,5}, {2}: 2*3 + 2*5 + 1*2
    assert oracle.sell_slots(rowptr, 2) == 18
    assert oracle.sell_slots(rowptr, 1) == lengths.sum()              # no padding with one row per slice
    assert oracle.sell_slots(rowptr, 5) == 5 * 5                      # one slice = ELL
    assert oracle.sell_slots(rowptr, 512) == 5 * 5                    # a short last slice counts its own rows only
    rng = np.random.default_rng(6)
    lengths = rng.poisson(9, 3000)
    rowptr = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    chain = [oracle.sell_slots(rowptr, c) for c in (1, 2, 4, 8, 16, 32, 512, 4096)]
    assert chain[0] == lengths.sum() and chain[-1] == 3000 * lengths.max()
    assert all(a <= b for a, b in zip(chain, chain[1:]))              # merging slices never removes padding
    uniform = np.arange(0, 7 * 1000 + 1, 7, dtype=np.int32)
    assert all(oracle.sell_slots(uniform, c) == 7000 for c in (16, 32, 512))


def test_o5_block_count_brute_force_and_closed_forms():
    rng = np.random.default_rng(7)
    for M, K, dens in ((37, 53, 0.08), (64, 64, 0.3), (100, 9, 0.2)):
        D = rng.random((M, K)) < dens
        rowptr = np.concatenate([[0], np.cumsum(D.sum(1))]).astype(np.int32)
        colind = np.nonzero(D)[1].astype(np.int32)
        assert oracle.block_count(rowptr, colind, 1) == D.sum()
        assert oracle.block_count(rowptr, colind, 1000) == 1
        for b in (4, 8, 16, 5):
            P = np.zeros(((M + b - 1) // b * b, (K + b - 1) // b * b), bool)
            P[:M, :K] = D
            want = int(P.reshape(P.shape[0] // b, b, P.shape[1] // b, b).any(axis=(1, 3)).sum())
            assert oracle.block_count(rowptr, colind, b) == want, (M, K, b)
        info = oracle.summary(rowptr, colind, M, K, 1)
        assert oracle.block_count(rowptr, colind, 16) == info.nnzb16
    # 5-point stencil on an n x n grid, natural ordering, b | n: a block-row is b consecutive points of
    # one grid line: its own block, the left / right neighbour blocks, one block in the line above / below
    for n, b in ((32, 4), (32, 8), (48, 16)):
        w = W.g2_stencil(n=n, N=1)
        nb = n // b
        assert oracle.block_count(w.rowptr, w.colind, b) == n * nb + 2 * n * (nb - 1) + 2 * (n - 1) * nb


def test_o5_column_degrees_are_the_row_lengths_of_the_transpose():
    sp = pytest.importorskip("scipy.sparse")
    w = W.g5_skewed(M=3000, N=1, scale_c=2.4e7 / 1024, cap=400)
    _, f = _features_of(w)
    At = sp.csr_matrix((np.ones(w.nnz, np.float32), w.colind, w.rowptr), shape=(w.M, w.K)).T.tocsr()
    At.sort_indices()
    t = oracle.summary(At.indptr.astype(np.int32), At.indices.astype(np.int32), w.K, w.M, 1)
    assert (f.col_max, f.col_empty, f.sum_d2) == (t.max_r, t.empty_rows, t.sum_r2)
    deg = np.bincount(w.colind, minlength=w.K)
    assert list(f.col_q) == [int(np.percentile(deg, 25 * q, method="inverted_cdf")) for q in (1, 2, 3)]
    lengths = np.diff(w.rowptr)
    assert list(f.row_q) == [int(np.percentile(lengths, 25 * q, method="inverted_cdf")) for q in (1, 2, 3)]


def test_o5_storage_estimates_paper_example_and_hand_case():
    # Sec. 3.3 worked example: m = 17,281, nnz = 553,562, longest row 62 -> CSR 4,497,624 B, rho_ELL ~ 1.9
    g = read_golden("sec3_3_shen_e40r0100.txt")
    m, nnz, mx = int(g["m"]), int(g["nnz"]), int(g["max_row_length"])
    lengths = np.full(m, 32, np.int64)
    lengths[:19] = mx
    assert lengths.sum() == nnz
    w = W.random_csr(m, m, 1, lengths, seed=3)
    _, f = _features_of(w, 4)
    assert f.rep_bytes[0] == int(g["csr_bytes_fp32_int32"])
    assert round(f.ell_slots / nnz, 1) == g["rho_ell_approx"]
    assert f.rep_bytes[1] == 8 * m * mx
    # hand case: 6 x 8, entries (0,0) (0,5) (3,4) (5,7): b = 4 -> blocks (0,0) (0,1) (1,1); b = 8 and 16 -> one block
    rowptr = np.array([0, 2, 2, 2, 3, 3, 4], np.int32)
    colind = np.array([0, 5, 4, 7], np.int32)
    info = oracle.summary(rowptr, colind, 6, 8, 1)
    f = oracle.features(rowptr, colind, 6, 8, info, 2)
    assert list(f.nnzb) == [3, 1, 1]
    assert f.rep_bytes[5] == (2 * 16 + 4) * 3 + 4 * 3      # BSR-4: two block-rows
    assert f.rep_bytes[6] == (2 * 64 + 4) * 1 + 4 * 2
    assert f.rep_bytes[7] == (2 * 256 + 4) * 1 + 4 * 2
    assert f.ell_slots == 12 and list(f.sell_slots) == [12, 12, 12]
    assert f.rep_bytes[2] == 6 * 12 + 4 * 2                # SELL-16: one slice, two offsets
    assert f.rep_bytes[0] == 6 * 4 + 4 * 7


def test_o5_shape_class_on_designed_distributions():
    cls = lambda w: oracle.SHAPE_NAMES[oracle.shape_class(oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N))]
    assert cls(W.g2_stencil(n=64, N=1)) == "uniform"
    assert cls(W.g1_tiny_uniform()) == "moderate"                                   # Poisson(8): CV^2 = 1/8
    assert cls(W.g5_skewed(M=1 << 14, N=1, scale_c=2.4e7 / 256, cap=800)) == "power-law"
    rng = np.random.default_rng(9)
    two = np.where(rng.random(4000) < 0.5, 2, 64)                                   # two populations, 32x apart
    assert cls(W.random_csr(4000, 5000, 1, two, seed=1)) == "bimodal"
    geo = np.minimum(rng.geometric(1 / 9.0, 4000) - 1, 4000)                        # CV^2 = 1 / (1 - p) > 1, no heavy tail
    assert cls(W.random_csr(4000, 5000, 1, geo, seed=2)) == "skewed"


def test_o4_hybrid_schedule_against_python_sets():
    """The hybrid schedule from dictionaries and sorts: heavy rows, their (row, window) pieces cut into runs,
    the window-major walk, and the light rows by falling length."""
    rng = np.random.default_rng(21)
    M, K, Wn, T, CH = 80, 333, 4, 9, 5
    lengths = rng.integers(0, 9, size=M)
    lengths[[3, 40, 41, 79]] = [60, 9, 8, 200]
    lengths[17] = 0
    wl = W.random_csr(M, K, 1, lengths, seed=4)
    heavy, chunk_ptr, ranges, order, light = oracle.hybrid_schedule(wl.rowptr, wl.colind, M, K, Wn, T, CH)
    wcols = -(-K // Wn)
    assert heavy.tolist() == [i for i in range(M) if lengths[i] >= T] and 40 in heavy and 41 not in heavy
    want_ranges, want_win, want_ptr = [], [], []
    for i in heavy:
        want_ptr.append(len(want_ranges))
        pieces = {}
        for p in range(wl.rowptr[i], wl.rowptr[i + 1]):
            pieces.setdefault(int(wl.colind[p]) // wcols, []).append(p)
        for win in sorted(pieces):
            ps = pieces[win]
            assert ps == list(range(ps[0], ps[-1] + 1))           # columns ascend: a piece is a range
            for j in range(0, len(ps), CH):
                want_ranges.append([ps[j], ps[min(j + CH, len(ps)) - 1] + 1])
                want_win.append(win)
    want_ptr.append(len(want_ranges))
    assert ranges.tolist() == want_ranges and chunk_ptr.tolist() == want_ptr
    # every nonzero of a heavy row lies in exactly one chunk, no chunk is longer than CH
    covered = np.concatenate([np.arange(a, b) for a, b in ranges]) if len(ranges) else np.zeros(0, int)
    heavy_nz = np.concatenate([np.arange(wl.rowptr[i], wl.rowptr[i + 1]) for i in heavy])
    assert np.array_equal(np.sort(covered), heavy_nz) and np.all(np.diff(ranges, axis=1) <= CH)
    # the walk: a stable sort of the chunk numbers by window
    assert order.tolist() == sorted(range(len(want_ranges)), key=lambda c: (want_win[c], c))
    assert light.tolist() == sorted((i for i in range(M) if lengths[i] < T), key=lambda i: (-lengths[i], i))
    assert sorted(heavy.tolist() + light.tolist()) == list(range(M))
    # one window: the walk is the numbering itself; a threshold above every row: nothing is heavy
    h1, p1, r1, o1, l1 = oracle.hybrid_schedule(wl.rowptr, wl.colind, M, K, 1, T, CH)
    assert o1.tolist() == list(range(len(r1))) and h1.tolist() == heavy.tolist()
    h2, p2, r2, o2, l2 = oracle.hybrid_schedule(wl.rowptr, wl.colind, M, K, Wn, 1000, CH)
    assert h2.size == 0 and r2.shape[0] == 0 and p2.tolist() == [0] and l2.size == M


def test_o4_hybrid_rule():
    """Hybrid in place of the merge family's schedules: ascending columns; with column windows rows of B of 64 to
    192 bytes (fp32 values) or 128 bytes (bf16 values), without them 5 columns and more up to 384-byte (256-byte) rows
    and at least 256 MiB gathered per call; the family rule applies it on top of the merge decision."""
    info = oracle.Info()
    info.M, info.K, info.nnz, info.unsorted_rows = 1 << 20, 1 << 22, 5 << 20, 0
    for dtype, es in ((oracle.F32, 4), (oracle.BF16, 2)):
        for N in (1, 4, 5, 8, 16, 17, 24, 32, 33, 48, 64, 65, 96, 128, 129, 256):
            info.N = N
            assert oracle.decide_hybrid(info, dtype, 8) == (64 <= N * es <= (192 if es == 4 else 128)), (dtype, N)
            for nnz in (5 << 20, 40 << 20):      # without windows the call must also gather at least 256 MiB
                info.nnz = nnz
                cap = 384 if es == 4 else 256
                assert oracle.decide_hybrid(info, dtype, 1) == (N >= 5 and N * es <= cap and nnz * N * es >= 1 << 28), (dtype, N)
            info.nnz = 5 << 20
    info.N, info.nnz = 64, (1 << 20) - 1             # 256-byte rows: one nonzero short of 256 MiB
    assert not oracle.decide_hybrid(info, oracle.F32, 1)
    info.nnz = 1 << 20
    assert oracle.decide_hybrid(info, oracle.F32, 1)
    info.nnz = 5 << 20
    info.N, info.unsorted_rows = 32, 3
    assert not oracle.decide_hybrid(info, oracle.F32, 8) and not oracle.decide_hybrid(info, oracle.F32, 1)
    # the family rule: a skewed summary whose B exceeds the L2 budget
    info.unsorted_rows, info.max_r, info.nnz_long_rows, info.sum_r2 = 0, 5000, info.nnz, 1 << 40
    info.nnzb16 = info.nnz                                         # one entry per 16x16 block: no block form
    l2 = 126 << 20
    assert oracle.decide(info, oracle.F32) == oracle.MERGE and oracle.decide_windows(info, oracle.F32, l2) == 8
    assert oracle.decide_family(info, oracle.F32, l2) == oracle.HYBRID
    info.N = 128                                                   # 512-byte rows, 32 windows: the windowed class split
    assert oracle.decide_family(info, oracle.F32, l2) == oracle.MERGE
    info.N, info.K = 32, 1 << 18                                   # B fits in L2: no windows, hybrid up to 384-byte rows
    assert oracle.decide_windows(info, oracle.F32, l2) == 1 and oracle.decide_family(info, oracle.F32, l2) == oracle.HYBRID
    info.N = 128
    assert oracle.decide_family(info, oracle.F32, l2) == oracle.MERGE
    info.N = 4                                                     # narrow widths keep the merge family (COO reduction)
    assert oracle.decide_family(info, oracle.F32, l2) == oracle.MERGE
    info.N, info.unsorted_rows = 32, 1
    assert oracle.decide_family(info, oracle.F32, l2) == oracle.MERGE
