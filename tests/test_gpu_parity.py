"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.
Tolerance (fp): |C - Cref| <= rel * (|alpha| sum|a||b| + |beta||Cin|) + 1e-6, rel = 1e-5 for
fp32 values and 1e-2 for bf16 values; integer work (plan summary, BSR, tile table) bit-exact."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2608_05033_b200 as sd
    from util import DeviceWorkload, run_spmm
else:  # collected but skipped
    sd = None

FAMILIES = {"rowsplit": 1, "merge": 2, "bsr": 3}


def check(w, got, c_in=None, alpha=None, beta=None):
    alpha = w.alpha if alpha is None else alpha
    beta = w.beta if beta is None else beta
    cin = c_in if c_in is not None else w.C0
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, cin, alpha, beta)
    assert r["ok"], r
    return r


def shape_lengths(kind, M, K, rng):
    if kind == "uniform":
        return np.clip(rng.poisson(8, M), 0, K)
    if kind == "short":
        return rng.integers(0, 4, M)
    if kind == "skewed":
        r = np.clip((2000.0 * np.arange(1, M + 1) ** -1.2).astype(np.int64), 1, min(K, 3000))
        return rng.permutation(r)
    if kind == "onelong":
        r = np.zeros(M, np.int64)
        r[M // 3] = K
        r[M - 1] = K // 2
        return r
    raise ValueError(kind)


@pytest.mark.parametrize("family", ["rowsplit", "merge"])
@pytest.mark.parametrize("kind", ["uniform", "short", "skewed", "onelong"])
@pytest.mark.parametrize("N", [1, 4, 8, 32, 64, 128, 256, 7, 100])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_forced_family_small(family, kind, N, dtype):
    rng = np.random.default_rng(hash((family, kind, N)) % 2**32)
    M, K = 1237, 3001   # ragged: not multiples of any tile
    w = W.random_csr(M, K, N, shape_lengths(kind, M, K, rng), seed=N * 7 + 1, dtype=dtype, alpha=1.25, beta=-0.5)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=FAMILIES[family], windows=1 if family == "merge" else 0)   # merge: the row-ordered tile kernel
    assert plan.info().family == FAMILIES[family]
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    # run again: bit-identical (no float atomics)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)
    # beta == 0 must not read C: poison it
    poison = np.full((M, N), np.nan, np.float32)
    got3, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got3, beta=0.0)
    plan.close()


@pytest.mark.parametrize("family", ["rowsplit", "merge", "bsr"])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_padding_and_misalignment(family, dtype):
    rng = np.random.default_rng(5)
    M, K, N = 300, 517, 32
    w = W.random_csr(M, K, N, np.clip(rng.poisson(6, M), 0, K), seed=77, dtype=dtype, beta=0.75)
    dw = DeviceWorkload(w)
    for windows in ((1, -1) if family == "merge" else (0,)):   # merge: tile kernel, then the class split
        plan = dw.plan(family=FAMILIES[family], windows=windows)
        for pad_b, pad_c, off in [(3, 5, 0), (4, 8, 0), (0, 0, 1), (1, 2, 3), (8, 4, 4)]:
            got, intact = run_spmm(plan, w, pad_b=pad_b, pad_c=pad_c, offset=off)
            assert intact, (pad_b, pad_c, off)
            check(w, got)
        plan.close()


@pytest.mark.parametrize("family", ["rowsplit", "merge", "bsr"])
def test_degenerate_cases(family):
    fam = FAMILIES[family]
    # alpha == 0: C = beta*C, A and B untouched
    w = W.random_csr(64, 64, 8, np.full(64, 3), seed=3, beta=2.0)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=fam)
    got, _ = run_spmm(plan, w, alpha=0.0)
    assert np.array_equal(got, np.float32(2.0) * w.C0)
    plan.close()
    # no nonzeros at all
    w = W.random_csr(50, 40, 4, np.zeros(50, np.int64), seed=4, beta=0.0)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=fam)
    assert plan.info().nnz == 0
    got, _ = run_spmm(plan, w, c_fill=np.full((50, 4), np.nan, np.float32))
    assert np.array_equal(got, np.zeros((50, 4), np.float32))
    plan.close()
    # M == 0 and N == 0: nothing launched, SD_OK
    rp = torch.zeros(1, dtype=torch.int32, device="cuda")
    p0 = sd.Plan(rp, rp, torch.zeros(1, device="cuda"), 0, 10, 4, family=fam)
    sd.sd_spmm(p0.handle, 0, 4, 0, 4, 1.0, 0.0)
    p0.close()
    w = W.random_csr(8, 8, 1, np.full(8, 2), seed=9)
    dw = DeviceWorkload(w)
    pn = dw.plan(family=fam, N=0)
    sd.sd_spmm(pn.handle, 0, 0, 0, 0, 1.0, 0.0)
    pn.close()


def test_invalid_arguments_return_codes():
    w = W.random_csr(16, 16, 4, np.full(16, 2), seed=1)
    dw = DeviceWorkload(w)
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_create_ex(None, dw.colind, dw.vals, 16, 16, 4)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_create_ex(dw.rowptr, dw.colind, dw.vals, -1, 16, 4)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_create_ex(dw.rowptr, dw.colind, dw.vals, 16, 16, 4, dtype=7)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_create_ex(dw.rowptr, dw.colind, dw.vals, 16, 16, 4, family=9)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    # malformed CSR is caught by validation
    bad = dw.colind.clone()
    bad[3] = 99
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_create_ex(dw.rowptr, bad, dw.vals, 16, 16, 4, validate=True)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    plan = dw.plan()
    B = torch.zeros(16, 4, device="cuda")
    Cm = torch.zeros(16, 4, device="cuda")
    with pytest.raises(sd.SdError) as e:
        sd.sd_spmm(plan.handle, B, 3, Cm, 4, 1.0, 0.0)     # ldb < N
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_spmm(plan.handle, B, 4, None, 4, 1.0, 0.0)   # null C
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_spmm(None, B, 4, Cm, 4, 1.0, 0.0)
    assert e.value.code == sd.SD_ERR_INVALID_ARG
    with pytest.raises(sd.SdError) as e:
        sd.sd_plan_get_bsr(plan.handle)
    assert e.value.code == sd.SD_ERR_UNSUPPORTED
    sd.sd_plan_destroy(None)   # no-op
    plan.close()
    # the context is still healthy
    torch.cuda.synchronize()


def small_configs():
    return {
        "tiny_uniform": W.g1_tiny_uniform(),
        "stencil": W.g2_stencil(n=96, N=64),
        "gcn_rmat": W.g3_gcn_rmat(scale=13, N=128),
        "block16_f32": W.g4_block(Mb=128, Kb=128, N=256, nblocks=300),
        "block16_bf16": W.g4_block(Mb=128, Kb=128, N=256, nblocks=300, dtype=W.SD_BF16),
        "skewed": W.g5_skewed(M=1 << 16, N=32, scale_c=2.4e7 / 64, cap=4000),
    }


EXPECTED_FAMILY = {"tiny_uniform": 1, "stencil": 1, "gcn_rmat": 2, "block16_f32": 3, "block16_bf16": 3, "skewed": 2}


@pytest.mark.parametrize("name", list(EXPECTED_FAMILY))
def test_scaled_configs_auto_plan_and_plan_parity(name):
    w = small_configs()[name]
    dw = DeviceWorkload(w)
    plan = dw.plan(validate=True)
    info = plan.info()
    # plan metadata: bit-exact against the oracle's own summary and rule
    ref = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    mine = info.as_dict()
    for k, v in ref.as_dict().items():
        assert mine[k] == v, k
    assert info.family == oracle.decide_family(ref, w.dtype, info.l2_bytes) == EXPECTED_FAMILY[name]
    if info.family == sd.SD_MERGE:
        assert bool(info.class_split) == (info.windows > 1 or oracle.decide_class_split(ref, w.dtype))
    if info.family == sd.SD_MERGE and not info.class_split:
        tiles = sd.sd_plan_get_tiles(plan.handle)
        assert np.array_equal(tiles, oracle.merge_coords(w.rowptr, info.tile_items))
        assert info.num_tiles == tiles.size - 1
    if info.family == sd.SD_MERGE and info.class_split:
        seg_ptr, seg_row, colind, vals, win_seg = sd.sd_plan_get_segments(plan.handle)
        rp, rr, perm, rw = oracle.window_segments(w.rowptr, w.colind, w.M, w.K, info.windows)
        assert np.array_equal(seg_ptr, rp) and np.array_equal(seg_row, rr) and np.array_equal(win_seg, rw)
        assert np.array_equal(colind, w.colind[perm]) and vals.tobytes() == w.vals[perm].tobytes()
    if info.family == sd.SD_HYBRID:
        assert info.windows == oracle.decide_windows(ref, w.dtype, info.l2_bytes) and info.heavy_len == 256
        got_s = sd.sd_plan_get_hybrid(plan.handle)
        ref_s = oracle.hybrid_schedule(w.rowptr, w.colind, w.M, w.K, info.windows, 256)
        assert all(np.array_equal(a, b) for a, b in zip(got_s, ref_s))
    if info.family == sd.SD_BSR_TC:
        browptr, bcol, bval = sd.sd_plan_get_bsr(plan.handle)
        rb, rc, rv = oracle.bsr16(w.rowptr, w.colind, w.vals, w.M, w.K)
        assert np.array_equal(browptr, rb) and np.array_equal(bcol, rc)
        assert bval.tobytes() == rv.tobytes()
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)
    plan.close()


def test_partially_filled_blocks_bsr_parity():
    # blocks on the last partial block-row / block-column, fill well below 100 %
    rng = np.random.default_rng(8)
    M, K, N = 1000 + 7, 500 + 3, 64
    w = W.random_csr(M, K, N, np.clip(rng.poisson(20, M), 0, K), seed=12, beta=1.5)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_BSR_TC)
    browptr, bcol, bval = sd.sd_plan_get_bsr(plan.handle)
    rb, rc, rv = oracle.bsr16(w.rowptr, w.colind, w.vals, M, K)
    assert np.array_equal(browptr, rb) and np.array_equal(bcol, rc) and bval.tobytes() == rv.tobytes()
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    plan.close()


def test_unsorted_and_duplicate_columns():
    # CSR families accept any order and sum duplicates; BSR is refused for such input
    rng = np.random.default_rng(4)
    M, K, N = 200, 90, 16
    w = W.random_csr(M, K, N, rng.integers(1, 12, M), seed=6)
    for i in range(0, M, 3):     # reverse some rows, duplicate an entry in others
        lo, hi = w.rowptr[i], w.rowptr[i + 1]
        w.colind[lo:hi] = w.colind[lo:hi][::-1].copy()
        w.vals[lo:hi] = w.vals[lo:hi][::-1].copy()
        if hi - lo >= 2 and i % 2 == 0:
            w.colind[lo + 1] = w.colind[lo]
    dw = DeviceWorkload(w)
    for fam in (sd.SD_ROWSPLIT, sd.SD_MERGE):
        plan = dw.plan(family=fam)
        assert plan.info().unsorted_rows == oracle.summary(w.rowptr, w.colind, M, K, N).unsorted_rows > 0
        got, _ = run_spmm(plan, w)
        check(w, got)
        plan.close()
    with pytest.raises(sd.SdError) as e:
        dw.plan(family=sd.SD_BSR_TC)
    assert e.value.code == sd.SD_ERR_UNSUPPORTED
    assert dw.plan().info().family != sd.SD_BSR_TC


def test_long_all_positive_row_stays_inside_tolerance():
    # 200,000 same-sign terms in one row: sequential fp32 summation would drift to the edge of
    # 1e-5; the tiled summation of the merge family and the chunked one of the hybrid family must stay well inside
    M, K, N = 64, 262144, 32
    r = np.full(M, 3, np.int64)
    r[17] = 200_000
    r[5], r[6], r[40] = 255, 254, 15     # the longest rows that the hybrid family still sums as one running sum
    w = W.random_csr(M, K, N, r, seed=31, positive=True)
    dw = DeviceWorkload(w)
    for fam in (sd.SD_MERGE, sd.SD_HYBRID, sd.SD_ROWSPLIT):
        plan = dw.plan(family=fam)
        got, _ = run_spmm(plan, w)
        res = check(w, got)
        if fam != sd.SD_ROWSPLIT:
            assert res["max_ratio"] < 0.5
        plan.close()
    assert dw.plan().info().family == sd.SD_MERGE      # a small call: the merge family (tiles at this size)


def test_one_row_holds_every_nonzero_and_rows_straddle_many_tiles():
    M, K, N = 5000, 40000, 8
    r = np.zeros(M, np.int64)
    r[4321] = 30000
    w = W.random_csr(M, K, N, r, seed=2)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE)
    got, _ = run_spmm(plan, w, c_fill=np.full((M, N), np.nan, np.float32))
    check(w, got)
    plan.close()
    # rows of ~2.5 tiles each, back to back
    r = np.full(40, 2600, np.int64)
    w = W.random_csr(40, 8192, 32, r, seed=3, beta=0.25)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE, windows=1)
    got, _ = run_spmm(plan, w)
    check(w, got)
    plan.close()


def test_identity_and_permutation_are_exact():
    n, N = 4096, 64
    rng = np.random.default_rng(0)
    perm = rng.permutation(n).astype(np.int32)
    B = rng.standard_normal((n, N)).astype(np.float32)
    w = W.Workload("perm", n, n, N, np.arange(n + 1, dtype=np.int32), perm, np.ones(n, np.float32), B, None)
    dw = DeviceWorkload(w)
    for fam in (sd.SD_ROWSPLIT, sd.SD_MERGE):
        plan = dw.plan(family=fam)
        got, _ = run_spmm(plan, w)
        assert np.array_equal(got, B[perm])
        plan.close()


def test_plan_reuse_with_second_dense_operand_and_host_entry():
    w = W.g1_tiny_uniform(M=512, K=700, N=32, seed=8)
    dw = DeviceWorkload(w)
    plan = dw.plan()
    got, _ = run_spmm(plan, w)
    check(w, got)
    w2 = W.g1_tiny_uniform(M=512, K=700, N=32, seed=8)
    w2.B = np.random.default_rng(1).standard_normal(w.B.shape).astype(np.float32)
    got2, _ = run_spmm(plan, w2)
    check(w2, got2)
    # host buffers through sd_spmm_host
    Bh = torch.from_numpy(w2.B).pin_memory()
    Ch = torch.full((w.M, w.N), float("nan")).pin_memory()
    plan.spmm_host(Bh, Ch, 1.0, 0.0)
    assert np.array_equal(Ch.numpy(), got2)
    Cin = np.random.default_rng(2).standard_normal((w.M, w.N)).astype(np.float32)
    Ch = torch.from_numpy(Cin.copy()).pin_memory()
    plan.spmm_host(Bh, Ch, 0.5, 2.0)
    check(w2, Ch.numpy(), c_in=Cin, alpha=0.5, beta=2.0)
    # the two-part form: two calls queued back to back on the plan's stream, one wait
    Ca = torch.full((w.M, w.N), float("nan")).pin_memory()
    Cb = torch.from_numpy(Cin.copy()).pin_memory()
    plan.spmm_host_async(Bh, Ca, 1.0, 0.0)
    plan.spmm_host_async(Bh, Cb, 0.5, 2.0)
    plan.sync()
    assert np.array_equal(Ca.numpy(), got2) and np.array_equal(Cb.numpy(), Ch.numpy())
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
@pytest.mark.parametrize("N", [1, 2, 3, 4])
@pytest.mark.parametrize("mean", [3, 9, 20, 40, 70, 300])
def test_rowsplit_narrow_widths_every_lane_group(mean, N, dtype):
    """Row-split family at one to four columns: 1, 2, 4, 8 or 16 lanes share a row according to the mean
    row length; empty rows, rows far longer than the mean (the two-level sum), ragged row count, padded and
    misaligned operands."""
    rng = np.random.default_rng(mean * 10 + N)
    M, K = 1031, 2500
    lengths = np.clip(rng.poisson(mean, M), 0, K)
    lengths[::17] = 0
    lengths[5] = K            # one row holds every column
    lengths[M - 1] = 1
    w = W.random_csr(M, K, N, lengths, seed=mean + N, dtype=dtype, alpha=-0.75, beta=0.5)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_ROWSPLIT)
    for kw in (dict(), dict(pad_b=3, pad_c=5), dict(offset=1), dict(offset=2, pad_b=1)):
        got, intact = run_spmm(plan, w, **kw)
        assert intact
        check(w, got)
    got2, _ = run_spmm(plan, w)
    got3, _ = run_spmm(plan, w)
    assert np.array_equal(got2, got3)
    poison = np.full((M, N), np.nan, np.float32)
    got4, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got4, beta=0.0)
    plan.close()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_row_and_column_shards_of_one_product(world, dtype):
    """The two collective-free splits of one product, every rank's share run in turn on this GPU
    (the shares do not wait on one another): row ranges with rebased pointers and all of B; column
    ranges through offset base pointers with the full leading dimensions."""
    from paper_2608_05033_b200.shard import column_shard, row_shard_bounds, row_shard_csr
    from util import dev
    w = W.config(2, scale=12, N=96, dtype=dtype)
    Bd = dev(w.B)
    # rows
    Cd = torch.full((w.M, w.N), float("nan"), device="cuda")
    b = row_shard_bounds(w.rowptr, world)
    for rank in range(world):
        r0, r1 = int(b[rank]), int(b[rank + 1])
        rp, cj, v = row_shard_csr(w.rowptr, w.colind, w.vals, r0, r1)
        plan = sd.Plan(dev(rp), dev(cj), dev(v), r1 - r0, w.K, w.N, dtype=dtype)
        plan.spmm(Bd, Cd[r0:r1], 1.0, 0.0)
        torch.cuda.synchronize()
        plan.close()
    check(w, Cd.cpu().numpy())
    # columns
    Cd = torch.full((w.M, w.N), float("nan"), device="cuda")
    dw = DeviceWorkload(w)
    for rank in range(world):
        c0, n = column_shard(w.N, world, rank, 8)
        plan = dw.plan(N=n)
        plan.spmm(Bd[:, c0:c0 + n], Cd[:, c0:c0 + n], 1.0, 0.0)
        torch.cuda.synchronize()
        plan.close()
    check(w, Cd.cpu().numpy())


@pytest.mark.parametrize("dtype,N", [(W.SD_F32, 8), (W.SD_F32, 16), (W.SD_F32, 32), (W.SD_F32, 64), (W.SD_BF16, 8),
                                     (W.SD_BF16, 16), (W.SD_BF16, 32), (W.SD_BF16, 64), (W.SD_BF16, 128)])
@pytest.mark.parametrize("mean", [20, 40, 70, 300])
def test_rowsplit_long_rows_several_lane_sets_per_row(mean, N, dtype):
    """Row-split family at 8 to 64 fp32 (8 to 128 bf16) columns with long rows: 2 to 16 lane sets share a
    row and meet by shuffles; empty rows, one row far beyond the mean (two-level sum), ragged row count,
    padded leading dimensions, and a misaligned call that must take the plain kernel."""
    rng = np.random.default_rng(mean * 100 + N)
    M, K = 517, 3000
    lengths = np.clip(rng.poisson(mean, M), 0, K)
    lengths[::13] = 0
    lengths[7] = K
    lengths[M - 1] = 1
    w = W.random_csr(M, K, N, lengths, seed=mean + N, dtype=dtype, alpha=1.5, beta=-0.25)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_ROWSPLIT)
    vw = 4 if dtype == W.SD_F32 else 8
    for kw in (dict(), dict(pad_b=vw, pad_c=4), dict(offset=1)):
        got, intact = run_spmm(plan, w, **kw)
        assert intact
        check(w, got)
    got2, _ = run_spmm(plan, w)
    got3, _ = run_spmm(plan, w)
    assert np.array_equal(got2, got3)
    poison = np.full((M, N), np.nan, np.float32)
    got4, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got4, beta=0.0)
    plan.close()


@pytest.mark.parametrize("N", [8, 32, 128])
def test_symmetric_adjacency_forward_plan_serves_the_backward_product(N):
    """Sec. 5, GCN evaluation: the backward aggregation is a product with the transposed adjacency;
    the normalised adjacency is symmetric, so the forward plan serves it.  The oracle gets the
    explicitly transposed CSR (a counting-sort transpose written here), the library the forward plan."""
    w = W.config(2, scale=12, N=N)
    M, nnz = w.M, w.nnz
    rows = np.repeat(np.arange(M, dtype=np.int64), np.diff(w.rowptr))
    order = np.lexsort((rows, w.colind))                      # transpose: sort by (column, row)
    t_rowptr = np.zeros(M + 1, np.int32)
    np.cumsum(np.bincount(w.colind, minlength=M), out=t_rowptr[1:])
    t_colind = rows[order].astype(np.int32)
    t_vals = w.vals[order]
    assert np.array_equal(t_rowptr, w.rowptr) and np.array_equal(t_colind, w.colind)   # pattern symmetric
    assert np.array_equal(t_vals, w.vals)                                               # values symmetric, bit for bit
    G = np.random.default_rng(N).standard_normal((M, N)).astype(np.float32)            # an upstream gradient
    dw = DeviceWorkload(w)
    plan = dw.plan()
    w.B = G
    got, _ = run_spmm(plan, w)
    r = oracle.check(t_rowptr, t_colind, t_vals, G, N, got, None, 1.0, 0.0)
    assert r["ok"], r
    plan.close()


@pytest.mark.parametrize("case", ["rowsplit", "merge", "merge_split", "merge_narrow", "merge_windows", "bsr_bf16", "bsr_f32"])
def test_update_values_same_pattern(case):
    # new values for an unchanged pattern: every representation that holds its own copy of the values
    # (window-major lists, 16x16 blocks and their tensor-core images) must follow
    rng = np.random.default_rng(11)
    dtype = W.SD_BF16 if case == "bsr_bf16" else W.SD_F32
    if case.startswith("bsr"):
        M, K, N = 16 * 21 + 3, 16 * 17, 128
        lengths = np.clip(rng.poisson(40, M), 0, K)
        family, windows = sd.SD_BSR_TC, 0
    else:
        M, K = 2100, 4000
        N = 3 if case == "merge_narrow" else 32
        lengths = shape_lengths("skewed", M, K, rng)
        family = sd.SD_ROWSPLIT if case == "rowsplit" else sd.SD_MERGE
        windows = {"merge_windows": 4, "merge_split": -1, "merge": 1}.get(case, 0)   # merge: row-ordered tiles
    w = W.random_csr(M, K, N, lengths, seed=77, dtype=dtype, alpha=1.0, beta=0.0)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=family, windows=windows)
    got, _ = run_spmm(plan, w)
    check(w, got)
    # second set of values, same pattern
    v2 = np.random.default_rng(12).standard_normal(w.nnz).astype(np.float32)
    w2 = W.Workload(w.name, w.M, w.K, w.N, w.rowptr, w.colind, W.f32_to_bf16_bits(v2) if dtype == W.SD_BF16 else v2,
                    w.B, None, 1.0, 0.0, dtype, {})
    from util import dev
    vals2 = dev(w2.vals)
    plan.update_values(vals2)
    got2, _ = run_spmm(plan, w2)
    assert plan.device_status() == 0
    check(w2, got2)
    assert not np.array_equal(got, got2)
    if case.startswith("bsr"):
        browptr, bcol, bval = sd.sd_plan_get_bsr(plan.handle)
        rb, rc, rv = oracle.bsr16(w2.rowptr, w2.colind, w2.vals, M, K)
        assert np.array_equal(browptr, rb) and np.array_equal(bcol, rc) and bval.tobytes() == rv.tobytes()
    if case == "merge_windows":
        seg_ptr, seg_row, colind, vals, win_seg = sd.sd_plan_get_segments(plan.handle)
        rp, rr, perm, rw = oracle.window_segments(w2.rowptr, w2.colind, M, K, 4)
        assert np.array_equal(colind, w2.colind[perm]) and vals.tobytes() == w2.vals[perm].tobytes()
    plan.close()


@pytest.mark.parametrize("lengths", [[1], [128], [129], [0, 0, 1, 0], [1000], [0, 127, 1, 0, 128, 0], [5] * 257,
                                     [0] * 40 + [300] + [0] * 40, [1] * 128 + [2] * 64])
def test_merge_narrow_operand_chunk_edges(lengths):
    # the 128-nonzero chunks of the narrow-width path: lists that end exactly on a chunk, one nonzero
    # past it, a single row over several chunks, rows that end exactly on chunk and 32-lane
    # boundaries, empty rows at both ends
    lengths = np.asarray(lengths, np.int64)
    M, K = len(lengths), 1200
    for N in (1, 4):
        w = W.random_csr(M, K, N, lengths, seed=int(lengths.sum()) + N, alpha=2.0, beta=0.5)
        dw = DeviceWorkload(w)
        plan = dw.plan(family=sd.SD_MERGE)
        got, intact = run_spmm(plan, w)
        assert intact
        check(w, got)
        plan.close()


@pytest.mark.parametrize("N", [1, 2, 3, 4])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_merge_narrow_operand_all_carry_levels(N, dtype):
    # dense widths up to 4 take the segmented reduction over (row, column, value) triples: enough
    # nonzeros that its carry list goes through the second level, one row holding every column (it
    # spans one to two thousand chunks), runs of empty rows, one-nonzero rows, a padded
    # and misaligned B
    rng = np.random.default_rng(N)
    M, K = 5003, 260_000
    lengths = np.clip((40000.0 * np.arange(1, M + 1) ** -0.9).astype(np.int64), 1, 30000)
    lengths = rng.permutation(lengths)
    lengths[100:140] = 0
    lengths[M // 2] = K
    lengths[M - 1] = 0
    w = W.random_csr(M, K, N, lengths, seed=40 + N, dtype=dtype, alpha=0.75, beta=-1.5)
    chunk = 256 if N <= 2 else 128
    assert 2 * ((w.nnz + chunk - 1) // chunk) > 4096   # the first carry list is longer than the direct-final limit
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE)
    assert plan.info().launches == 3
    for pad_b, offset in [(0, 0), (3, 1)]:
        got, intact = run_spmm(plan, w, pad_b=pad_b, pad_c=pad_b, offset=offset)
        assert intact
        check(w, got)
    got2, _ = run_spmm(plan, w, pad_b=3, pad_c=3, offset=1)
    assert np.array_equal(got, got2)
    poison = np.full((M, N), np.nan, np.float32)
    got3, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got3, beta=0.0)
    got4, _ = run_spmm(plan, w, beta=1.0)
    check(w, got4, beta=1.0)
    plan.close()


@pytest.mark.parametrize("N", [64, 128, 192, 256, 320, 512])
@pytest.mark.parametrize("beta", [0.0, -0.75])
@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_bsr_tensor_core_path(N, beta, dtype):
    # blocks on the tcgen05 path (bf16 directly, fp32 as three tf32 products): ragged M and K,
    # empty block-rows, partially filled blocks, padded leading dimensions (ldb kept a multiple of 8
    # so that the TMA alignment rules hold; ldc = N + 4 keeps the 16-byte stores of the epilogue,
    # ldc = N + 3 breaks them and must be served by the SIMT form with the same result)
    rng = np.random.default_rng(N)
    M, K = 16 * 37 + 5, 16 * 29 + 11
    lengths = np.clip(rng.poisson(30, M), 0, K)
    lengths[32:64] = 0        # two empty block-rows
    w = W.random_csr(M, K, N, lengths, seed=N + 1, dtype=dtype, alpha=1.5, beta=beta)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_BSR_TC)
    for pad_b, pad_c in [(0, 0), (8, 4), (8, 3)]:
        got, intact = run_spmm(plan, w, pad_b=pad_b, pad_c=pad_c)
        assert plan.device_status() == 0
        assert intact
        check(w, got)
    got2, _ = run_spmm(plan, w, pad_b=8, pad_c=3)
    assert np.array_equal(got, got2)
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_bsr_tensor_core_block_row_partition(dtype):
    # very uneven block-rows: one with 2,500 blocks (more than the kernel stages at once, so it goes
    # through the oversized-row path), runs of empty block-rows, a ragged tail; 512 dense columns =
    # two slabs per block-row.  The CTAs' block-row ranges come from the plan-time partition.
    rng = np.random.default_rng(17)
    M, K, N = 16 * 400 + 7, 16 * 2500, 512
    lengths = np.clip(rng.poisson(20, M), 0, K)
    lengths[16 * 40:16 * 90] = 0
    lengths[16 * 200] = K            # every block of this block-row is occupied
    lengths[16 * 399:] = 0
    w = W.random_csr(M, K, N, lengths, seed=23, dtype=dtype, alpha=-0.5, beta=0.25)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_BSR_TC)
    got, intact = run_spmm(plan, w)
    assert plan.device_status() == 0
    assert intact
    check(w, got)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
@pytest.mark.parametrize("fill", [0.5, 0.2])
def test_partially_filled_blocks_take_the_block_form_while_it_pays(dtype, fill):
    # 16x16 blocks thinned to a given fill: the automatic rule keeps the tensor-core block form down to
    # a fill of 1/rho_max(dtype, N) -- at N = 256: 33 % for fp32, 10 % for bf16 -- and the result is
    # right either way
    base = W.g4_block(Mb=96, Kb=80, N=256, nblocks=700, seed=9, dtype=W.SD_F32)
    rng = np.random.default_rng(int(fill * 100))
    keep = rng.random(base.nnz) < fill
    rows = np.repeat(np.arange(base.M), np.diff(base.rowptr))
    rowptr = np.zeros(base.M + 1, np.int32)
    np.cumsum(np.bincount(rows[keep], minlength=base.M), out=rowptr[1:])
    vals = base.vals[keep]
    B = base.B
    if dtype == W.SD_BF16:
        vals, B = W.f32_to_bf16_bits(vals), W.f32_to_bf16_bits(B).reshape(B.shape)
    w = W.Workload("thinned_blocks", base.M, base.K, base.N, rowptr, base.colind[keep], vals, B, None, 1.0, 0.0, dtype, {})
    dw = DeviceWorkload(w)
    plan = dw.plan()
    info = plan.info()
    ref = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    assert info.family == oracle.decide(ref, dtype)
    expect_tc = (dtype == W.SD_BF16) or fill == 0.5
    assert (info.family == sd.SD_BSR_TC) == expect_tc
    got, _ = run_spmm(plan, w)
    assert plan.device_status() == 0
    check(w, got)
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_bsr_tensor_core_dense_blocks_exact_products(dtype):
    # fully dense blocks, small integers: every product and partial sum is exact in fp32 (and the
    # lo halves of the fp32 split vanish), so the tensor-core result must equal the oracle bit for bit
    w = W.g4_block(Mb=96, Kb=80, N=256, nblocks=700, seed=5, dtype=dtype)
    rng = np.random.default_rng(1)
    iv = rng.integers(-4, 5, w.vals.shape).astype(np.float32)
    ib = rng.integers(-4, 5, w.B.shape).astype(np.float32)
    w.vals = W.f32_to_bf16_bits(iv) if dtype == W.SD_BF16 else iv
    w.B = W.f32_to_bf16_bits(ib).reshape(w.B.shape) if dtype == W.SD_BF16 else ib
    dw = DeviceWorkload(w)
    plan = dw.plan()
    assert plan.info().family == sd.SD_BSR_TC
    got, _ = run_spmm(plan, w)
    assert plan.device_status() == 0
    ref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, w.B, w.N)
    assert np.array_equal(got.astype(np.float64), ref)
    plan.close()


@pytest.mark.parametrize("kind", ["uniform", "short", "skewed", "onelong"])
@pytest.mark.parametrize("windows", [2, 8, 5])
@pytest.mark.parametrize("N,dtype", [(32, W.SD_F32), (8, W.SD_F32), (128, W.SD_BF16), (7, W.SD_F32)])
def test_merge_with_column_windows(kind, windows, N, dtype):
    rng = np.random.default_rng(windows * 100 + N)
    M, K = 1500, 3001
    lengths = shape_lengths(kind, M, K, rng)
    lengths[100:110] = 0     # empty rows must still receive beta*C
    w = W.random_csr(M, K, N, lengths, seed=N + windows, dtype=dtype, alpha=0.5, beta=1.25)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE, windows=windows)
    info = plan.info()
    assert info.windows == windows
    # plan metadata against the oracle's own window-major construction
    seg_ptr, seg_row, colind, vals, win_seg = sd.sd_plan_get_segments(plan.handle)
    rp, rr, perm, rw = oracle.window_segments(w.rowptr, w.colind, M, K, windows)
    assert np.array_equal(seg_ptr, rp) and np.array_equal(seg_row, rr) and np.array_equal(win_seg, rw)
    assert np.array_equal(colind, w.colind[perm]) and vals.tobytes() == w.vals[perm].tobytes()
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)
    poison = np.full((M, N), np.nan, np.float32)
    got3, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got3, beta=0.0)
    plan.close()


@pytest.mark.parametrize("kind", ["uniform", "skewed", "onelong"])
@pytest.mark.parametrize("N,dtype", [(16, W.SD_F32), (32, W.SD_F32), (64, W.SD_BF16), (8, W.SD_F32), (100, W.SD_F32)])
def test_merge_class_split_with_one_window(kind, N, dtype):
    """windows = -1: the window-major schedule (chunks, one group per short segment, flat one-nonzero rows)
    without column windows; segment list against the oracle's construction, results against the oracle."""
    rng = np.random.default_rng(N)
    M, K = 1500, 3001
    lengths = shape_lengths(kind, M, K, rng)
    lengths[100:110] = 0
    w = W.random_csr(M, K, N, lengths, seed=N + 3, dtype=dtype, alpha=0.5, beta=1.25)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE, windows=-1)
    info = plan.info()
    assert info.windows == 1 and info.class_split == 1
    seg_ptr, seg_row, colind, vals, win_seg = sd.sd_plan_get_segments(plan.handle)
    rp, rr, perm, rw = oracle.window_segments(w.rowptr, w.colind, M, K, 1)
    assert np.array_equal(seg_ptr, rp) and np.array_equal(seg_row, rr) and np.array_equal(win_seg, rw)
    assert np.array_equal(colind, w.colind[perm]) and vals.tobytes() == w.vals[perm].tobytes()
    assert not np.any(seg_row < 0)       # one window: no row is written twice
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)
    poison = np.full((M, N), np.nan, np.float32)
    got3, _ = run_spmm(plan, w, c_fill=poison, beta=0.0)
    check(w, got3, beta=0.0)
    plan.close()


def test_automatic_schedule_of_a_skewed_matrix_matches_the_rules():
    """Without column windows: the hybrid family from 5 columns up to 384-byte (fp32 values) or 256-byte (bf16 values)
    rows of B when the call gathers at least 256 MiB, else the merge family (tiles; the COO reduction up to 4 columns).  A forced merge plan still takes its
    class split by the width rule."""
    rng = np.random.default_rng(77)
    M, K = 20_000, 30_000
    lengths = rng.permutation(np.clip((250000.0 * np.arange(1, M + 1) ** -1.1).astype(np.int64), 1, 25000))
    for N, dtype in ((64, W.SD_F32), (96, W.SD_F32), (128, W.SD_F32), (32, W.SD_F32), (128, W.SD_BF16), (192, W.SD_BF16),
                     (256, W.SD_BF16), (4, W.SD_F32)):
        w = W.random_csr(M, K, N, lengths, seed=21, dtype=dtype)
        dw = DeviceWorkload(w)
        plan = dw.plan()
        info = plan.info()
        ref = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
        assert oracle.decide(ref, dtype) == oracle.MERGE
        assert info.windows == oracle.decide_windows(ref, dtype, info.l2_bytes) == 1
        row_bytes = N * (4 if dtype == W.SD_F32 else 2)
        hybrid = N >= 5 and row_bytes <= (384 if dtype == W.SD_F32 else 256) and w.nnz * row_bytes >= 1 << 28
        assert info.family == oracle.decide_family(ref, dtype, info.l2_bytes) == (sd.SD_HYBRID if hybrid else sd.SD_MERGE), (N, dtype)
        got, _ = run_spmm(plan, w)
        check(w, got)
        plan.close()
        forced = dw.plan(family=sd.SD_MERGE)
        fi = forced.info()
        assert fi.family == sd.SD_MERGE
        assert bool(fi.class_split) == oracle.decide_class_split(ref, dtype) == ((16 if dtype == W.SD_F32 else 8) <= N <= (64 if dtype == W.SD_F32 else 32))
        got, _ = run_spmm(forced, w)
        check(w, got)
        forced.close()
    assert 1_100_000 < w.nnz < 2_000_000      # 256-byte rows and more reach 256 MiB, 128-byte rows do not


def test_automatic_window_choice_matches_the_rule():
    w = W.g5_skewed(M=1 << 16, N=32, scale_c=2.4e7 / 64, cap=4000)
    dw = DeviceWorkload(w)
    plan = dw.plan()
    info = plan.info()
    ref = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    assert info.windows == oracle.decide_windows(ref, oracle.F32, info.l2_bytes) == 1   # B fits in L2 here
    plan.close()


def _without_column_zero(w, poison):
    """The same matrix with every column index moved up by one (so column 0 is never referenced) and a new
    row 0 of B holding `poison`."""
    es = np.float32 if w.dtype == W.SD_F32 else np.uint16
    row0 = np.full((1, w.N), poison, dtype=np.float32)
    if w.dtype == W.SD_BF16:
        row0 = W.f32_to_bf16_bits(row0).reshape(1, w.N)
    B = np.concatenate([row0.astype(es), w.B], axis=0)
    return W.Workload(w.name + "_no_col0", w.M, w.K + 1, w.N, w.rowptr, (w.colind + 1).astype(np.int32), w.vals, B,
                      w.C0, w.alpha, w.beta, w.dtype, dict(w.meta))


@pytest.mark.parametrize("poison", [np.inf, np.nan])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
@pytest.mark.parametrize("N,windows", [(32, -1), (32, 4), (8, -1), (1, 1), (3, 1), (4, 1), (64, 1)])
def test_non_finite_row_zero_of_b_stays_out_of_rows_that_do_not_name_it(poison, dtype, N, windows):
    """Kernels that pad a batch of nonzeros with (column 0, value 0) must not let B[0, :] into the sum: with
    B[0, :] = Inf or NaN and no entry in column 0, every result is finite and right.  Long segments of 129 to
    255 nonzeros (a partly filled last chunk) under the class split and under column windows, and one to four
    columns with a nonzero count that is not a multiple of the reduction's chunk."""
    rng = np.random.default_rng(99 + N)
    M, K = 700, 2600
    lengths = rng.integers(0, 6, M)
    lengths[rng.choice(M, 40, replace=False)] = rng.integers(129, 256, 40)
    lengths[5] = 2047
    w0 = W.random_csr(M, K, N, lengths, seed=321 + N, dtype=dtype)
    assert w0.nnz % 256 != 0 and w0.nnz % 128 != 0
    w = _without_column_zero(w0, poison)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_MERGE, windows=windows)
    got, intact = run_spmm(plan, w)
    assert intact and np.all(np.isfinite(got))
    # the oracle on the shifted matrix never touches row 0 of B either; compare with the original problem
    r = oracle.check(w0.rowptr, w0.colind, w0.vals, w0.B, w0.N, got, None, w0.alpha, w0.beta)
    assert r["ok"], r
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
def test_row_split_with_row_sharded_b_gathers_into_local_memory_first(dtype):
    """The row split whose dense operand is dealt out by rows: every rank's piece goes into the exchange layout
    (equal, padded pieces), the gather lands them in one local buffer, and the rank's plan reads B from there.
    One process here: the gather is the single-rank copy, and the pieces of a three-rank deal are put together
    by hand the way all_gather_into_tensor lays them out, then every rank's rows are run in turn."""
    from paper_2608_05033_b200.shard import RowSplitSpmm, b_row_shard, row_shard_bounds, row_shard_csr
    from util import dev
    w = W.config(2, scale=11, N=64, dtype=dtype)
    K = w.K
    # single rank through the class: B travels through the gather buffer
    one = RowSplitSpmm(w.rowptr, w.colind, w.vals, w.M, K, w.N, dtype, "cuda")
    assert (one.r0, one.r1, one.per) == (0, w.M, K)
    Cd = torch.full((w.M, w.N), float("nan"), device="cuda")
    one.run(dev(w.B), Cd)
    torch.cuda.synchronize()
    check(w, Cd.cpu().numpy())
    one.close()
    # three ranks' pieces laid out as the collective would, the last piece short
    world = 3
    per = b_row_shard(K, world, 0)[2]
    full = np.full((world * per, w.N), 0x7FC0 if dtype == W.SD_BF16 else np.nan, dtype=w.B.dtype)
    for rank in range(world):
        k0, k1, _ = b_row_shard(K, world, rank)
        full[rank * per:rank * per + (k1 - k0)] = w.B[k0:k1]
    assert np.array_equal(full[:K], w.B)                      # consecutive pieces: the first K rows are B
    Bd = dev(full)[:K]
    Cd = torch.full((w.M, w.N), float("nan"), device="cuda")
    b = row_shard_bounds(w.rowptr, world)
    for rank in range(world):
        r0, r1 = int(b[rank]), int(b[rank + 1])
        rp, cj, v = row_shard_csr(w.rowptr, w.colind, w.vals, r0, r1)
        plan = sd.Plan(dev(rp), dev(cj), dev(v), r1 - r0, K, w.N, dtype=dtype)
        plan.spmm(Bd, Cd[r0:r1], 1.0, 0.0)
        torch.cuda.synchronize()
        plan.close()
    check(w, Cd.cpu().numpy())
