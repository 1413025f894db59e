"""The hybrid family (light rows row-wise, heavy rows as chunks of the caller's CSR arrays taken window by
window): its schedule bit-exact against the oracle's sequential definition, its results against the oracle
with the tolerance of the other parity tests (|C - Cref| <= rel * (|alpha| sum|a||b| + |beta||Cin|) + 1e-6,
rel = 1e-5 fp32 / 1e-2 bf16), and the rule that makes AUTO take it."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2608_05033_b200 as sd
    from util import DeviceWorkload, dev, run_spmm
else:
    sd = None


def check(w, got, c_in=None, alpha=None, beta=None):
    alpha = w.alpha if alpha is None else alpha
    beta = w.beta if beta is None else beta
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, c_in if c_in is not None else w.C0, alpha, beta)
    assert r["ok"], r


def lengths_of(kind, M, K, rng):
    if kind == "skewed":
        return rng.permutation(np.clip((3000.0 * np.arange(1, M + 1) ** -1.1).astype(np.int64), 0, min(K, 2500)))
    if kind == "edges":      # lengths around the threshold (16) and around one and two chunks inside a window
        r = rng.integers(0, 4, M)
        r[:12] = [15, 16, 17, 0, 127, 128, 129, 255, 256, 257, 1, 16]
        return rng.permutation(r)
    if kind == "all_heavy":
        return rng.integers(16, 60, M)
    if kind == "no_heavy":
        return rng.integers(0, 16, M)
    if kind == "giant":      # rows of more than 64 chunks: the reduction of a whole CTA
        r = rng.integers(0, 3, M)
        r[5], r[M - 2], r[M // 2] = 128 * 64 + 1, 128 * 70, 128 * 64
        return r
    raise ValueError(kind)


@pytest.mark.parametrize("kind,M,K", [("skewed", 1237, 3001), ("edges", 301, 700), ("all_heavy", 97, 400),
                                      ("no_heavy", 500, 300), ("giant", 333, 9500)])
@pytest.mark.parametrize("windows", [1, 3, 8])
def test_schedule_is_the_sequential_definition(kind, M, K, windows):
    rng = np.random.default_rng(M + windows)
    w = W.random_csr(M, K, 32, lengths_of(kind, M, K, rng), seed=M + 3)
    plan = DeviceWorkload(w).plan(family=sd.SD_HYBRID, windows=windows, heavy_len=16)
    info = plan.info()
    assert (info.family, info.windows, info.heavy_len) == (sd.SD_HYBRID, windows, 16)
    heavy, chunk_ptr, ranges, order, light = sd.sd_plan_get_hybrid(plan.handle)
    rh, rc, rr, ro, rl = oracle.hybrid_schedule(w.rowptr, w.colind, M, K, windows, 16)
    assert np.array_equal(heavy, rh) and np.array_equal(chunk_ptr, rc)
    assert np.array_equal(ranges, rr) and np.array_equal(order, ro) and np.array_equal(light, rl)
    assert (info.num_tiles, info.num_segments) == (rh.size, rr.shape[0])
    giants = int(np.sum(np.diff(rc) > 64)) if rh.size else 0
    assert info.launches == 1 + (1 if rh.size else 0) + (1 if giants else 0)   # fused kernel, chunk sums, those of very long rows
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    plan.close()


@pytest.mark.parametrize("N", [1, 4, 7, 8, 24, 32, 33, 64, 100, 128, 256])
@pytest.mark.parametrize("dtype", [W.SD_F32, W.SD_BF16])
@pytest.mark.parametrize("kind", ["skewed", "edges"])
def test_forced_hybrid_parity(N, dtype, kind):
    rng = np.random.default_rng(N + 17)
    M, K = (1237, 3001) if kind == "skewed" else (301, 700)
    w = W.random_csr(M, K, N, lengths_of(kind, M, K, rng), seed=N * 5 + 2, dtype=dtype, alpha=1.25, beta=-0.5)
    plan = DeviceWorkload(w).plan(family=sd.SD_HYBRID, windows=4, heavy_len=16 if kind == "edges" else 0)
    assert plan.info().family == sd.SD_HYBRID
    got, intact = run_spmm(plan, w)
    assert intact
    check(w, got)
    got2, _ = run_spmm(plan, w)
    assert np.array_equal(got, got2)                    # fixed summation order: identical bits
    got, intact = run_spmm(plan, w, pad_b=3, pad_c=5, offset=1)   # scalar kernels, padded leading dimensions
    assert intact
    check(w, got)
    nan_c = np.full((M, N), np.nan, np.float32)         # beta = 0 never reads C
    got, _ = run_spmm(plan, w, c_fill=nan_c, beta=0.0)
    check(w, got, beta=0.0)
    cin = rng.standard_normal((M, N)).astype(np.float32)
    got, _ = run_spmm(plan, w, c_fill=cin, alpha=0.0, beta=2.0)   # alpha = 0: C = beta * C
    assert np.array_equal(got, np.float32(2.0) * cin)
    plan.close()


def test_rows_that_never_name_column_zero_ignore_a_non_finite_row_zero_of_b():
    """Entries beyond the end of a chunk or a light row are (column 0, value 0): they must not be gathered."""
    rng = np.random.default_rng(2)
    M, K, N = 400, 900, 32
    r = rng.integers(0, 5, M)
    r[::37] = rng.integers(16, 300, r[::37].size)
    w0 = W.random_csr(M, K - 1, N, r, seed=8)
    B = rng.standard_normal((K, N)).astype(np.float32)
    B[0, :] = np.inf
    B[0, ::2] = np.nan
    w = W.Workload("shifted", M, K, N, w0.rowptr, w0.colind + np.int32(1), w0.vals, B, None, 1.0, 0.0, W.SD_F32, {})
    plan = DeviceWorkload(w).plan(family=sd.SD_HYBRID, windows=2, heavy_len=16)
    got, _ = run_spmm(plan, w)
    assert np.all(np.isfinite(got))
    Bf = B.copy()
    Bf[0, :] = 0.0                                       # no row names column 0: the oracle must not meet Inf * 0 either
    check(W.Workload("shifted", M, K, N, w.rowptr, w.colind, w.vals, Bf, None, 1.0, 0.0, W.SD_F32, {}), got)
    plan.close()


def test_unsorted_columns_are_refused_when_forced_and_fall_back_otherwise():
    rng = np.random.default_rng(4)
    M, K, N = 300, 500, 32
    w = W.random_csr(M, K, N, rng.integers(2, 40, M), seed=6)
    lo, hi = w.rowptr[7], w.rowptr[8]
    w.colind[lo:hi] = w.colind[lo:hi][::-1].copy()
    dw = DeviceWorkload(w)
    with pytest.raises(sd.SdError) as e:
        dw.plan(family=sd.SD_HYBRID)
    assert e.value.code == sd.SD_ERR_UNSUPPORTED
    plan = dw.plan()
    assert plan.info().family != sd.SD_HYBRID
    got, _ = run_spmm(plan, w)
    check(w, got)
    plan.close()


def test_new_values_are_read_from_the_new_array():
    rng = np.random.default_rng(5)
    M, K, N = 700, 1500, 32
    w = W.random_csr(M, K, N, lengths_of("skewed", M, K, rng), seed=9)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=sd.SD_HYBRID, windows=2, heavy_len=32)
    got, _ = run_spmm(plan, w)
    check(w, got)
    w2 = W.Workload(w.name, M, K, N, w.rowptr, w.colind, (w.vals * np.float32(-3.0)).astype(np.float32), w.B, None, 1.0,
                    0.0, w.dtype, {})
    v2 = dev(w2.vals)
    plan.update_values(v2)
    got, _ = run_spmm(plan, w2)
    check(w2, got)
    plan.close()


def test_auto_takes_the_hybrid_family_where_the_rule_says_so():
    """B beyond 60 % of L2 and short rows on average: column windows; 128-byte rows of B: the hybrid family
    in place of the windowed class split (and not at 64 fp32 columns)."""
    rng = np.random.default_rng(6)
    M, K = 60_000, 700_000
    lengths = rng.permutation(np.clip((40000.0 * np.arange(1, M + 1) ** -1.1).astype(np.int64), 1, 30000))
    for N, dtype, want in [(32, W.SD_F32, sd.SD_HYBRID), (64, W.SD_F32, sd.SD_MERGE), (64, W.SD_BF16, sd.SD_HYBRID)]:
        w = W.random_csr(M, K, N, lengths, seed=12, dtype=dtype)
        plan = DeviceWorkload(w).plan()
        info = plan.info()
        ref = oracle.summary(w.rowptr, w.colind, M, K, N)
        windows = oracle.decide_windows(ref, dtype, info.l2_bytes)
        assert windows > 1 and info.windows == windows
        assert info.family == oracle.decide_family(ref, dtype, info.l2_bytes) == want
        if want == sd.SD_HYBRID:
            assert info.heavy_len == 256 and info.launches <= 3
            got = sd.sd_plan_get_hybrid(plan.handle)
            ref_s = oracle.hybrid_schedule(w.rowptr, w.colind, M, K, windows, 256)
            assert all(np.array_equal(a, b) for a, b in zip(got, ref_s))
        got, _ = run_spmm(plan, w)
        check(w, got)
        plan.close()


@pytest.mark.parametrize("family,windows", [(4, 4), (2, 4)], ids=["hybrid", "windowed_class_split"])
def test_calls_can_be_captured_into_a_cuda_graph(family, windows):
    """The hybrid family launches on the caller's stream only; the windowed class split forks plan-owned side streams
    from it and joins them back with events, so a stream capture takes them in: two calls captured (the second adds to
    the first's result), replayed, checked."""
    rng = np.random.default_rng(3)
    M, K, N = 3000, 5000, 32
    w = W.random_csr(M, K, N, lengths_of("skewed", M, K, rng), seed=5)
    plan = DeviceWorkload(w).plan(family=family, windows=windows, heavy_len=64 if family == 4 else 0)
    B = dev(w.B)
    C = torch.full((M, N), float("nan"), device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        plan.spmm(B, C, 1.0, 0.0, side)                 # first call outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        plan.spmm(B, C, 1.0, 0.0, torch.cuda.current_stream())
        plan.spmm(B, C, 1.0, 1.0, torch.cuda.current_stream())
    for _ in range(2):
        C.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        check(w, C.cpu().numpy() / np.float32(2.0))      # C = A B + (A B): halving is exact
    plan.close()
