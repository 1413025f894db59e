"""sd_spmm_merge_static -- the entry point for callers that must not allocate device memory
(their framework already owns the GPU's free memory, or they cannot take cudaMalloc's
synchronisation) -- against the plan-based sd_spmm on the same inputs.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.  Tolerance as in the other parity tests:
|C - Cref| <= 1e-5 * (|alpha| sum|a||b| + |beta||Cin|) + 1e-6 per entry."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_static_scratch_entry_point_matches_planned_spmm_twice_in_a_row():
    import paper_2608_05033_b200 as sd

    # skewed rows: long rows span many tiles, so the carry-out scratch is really exercised
    w = W.g5_skewed(M=1 << 15, N=32, scale_c=2.4e7 / 128, cap=9000, seed=77)
    alpha, beta = 1.25, -0.5
    rng = np.random.default_rng(5)
    rowptr, colind, vals = _dev(w.rowptr), _dev(w.colind), _dev(w.vals)
    plan = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, family=sd.SD_MERGE, windows=1)
    for call in range(2):   # the second call finds the first one's leftovers in the scratch
        Bh = rng.standard_normal((w.K, w.N)).astype(np.float32)
        Cin = rng.standard_normal((w.M, w.N)).astype(np.float32)
        B = _dev(Bh)
        c_plan, c_static = _dev(Cin), _dev(Cin)
        plan.spmm(B, c_plan, alpha, beta)
        sd.sd_spmm_merge_static(rowptr, colind, vals, w.M, w.K, w.N, w.nnz, B, w.N, c_static, w.N, alpha, beta)
        torch.cuda.synchronize()
        got_plan, got_static = c_plan.cpu().numpy(), c_static.cpu().numpy()
        _, S = oracle.spmm(w.rowptr, w.colind, w.vals, Bh, w.N, Cin, alpha, beta)
        bound = 1e-5 * (abs(alpha) * S + abs(beta) * np.abs(Cin)) + 1e-6
        # each within the bound of the exact result, so at most two bounds apart
        assert np.all(np.abs(got_static.astype(np.float64) - got_plan.astype(np.float64)) <= 2 * bound), call
        assert oracle.check(w.rowptr, w.colind, w.vals, Bh, w.N, got_static, Cin, alpha, beta)["ok"], call
    plan.close()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    import paper_2608_05033_b200 as sd

    # 4M rows + 4M nonzeros at N = 128 need 8 MiB of carry-out rows: twice the fixed array.  The
    # call must refuse before it touches any operand, so small stand-in buffers are enough.
    M, N = 1 << 22, 128
    rowptr = torch.arange(M + 1, dtype=torch.int32, device="cuda")
    colind = torch.zeros(16, dtype=torch.int32, device="cuda")
    vals = torch.ones(16, device="cuda")
    B = torch.zeros(16, N, device="cuda")
    Cm = torch.full((16, N), 3.0, device="cuda")
    with pytest.raises(sd.SdError) as e:
        sd.sd_spmm_merge_static(rowptr, colind, vals, M, M, N, M, B, N, Cm, N, 1.0, 0.0)
    assert e.value.code == sd.SD_ERR_UNSUPPORTED and "4194304" in str(e.value)
    torch.cuda.synchronize()
    assert float(Cm[0, 0]) == 3.0      # nothing was launched


@pytest.mark.parametrize("N,offset", [(7, 0), (32, 1), (128, 0)])
def test_static_scratch_entry_point_scalar_paths_empty_rows_and_scalars(N, offset):
    """Dense widths and base pointers that force the scalar kernels, leading and trailing rows without
    nonzeros, beta = 0 over a NaN-filled C, alpha = 0, and a small call after a larger one (the larger call's
    leftovers beyond the small call's tiles must not matter)."""
    import paper_2608_05033_b200 as sd

    rng = np.random.default_rng(11 + N)
    M, K = 900, 1500
    lengths = rng.integers(0, 9, M)
    lengths[:17] = 0
    lengths[-9:] = 0
    lengths[400] = 1400
    w = W.random_csr(M, K, N, lengths, seed=55 + N)
    big = W.g5_skewed(M=1 << 14, N=N, scale_c=2.4e7 / 256, cap=5000, seed=3)
    rowptr, colind, vals = _dev(w.rowptr), _dev(w.colind), _dev(w.vals)

    def run(ws, rp, ci, va, alpha, beta, cin):
        Bh = np.zeros(ws.K * ws.N + offset + 4, dtype=np.float32)
        Bh[offset:offset + ws.K * ws.N] = ws.B.reshape(-1)
        Ch = np.zeros(ws.M * ws.N + offset + 4, dtype=np.float32)
        Ch[offset:offset + ws.M * ws.N] = cin.reshape(-1)
        Bd, Cd = _dev(Bh), _dev(Ch)
        sd.sd_spmm_merge_static(rp, ci, va, ws.M, ws.K, ws.N, ws.nnz, Bd.data_ptr() + 4 * offset, ws.N,
                                Cd.data_ptr() + 4 * offset, ws.N, alpha, beta)
        torch.cuda.synchronize()
        return Cd.cpu().numpy()[offset:offset + ws.M * ws.N].reshape(ws.M, ws.N)

    # a larger problem first: it leaves more tiles' worth of carry rows in the shared array
    cb = run(big, _dev(big.rowptr), _dev(big.colind), _dev(big.vals), 1.0, 0.0, np.zeros((big.M, big.N), np.float32))
    assert oracle.check(big.rowptr, big.colind, big.vals, big.B, big.N, cb, None, 1.0, 0.0)["ok"]
    nan_c = np.full((M, N), np.nan, np.float32)
    got = run(w, rowptr, colind, vals, 1.5, 0.0, nan_c)                 # beta = 0 never reads C
    assert oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, None, 1.5, 0.0)["ok"]
    assert np.all(got[:17] == 0) and np.all(got[-9:] == 0)              # rows without nonzeros are written
    cin = rng.standard_normal((M, N)).astype(np.float32)
    got = run(w, rowptr, colind, vals, 0.0, 0.5, cin)                   # alpha = 0: C = beta * C
    assert np.array_equal(got, np.float32(0.5) * cin)
    got = run(w, rowptr, colind, vals, -0.75, 2.0, cin)
    assert oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, cin, -0.75, 2.0)["ok"]
