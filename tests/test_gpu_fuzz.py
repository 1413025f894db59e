"""Seeded random shapes through every family against the oracle: sizes that are not multiples of anything, dense widths on
and off the vector paths, both value types, empty and very long rows, padded leading dimensions and unaligned base
pointers, forced window counts and long-row thresholds, and a save / load round trip now and then.
Tolerance as in the other parity tests (|C - Cref| <= rel * (|alpha| sum|a||b| + |beta||Cin|) + 1e-6, rel = 1e-5 / 1e-2)."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2608_05033_b200 as sd
    from util import DeviceWorkload, run_spmm
else:
    sd = None


def _lengths(kind, M, K, rng):
    if kind == "uniform":
        L = rng.poisson(6, M)
    elif kind == "short":
        L = rng.integers(0, 3, M)
    elif kind == "skewed":
        L = rng.permutation((K * 0.9 * np.arange(1, M + 1) ** -1.1).astype(np.int64))
    elif kind == "onelong":
        L = rng.integers(0, 2, M)
        L[rng.integers(0, M)] = K
    elif kind == "empty":
        L = np.zeros(M, np.int64)
    else:
        L = rng.poisson(3, M)
        idx = rng.integers(0, M, max(1, M // 20))
        L[idx] = rng.integers(0, K + 1, idx.size)
    return np.clip(L, 0, K)


@pytest.mark.parametrize("seed", range(48))
def test_random_case_through_every_family(seed):
    rng = np.random.default_rng(7000 + seed)
    M = int(rng.choice([1, 2, 7, 31, 64, 257, 1000, 3333]))
    K = int(rng.choice([1, 3, 17, 100, 513, 2048, 7001]))
    N = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16, 24, 31, 32, 40, 48, 64, 96, 100, 128, 160, 256]))
    dtype = int(rng.choice([W.SD_F32, W.SD_BF16]))
    kind = str(rng.choice(["uniform", "short", "skewed", "onelong", "empty", "mixed"]))
    alpha = float(rng.choice([1.0, -0.75, 0.0, 2.5]))
    beta = float(rng.choice([0.0, 0.0, 1.0, -0.5]))
    w = W.random_csr(M, K, N, _lengths(kind, M, K, rng), seed=7000 + seed, dtype=dtype, alpha=alpha, beta=beta)
    dw = DeviceWorkload(w)
    plans = [(sd.SD_AUTO, {}), (sd.SD_ROWSPLIT, {}), (sd.SD_MERGE, dict(windows=1)), (sd.SD_MERGE, dict(windows=-1)),
             (sd.SD_MERGE, dict(windows=int(rng.integers(2, 6)))),
             (sd.SD_HYBRID, dict(windows=int(rng.integers(1, 6)), heavy_len=int(rng.choice([0, 2, 16, 17, 40, 200])))),
             (sd.SD_BSR_TC, {})]
    pad_b, pad_c, off = int(rng.choice([0, 0, 3, 8])), int(rng.choice([0, 0, 5, 4])), int(rng.choice([0, 0, 1, 4]))
    for family, kw in plans:
        try:
            plan = dw.plan(family=family, **kw)
        except sd.SdError as e:
            assert family == sd.SD_BSR_TC and e.code == sd.SD_ERR_UNSUPPORTED, (family, kw, str(e))
            continue
        got, intact = run_spmm(plan, w, pad_b=pad_b, pad_c=pad_c, offset=off)
        r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, w.C0, alpha, beta)
        assert r["ok"] and intact and plan.device_status() == 0, (family, kw, kind, (M, K, N), dtype, (pad_b, pad_c, off), r)
        if family in (sd.SD_MERGE, sd.SD_HYBRID) and w.nnz and rng.random() < 0.3:
            blob = plan.save()
            plan.close()
            plan = sd.Plan.load(blob, dw.rowptr, dw.colind, dw.vals)
            again, _ = run_spmm(plan, w, pad_b=pad_b, pad_c=pad_c, offset=off)
            assert np.array_equal(got, again, equal_nan=True), (family, kw)
        plan.close()
