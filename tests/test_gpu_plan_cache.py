"""sd_plan_save / sd_plan_load: the analogue of the paper's cache of winning implementations (Sec. 3.4: cached
per sparsity pattern, operator, platform and dense width).  A saved plan, destroyed and loaded again, must be the
same plan: equal summary and decision, equal representation, bit-identical results; a blob for another pattern is
refused; new values for the saved pattern are taken at load time."""
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


def _cases():
    rng = np.random.default_rng(2608)
    skew = np.clip((3000.0 * np.arange(1, 1501) ** -1.2).astype(np.int64), 1, 2500)
    yield "rowsplit", W.g2_stencil(n=40, N=64), dict(family=1), None
    yield "merge_tiles", W.random_csr(1500, 4000, 128, rng.permutation(skew), seed=1, beta=0.5), dict(family=2, windows=1), "tiles"
    yield "merge_class_split", W.random_csr(1500, 4000, 32, rng.permutation(skew), seed=2), dict(family=2, windows=-1), "segments"
    yield "merge_windows", W.random_csr(1500, 4000, 32, rng.permutation(skew), seed=3, beta=-1.0), dict(family=2, windows=4), "segments"
    yield "merge_narrow", W.random_csr(1500, 4000, 2, rng.permutation(skew), seed=4), dict(family=2, windows=1), "tiles"
    yield "hybrid", W.random_csr(1500, 4000, 32, rng.permutation(skew), seed=5, beta=0.25), dict(family=4, windows=4, heavy_len=40), "hybrid"
    yield "hybrid_giant_row", W.random_csr(300, 9500, 64, np.r_[9000, rng.integers(0, 5, 299)], seed=6, dtype=W.SD_BF16), dict(family=4, windows=2), "hybrid"
    yield "blocks_bf16", W.g4_block(Mb=48, Kb=64, N=256, nblocks=150, dtype=W.SD_BF16), dict(family=3), "bsr"
    yield "blocks_fp32", W.g4_block(Mb=48, Kb=64, N=128, nblocks=150, dtype=W.SD_F32), dict(family=3), "bsr"
    yield "automatic", W.g1_tiny_uniform(), dict(), None


def _representation(plan, kind):
    if kind == "tiles":
        return [sd.sd_plan_get_tiles(plan.handle)]
    if kind == "segments":
        return list(sd.sd_plan_get_segments(plan.handle))
    if kind == "hybrid":
        return list(sd.sd_plan_get_hybrid(plan.handle))
    if kind == "bsr":
        return list(sd.sd_plan_get_bsr(plan.handle))
    return []


@pytest.mark.parametrize("name,w,opts,kind", list(_cases()), ids=[c[0] for c in _cases()])
def test_saved_plan_loads_as_the_same_plan(name, w, opts, kind):
    dw = DeviceWorkload(w)
    plan = dw.plan(**opts)
    info = plan.info().as_dict()
    rep = _representation(plan, kind)
    want, _ = run_spmm(plan, w)
    blob = plan.save()
    assert blob == plan.save()                       # the blob is a function of the plan alone
    plan.close()

    again = sd.Plan.load(blob, dw.rowptr, dw.colind, dw.vals)
    assert again.info().as_dict() == info
    for a, b in zip(_representation(again, kind), rep):
        assert a.dtype == b.dtype and np.array_equal(a, b)
    got, intact = run_spmm(again, w)
    assert intact and np.array_equal(got, want)      # bit-identical
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, w.C0, w.alpha, w.beta)
    assert r["ok"], r
    assert again.device_status() == 0

    # same pattern, new values: taken from the array given at load time
    if w.dtype == W.SD_F32 and w.nnz:
        v2 = (w.vals * np.float32(-0.5) + np.float32(0.25)).astype(np.float32)
        v2d = torch.from_numpy(v2).cuda()
        fresh = sd.Plan.load(blob, dw.rowptr, dw.colind, v2d)
        got2, _ = run_spmm(fresh, w)
        r = oracle.check(w.rowptr, w.colind, v2, w.B, w.N, got2, w.C0, w.alpha, w.beta)
        assert r["ok"], r
        fresh.close()
    again.close()


def test_blob_for_another_pattern_or_a_damaged_blob_is_refused():
    rng = np.random.default_rng(5)
    w = W.random_csr(400, 900, 32, rng.integers(0, 12, 400), seed=9)
    dw = DeviceWorkload(w)
    plan = dw.plan(family=2, windows=-1)
    blob = plan.save()
    plan.close()
    # one column index changed (same counts): the pattern hash must notice
    col2 = w.colind.copy()
    j = int(np.flatnonzero(np.diff(w.rowptr) >= 1)[0])
    p = w.rowptr[j + 1] - 1
    col2[p] = col2[p] + 1 if col2[p] + 1 < w.K and (p + 1 == w.rowptr[j + 1]) else col2[p] - 1
    with pytest.raises(sd.SdError) as e:
        sd.Plan.load(blob, dw.rowptr, torch.from_numpy(col2).cuda(), dw.vals)
    assert e.value.code == sd.SD_ERR_INVALID_ARG and "pattern" in str(e.value)
    # a different row split of the same nonzeros
    rp2 = w.rowptr.copy()
    k = int(np.flatnonzero((np.diff(w.rowptr)[:-1] >= 1))[0])
    rp2[k + 1] -= 1
    with pytest.raises(sd.SdError):
        sd.Plan.load(blob, torch.from_numpy(rp2).cuda(), dw.colind, dw.vals)
    with pytest.raises(sd.SdError):
        sd.Plan.load(blob[:len(blob) // 2], dw.rowptr, dw.colind, dw.vals)      # truncated
    with pytest.raises(sd.SdError):
        sd.Plan.load(b"\x00" * 4096, dw.rowptr, dw.colind, dw.vals)              # not a blob
    ok = sd.Plan.load(blob, dw.rowptr, dw.colind, dw.vals)                       # the right arrays still load
    ok.close()
