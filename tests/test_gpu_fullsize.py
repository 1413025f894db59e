"""The five benchmark workloads at full size, planned and launched exactly as bench.py does
(automatic family and windows), checked entry by entry against the CPU oracle with the stated
tolerance, plus plan-metadata parity where the oracle finishes in seconds."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

CASES = [("tiny_uniform", 0, W.SD_F32, 1), ("stencil", 1, W.SD_F32, 1), ("gcn_rmat", 2, W.SD_F32, 2),
         ("block16_f32", 3, W.SD_F32, 3), ("block16_bf16", 3, W.SD_BF16, 3), ("skewed", 4, W.SD_F32, 4),
         # narrow dense operands of the two merge-family workloads (SpMV and four columns)
         ("skewed_spmv", 4, W.SD_F32, 2), ("gcn_rmat_n4", 2, W.SD_F32, 2)]
NARROW = {"skewed_spmv": 1, "gcn_rmat_n4": 4}


@pytest.mark.parametrize("name,ci,dtype,family", CASES)
def test_full_size_config_matches_oracle(name, ci, dtype, family):
    import paper_2608_05033_b200 as sd
    from util import DeviceWorkload, dev

    w = W.config(ci, dtype=dtype, **({"N": NARROW[name]} if name in NARROW else {}))
    dw = DeviceWorkload(w)
    plan = dw.plan()
    info = plan.info()
    assert info.family == family
    ref = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    mine = info.as_dict()
    for k, v in ref.as_dict().items():
        assert mine[k] == v, k
    assert info.family == oracle.decide_family(ref, dtype, info.l2_bytes)
    if info.family in (sd.SD_MERGE, sd.SD_HYBRID):
        assert info.windows == oracle.decide_windows(ref, dtype, info.l2_bytes)
    if name not in NARROW:   # extended analysis (quartiles, column degrees, SELL / BSR slots), every count exact
        fo = oracle.features(w.rowptr, w.colind, w.M, w.K, ref, 4 if dtype == W.SD_F32 else 2)
        fm = plan.features()
        for k, v in fo.as_dict().items():
            g = getattr(fm, k)
            assert (list(g) if hasattr(g, "__len__") else int(g)) == v, k
    if name == "skewed":
        assert w.nnz == 59_839_586 and info.windows == 8
    if name == "stencil":
        assert w.nnz == 5_238_784
    Bd = dev(w.B)
    Cd = dev(w.C0) if w.C0 is not None else torch.full((w.M, w.N), float("nan"), device="cuda")
    plan.spmm(Bd, Cd, w.alpha, w.beta)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    got = Cd.cpu().numpy()
    r = oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, got, w.C0, w.alpha, w.beta)
    assert r["ok"], r
    # a second launch gives the same bits (beta != 0 needs C restored first)
    Cd2 = dev(w.C0) if w.C0 is not None else torch.full((w.M, w.N), float("nan"), device="cuda")
    plan.spmm(Bd, Cd2, w.alpha, w.beta)
    torch.cuda.synchronize()
    assert torch.equal(Cd, Cd2)
    plan.close()
