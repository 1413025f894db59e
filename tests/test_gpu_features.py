"""sd_plan_get_features against the oracle: every count bit-exact (integer work), the working-set
figures against the closed forms of Eq. 10-13."""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2608_05033_b200 as sd
    from util import DeviceWorkload
else:  # collected but skipped
    sd = None

COUNT_FIELDS = ["row_q", "col_q", "col_max", "col_empty", "sum_d2", "ell_slots", "sell_slots", "nnzb", "rep_bytes",
                "shape_class", "value_bytes"]


def as_dict(f, fields):
    out = {}
    for name in fields:
        v = getattr(f, name)
        out[name] = list(v) if hasattr(v, "__len__") else int(v)
    return out


def compare(w, plan):
    info = oracle.summary(w.rowptr, w.colind, w.M, w.K, w.N)
    vb = 4 if w.dtype == W.SD_F32 else 2
    want = oracle.features(w.rowptr, w.colind, w.M, w.K, info, vb)
    got = plan.features()
    assert as_dict(got, COUNT_FIELDS) == as_dict(want, COUNT_FIELDS)
    pinfo = plan.info()
    # Eq. 11-12 for the plan as built
    reads_csr = pinfo.family in (sd.SD_ROWSPLIT, sd.SD_HYBRID) or (pinfo.family == sd.SD_MERGE and not pinfo.class_split)
    assert got.borrowed_bytes == (oracle.csr_bytes(info, vb) if reads_csr else 0)
    assert got.plan_bytes == pinfo.plan_bytes
    m_r, m_t = oracle.working_set_bytes(got.borrowed_bytes + got.plan_bytes, info, vb)
    assert (got.m_r, got.m_t) == (m_r, m_t)
    assert (got.d_r, got.d_s) == (w.K * w.N * vb, 4 * w.M * w.N)
    units = {sd.SD_ROWSPLIT: w.M, sd.SD_MERGE: pinfo.num_segments if pinfo.class_split else pinfo.num_tiles,
             sd.SD_BSR_TC: (w.M + 15) // 16,
             sd.SD_HYBRID: pinfo.num_segments + w.M - pinfo.num_tiles}[pinfo.family]
    assert got.work_units == units
    assert (got.sm_count, got.l2_bytes) == (pinfo.sm_count, pinfo.l2_bytes)
    return got


CASES = {
    "tiny_uniform": lambda: W.config(0),
    "stencil": lambda: W.config(1, n=96),
    "gcn_rmat": lambda: W.config(2, scale=13),
    "block16": lambda: W.config(3, Mb=96, Kb=96),
    "block16_bf16": lambda: W.config(3, Mb=96, Kb=96, dtype=W.SD_BF16),
    "skewed": lambda: W.config(4, M=1 << 15, scale_c=2.4e7 / 64, cap=3000),
    "ragged": lambda: W.random_csr(1237, 3001, 8, np.random.default_rng(3).integers(0, 40, 1237), seed=5),
    "wide_short": lambda: W.random_csr(9, 70001, 4, [0, 5, 0, 70001, 1, 0, 0, 33, 2], seed=6),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_features_match_the_oracle(case):
    w = CASES[case]()
    plan = DeviceWorkload(w).plan()
    got = compare(w, plan)
    # a second call returns the stored analysis
    again = plan.features()
    assert bytes(again) == bytes(got)
    plan.close()


def test_features_of_a_rowsplit_plan_are_the_csr_closed_forms():
    w = W.config(1, n=64)
    plan = DeviceWorkload(w).plan(family=sd.SD_ROWSPLIT)
    f = compare(w, plan)
    assert f.plan_bytes == 0 and f.m_r == 8 * w.nnz + 4 * (w.M + 1) + 4 * w.K * w.N
    assert sd.SHAPE_NAMES[f.shape_class] == "uniform"
    plan.close()


def test_features_with_windows_and_forced_families():
    w = W.config(4, M=1 << 14, scale_c=2.4e7 / 256, cap=800)
    dw = DeviceWorkload(w)
    for kw in (dict(family=sd.SD_MERGE, windows=4), dict(family=sd.SD_MERGE, windows=1), dict(family=sd.SD_MERGE, windows=-1),
               dict(family=sd.SD_ROWSPLIT)):
        plan = dw.plan(**kw)
        f = compare(w, plan)
        assert sd.SHAPE_NAMES[f.shape_class] == "power-law"
        plan.close()


def test_features_of_degenerate_matrices():
    # no nonzeros at all; a single entry; one row
    for M, K, lengths in ((5, 7, [0] * 5), (3, 3, [0, 1, 0]), (1, 40, [40])):
        w = W.random_csr(M, K, 2, lengths, seed=M)
        plan = DeviceWorkload(w).plan()
        compare(w, plan)
        plan.close()
