"""What the tensor-core path (family (c): 16x16 blocks on tcgen05, paper Sec. 2.1 "dense sparse tiles can
enable Tensor Cores") only assumed, tested on the smallest cases:

* one 16x16 block times one 16x256 slab, against a plain triple loop written out here, with operands
  chosen so that any mix-up of the operand layouts (block image, slab image, accumulator rows and
  columns) or of the fp32 hi / lo split moves the result far outside the tolerance;
* a wait inside the kernel that runs out: the kernel must return by itself and report it.
"""
import numpy as np
import pytest

import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _dev(a):
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()


def _one_block_csr():
    rowptr = (np.arange(17) * 16).astype(np.int32)
    colind = np.tile(np.arange(16, dtype=np.int32), 16)
    return rowptr, colind


def _triple_loop(A, B):
    """C[r][n] = sum_k A[r][k] * B[k][n] in double, term by term."""
    C = np.zeros((16, B.shape[1]), dtype=np.float64)
    for r in range(16):
        for k in range(16):
            C[r, :] += float(A[r, k]) * B[k, :].astype(np.float64)
    return C


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_one_block_selector_operands_are_bit_exact(dtype):
    """B picks one column of the block per output column (scaled by a power of two), so every entry of C is
    one entry of A times a power of two: exact in every arithmetic, and a transposed or permuted operand
    image, a wrong core-matrix stride or a wrong accumulator row shows up as a wrong number."""
    import paper_2608_05033_b200 as sd
    rowptr, colind = _one_block_csr()
    A = np.arange(256, dtype=np.float32).reshape(16, 16) - 128.0      # 256 distinct values, each exact in bf16
    N = 256
    B = np.zeros((16, N), dtype=np.float32)
    for n in range(N):
        B[n % 16, n] = 2.0 ** (n // 16 - 8)
    want = _triple_loop(A, B)
    if dtype == W.SD_BF16:
        a_dev, b_dev = _dev(W.f32_to_bf16_bits(A.reshape(-1))), _dev(W.f32_to_bf16_bits(B).reshape(16, N))
        assert np.array_equal(W.bf16_bits_to_f32(W.f32_to_bf16_bits(A.reshape(-1))), A.reshape(-1))
    else:
        a_dev, b_dev = _dev(A.reshape(-1).copy()), _dev(B)
    plan = sd.Plan(_dev(rowptr), _dev(colind), a_dev, 16, 16, N, dtype=dtype, family=sd.SD_BSR_TC)
    assert plan.info().family == sd.SD_BSR_TC and plan.info().nnzb16 == 1
    Cd = torch.full((16, N), float("nan"), device="cuda")
    plan.spmm(b_dev, Cd, 1.0, 0.0)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    assert np.array_equal(Cd.cpu().numpy().astype(np.float64), want)
    plan.close()


def test_one_block_fp32_low_mantissa_bits_are_truncated_not_rounded():
    """fp32 runs as tf32 products of a hi / lo split, and the raw fp32 slab is handed to the tensor core as the
    `hi` operand: that is only right if the tensor core DROPS the low 13 mantissa bits of a 32-bit operand.
    Every entry of B here has all 13 of them set, so an operand rounded to nearest instead would be one tf32
    ulp (2^-10 relative) too large and the result would be off by about 1e-3 relative: a hundred times the
    tolerance, a thousand times the bound asserted here."""
    import paper_2608_05033_b200 as sd
    rng = np.random.default_rng(20260805)
    rowptr, colind = _one_block_csr()
    A = rng.uniform(0.5, 1.0, size=(16, 16)).astype(np.float32)
    A = (A.view(np.uint32) | np.uint32(0x1FFF)).view(np.float32)            # low bits set in the block as well
    N = 256
    B = rng.uniform(0.5, 1.0, size=(16, N)).astype(np.float32)
    B = (B.view(np.uint32) | np.uint32(0x1FFF)).view(np.float32)
    want = _triple_loop(A, B)
    S = _triple_loop(np.abs(A), np.abs(B))
    plan = sd.Plan(_dev(rowptr), _dev(colind), _dev(A.reshape(-1).copy()), 16, 16, N, dtype=W.SD_F32,
                   family=sd.SD_BSR_TC)
    Cd = torch.full((16, N), float("nan"), device="cuda")
    plan.spmm(_dev(B), Cd, 1.0, 0.0)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    err = np.abs(Cd.cpu().numpy().astype(np.float64) - want)
    # four tf32 products of exact halves, fp32 accumulation of 64 terms: a few 2^-24 of S
    assert np.all(err <= 1e-6 * S), float((err / S).max())
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_one_block_random_against_triple_loop(dtype):
    import paper_2608_05033_b200 as sd
    rng = np.random.default_rng(7 + dtype)
    rowptr, colind = _one_block_csr()
    A = rng.standard_normal((16, 16)).astype(np.float32)
    N = 256
    B = rng.standard_normal((16, N)).astype(np.float32)
    if dtype == W.SD_BF16:
        a_bits, b_bits = W.f32_to_bf16_bits(A.reshape(-1)), W.f32_to_bf16_bits(B).reshape(16, N)
        A, B = W.bf16_bits_to_f32(a_bits).reshape(16, 16), W.bf16_bits_to_f32(b_bits.reshape(-1)).reshape(16, N)
        a_dev, b_dev = _dev(a_bits), _dev(b_bits)
    else:
        a_dev, b_dev = _dev(A.reshape(-1).copy()), _dev(B)
    want = _triple_loop(A, B)
    S = _triple_loop(np.abs(A), np.abs(B))
    plan = sd.Plan(_dev(rowptr), _dev(colind), a_dev, 16, 16, N, dtype=dtype, family=sd.SD_BSR_TC)
    Cd = torch.full((16, N), float("nan"), device="cuda")
    plan.spmm(b_dev, Cd, 1.0, 0.0)
    torch.cuda.synchronize()
    err = np.abs(Cd.cpu().numpy().astype(np.float64) - want)
    assert np.all(err <= 1e-6 * S + 1e-7)       # bf16 products are exact in fp32; 16 fp32 additions
    plan.close()


@pytest.mark.parametrize("dtype", [W.SD_BF16, W.SD_F32])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(dtype):
    """The test-only plan option makes the first CTA's copy thread withhold its ring slots and shortens the spin
    limit, so the tensor-core issuer's wait for operands runs out.  Nothing may trap or spin forever: the kernel
    returns, the plan's device status is non-zero (and reads as zero again afterwards), and a fresh plan on the
    same inputs gives the right result."""
    import oracle
    import paper_2608_05033_b200 as sd
    w = W.g4_block(Mb=64, Kb=64, N=256, nblocks=200, dtype=dtype)
    rowptr, colind, vals, B = _dev(w.rowptr), _dev(w.colind), _dev(w.vals), _dev(w.B)
    bad = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, dtype=dtype, family=sd.SD_BSR_TC, test_wait_expiry=1)
    Cd = torch.zeros((w.M, w.N), device="cuda")
    bad.spmm(B, Cd, 1.0, 0.0)
    torch.cuda.synchronize()                      # returns: no wait is endless
    status = bad.device_status()
    assert status != 0, "the expired wait must be recorded"
    assert bad.device_status() == 0               # reading clears it
    bad.close()
    good = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, dtype=dtype, family=sd.SD_BSR_TC)
    Cd = torch.full((w.M, w.N), float("nan"), device="cuda")
    good.spmm(B, Cd, 1.0, 0.0)
    torch.cuda.synchronize()
    assert good.device_status() == 0
    assert oracle.check(w.rowptr, w.colind, w.vals, w.B, w.N, Cd.cpu().numpy(), None, 1.0, 0.0)["ok"]
    good.close()
