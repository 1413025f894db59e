"""sd_probe_gather: the gather replay used as a measured ceiling must really fetch every row.

The sink holds one partial sum per thread; with small integer table entries the sums are exact in
fp32, so the column sums of the gathered rows are checked bit for bit against numpy."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("row_bytes", [16, 32, 64, 128, 256, 512])
@pytest.mark.parametrize("count", [0, 1, 4099, 200_001])
def test_probe_gather_sums(row_bytes, count):
    import paper_2608_05033_b200 as sd
    rng = np.random.default_rng(0x5D17 + row_bytes + count)
    rows, width = 777, row_bytes // 4
    table = rng.integers(-3, 4, size=(rows, width)).astype(np.float32)
    idx = rng.integers(0, rows, size=count).astype(np.int32)
    dev = torch.device("cuda:0")
    t = torch.from_numpy(table).to(dev)
    i = torch.from_numpy(idx).to(dev) if count else torch.zeros(1, dtype=torch.int32, device=dev)
    need = sd.sd_probe_gather(None, 0, None, row_bytes)
    assert need > 0 and need % 4 == 0
    sink = torch.full((need,), float("nan"), dtype=torch.float32, device=dev)
    sd.sd_probe_gather(i, count, t, row_bytes, sink)
    torch.cuda.synchronize()
    s = sink.cpu().numpy().astype(np.float64).reshape(-1, 4)      # one float4 per thread
    lpr = row_bytes // 16
    got = s.reshape(-1, lpr, 4).sum(axis=0).reshape(width)         # thread t holds float4 slot t % lpr
    want = table[idx].astype(np.float64).sum(axis=0) if count else np.zeros(width)
    assert np.array_equal(got, want)


def test_probe_gather_rejects_bad_row_bytes():
    import paper_2608_05033_b200 as sd
    dev = torch.device("cuda:0")
    t = torch.zeros(64, dtype=torch.float32, device=dev)
    i = torch.zeros(4, dtype=torch.int32, device=dev)
    sink = torch.zeros(sd.sd_probe_gather(None, 0, None, 16), dtype=torch.float32, device=dev)
    with pytest.raises(sd.SdError):
        sd.sd_probe_gather(i, 4, t, 48, sink)
