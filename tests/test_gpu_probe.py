"""The gather replays of bench_probes (bench.py --probe / --probe-paths), used as measured ceilings,
must really fetch every row: the sink holds one partial sum per thread; with small integer table
entries the sums are exact in fp32, so the column sums of the gathered rows are checked bit for bit
against numpy, for every fetch path."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu


def _probes():
    import bench_probes
    bench_probes.build()
    return bench_probes


@pytest.mark.parametrize("row_bytes", [16, 32, 64, 128, 256, 512])
@pytest.mark.parametrize("count", [1, 4099, 200_001])
def test_plain_path_sums_any_row_size(row_bytes, count):
    bp = _probes()
    rng = np.random.default_rng(0x5D17 + row_bytes + count)
    rows, width = 777, row_bytes // 4
    table = rng.integers(-3, 4, size=(rows, width)).astype(np.float32)
    idx = rng.integers(0, rows, size=count).astype(np.int32)
    dev = torch.device("cuda:0")
    t, i = torch.from_numpy(table).to(dev), torch.from_numpy(idx).to(dev)
    sink = torch.zeros(bp.sink_floats(), dtype=torch.float32, device=dev)
    bp.gather(0, i, count, t, row_bytes, sink)
    torch.cuda.synchronize()
    s = sink.cpu().numpy().astype(np.float64).reshape(-1, 4)      # one float4 per thread
    lpr = row_bytes // 16
    got = s.reshape(-1, lpr, 4).sum(axis=0).reshape(width)         # thread t holds float4 slot t % lpr
    assert np.array_equal(got, table[idx].astype(np.float64).sum(axis=0))


@pytest.mark.parametrize("path", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13])
@pytest.mark.parametrize("count", [5, 70_003])
def test_every_512_byte_path_fetches_every_row(path, count):
    bp = _probes()
    rng = np.random.default_rng(0xABC + path + count)
    rows = 5000
    table = rng.integers(-3, 4, size=(rows, 128)).astype(np.float32)
    idx = rng.integers(0, rows, size=count).astype(np.int32)
    dev = torch.device("cuda:0")
    t = torch.from_numpy(table).to(dev)
    sink = torch.zeros(bp.sink_floats(), dtype=torch.float32, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    hub = None
    stream_idx = idx
    if path in bp.HUB_CLUSTER:   # the first CL * 256 rows of the table are the hub rows; their indices carry bit 31
        nh = bp.HUB_CLUSTER[path] * bp.HUB_ROWS_PER_CTA
        hub = torch.arange(nh, dtype=torch.int32, device=dev)
        stream_idx = np.where(idx < nh, idx.astype(np.int64) | 0x80000000, idx).astype(np.uint32).view(np.int32)
    i = torch.from_numpy(stream_idx).to(dev)
    bp.gather(path, i, count, t, 512, sink, err=err, hubrows=hub)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    s = sink.cpu().numpy().astype(np.float64).reshape(-1, 4)
    want = table[idx].astype(np.float64).sum(axis=0)
    if path == 6:    # two float4 per thread: columns (t % 16) * 4 and 64 + (t % 16) * 4
        s = s.reshape(-1, 16, 2, 4).sum(axis=0)                    # [lane in half warp][vector][4]
        got = np.concatenate([s[:, 0, :].reshape(64), s[:, 1, :].reshape(64)])
    else:
        got = s.reshape(-1, 32, 4).sum(axis=0).reshape(128)
    assert np.array_equal(got, want)


def test_bad_arguments_are_refused():
    bp = _probes()
    dev = torch.device("cuda:0")
    t = torch.zeros(64, dtype=torch.float32, device=dev)
    i = torch.zeros(4, dtype=torch.int32, device=dev)
    sink = torch.zeros(bp.sink_floats(), dtype=torch.float32, device=dev)
    with pytest.raises(RuntimeError):
        bp.gather(0, i, 4, t, 48, sink)          # row size not a power of two of 16 bytes
    with pytest.raises(RuntimeError):
        bp.gather(3, i, 4, t, 256, sink)         # the path variants take 512-byte rows only
