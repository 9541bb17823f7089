"""The measurement aid of bench.py (paper_2311_09549_b200/probe): both gather families must read the rows they
are asked for, otherwise the "ceiling of the access pattern" in the bench line measures something else."""
import ctypes
import os

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _lib():
    from paper_2311_09549_b200 import build
    lib = ctypes.CDLL(build.build_probe())
    vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    lib.sa_probe_tma_gather.argtypes = [vp, i64, i64, ci, vp, i64, vp, ci, ci, vp, vp]
    lib.sa_probe_tma_gather.restype = ci
    lib.sa_probe_row_gather.argtypes = [vp, i64, i64, ci, vp, i64, vp, ci, ci, ci, vp]
    lib.sa_probe_row_gather.restype = ci
    return lib


@pytest.mark.parametrize("cols,ld", [(32, 32), (16, 16), (32, 40)])
def test_copy_engine_gather_reads_the_named_rows(cols, ld):
    import torch
    assert torch.cuda.is_available()
    lib = _lib()
    rows, n = 5000, 1 << 18
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    full = torch.rand(rows, ld, device="cuda", generator=g)
    table = full[:, :cols]
    idx = torch.randint(0, rows, (n,), dtype=torch.int32, device="cuda", generator=g)
    stream = torch.cuda.current_stream().cuda_stream
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for stages, bps in ((1, 1), (3, 2), (8, 1)):
        sink = torch.zeros(2, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        rc = lib.sa_probe_tma_gather(table.data_ptr(), rows, ld, cols, idx.data_ptr(), n, sink.data_ptr(), stages, bps,
                                     status.data_ptr(), stream)
        assert rc == 0
        torch.cuda.synchronize()
        assert int(status[0]) == 0, "a wait for landed rows gave up"
        warps = sms * bps * 4
        per = (n // warps) // 16 * 16               # every warp reads a contiguous share, a multiple of 16 rows
        sel = idx[:warps * per].long()
        want = float(table[sel].double().sum())
        assert abs(float(sink[1]) - want) <= 1e-4 * want, (stages, bps, float(sink[1]), want)


def test_probe_rejects_bad_arguments():
    import torch
    lib = _lib()
    t = torch.zeros(64, 32, device="cuda")
    idx = torch.zeros(64, dtype=torch.int32, device="cuda")
    sink = torch.zeros(2, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert lib.sa_probe_tma_gather(t.data_ptr(), 64, 32, 32, idx.data_ptr(), 64, sink.data_ptr(), 0, 1, status.data_ptr(), s) == 1
    assert lib.sa_probe_tma_gather(t.data_ptr(), 64, 32, 24, idx.data_ptr(), 64, sink.data_ptr(), 2, 1, status.data_ptr(), s) == 1
    assert lib.sa_probe_tma_gather(t.data_ptr(), 64, 30, 32, idx.data_ptr(), 64, sink.data_ptr(), 2, 1, status.data_ptr(), s) == 1
    assert lib.sa_probe_row_gather(t.data_ptr(), 64, 32, 32, idx.data_ptr(), 64, sink.data_ptr(), 5, 8, 4, s) != 0
    torch.cuda.synchronize()
