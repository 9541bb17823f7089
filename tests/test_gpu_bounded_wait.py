"""The bounded device-side waits of the tcgen05 dense stage.  A test library (built with -DSA_TEST_HOOKS and a
2 ms limit instead of 2 s) lets one arrival of the first operand hand-off stay away: the product warp's wait has
to run out, every role has to leave its loop, tensor memory has to be released and the status word has to read
SA_E_TIMEOUT -- after which the same handle must run normally again.  No wait in the kernel is unbounded, with or
without the hook, so nothing here can hang.  Runs in a child process (the binding loads one library per process)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import ctypes
import time
import numpy as np
import torch
import oracle
import paper_2311_09549_b200 as sa
from workloads import configs
from util import TOL_FP32, assert_close

assert sa.LIB_PATH.endswith("libsparseauto_waittest.so"), sa.LIB_PATH
hook = sa._lib.sa_test_set_status_word
hook.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_void_p]
hook.restype = ctypes.c_int
stream = torch.cuda.current_stream().cuda_stream

w = configs.make(4, "mini")                      # <SpMM,GEMM> as B.(C.D): the dense stage runs first
A_ref, S_ref = oracle.evaluate(w)
t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSR, device=0)
ops = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in w.dense]


def run():
    out, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_ASSOC_RIGHT)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


assert_close(run(), A_ref, S_ref, TOL_FP32, "before the hook")
assert sa.sa_last_device_status(t.handle, stream) == sa.SA_OK
# arm the hook: the next dense-stage launch loses one arrival
assert hook(t.handle, 3, 0x7e57, stream) == sa.SA_OK
t0 = time.perf_counter()
run()                                            # returns: every wait is bounded (a few ms here)
dt = time.perf_counter() - t0
assert dt < 5.0, "the kernel must give up after milliseconds, took %.2f s" % dt
assert sa.sa_last_device_status(t.handle, stream) == sa.SA_E_TIMEOUT       # also clears the words, hook included
assert sa.sa_last_device_status(t.handle, stream) == sa.SA_OK
# the context, tensor memory and the handle are intact
assert_close(run(), A_ref, S_ref, TOL_FP32, "after the time-out")
assert sa.sa_last_device_status(t.handle, stream) == sa.SA_OK
print("WAIT-OK %.4f" % dt)
"""


def test_dense_stage_wait_runs_out_and_the_handle_recovers():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_sa_build", os.path.join(ROOT, "paper_2311_09549_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    lib = mod.build_waittest()
    env = dict(os.environ, SPARSEAUTO_LIB=lib,
               PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests"), os.environ.get("PYTHONPATH", "")]))
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "WAIT-OK" in r.stdout, r.stdout[-2000:] + "\n" + r.stderr[-4000:]
