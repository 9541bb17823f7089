"""The self-checking build (-DSA_DEBUG_BOUNDS, libsparseauto_checked.so) on the mini configurations and the edge
tensors: every index that the kernels take out of the tensor's arrays or work lists is checked on the device
before it becomes an address.  The run must leave the status word at SA_OK (no check fired) and agree with the
oracle like the normal build.  It stands in for a memory checker on the small cases; nothing here can fault: a
failing check records its number and redirects the access.

The binding loads one library per process, so the checked one runs in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
import numpy as np
import torch
import oracle
import paper_2311_09549_b200 as sa
from workloads import configs
from util import TOL_FP32, assert_close, fmt_of

assert sa.LIB_PATH.endswith("libsparseauto_checked.so"), sa.LIB_PATH
stream = torch.cuda.current_stream().cuda_stream


def check(w, sched=None):
    t = sa.SparseTensor(w.dims, w.coords, w.vals, fmt_of(sa, w), device=0)
    ops = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in w.dense]
    out, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_DEFAULT if sched is None else sched)
    torch.cuda.synchronize()
    words = sa.sa_device_status_words(t.handle, stream)
    assert words[0] == sa.SA_OK, "%s: check %d fired on value %d (thread %d)" % (w.name, words[1], words[2], words[3])
    A_ref, S_ref = oracle.evaluate(w)
    assert_close(out.cpu().numpy().astype(np.float64), A_ref, S_ref, TOL_FP32, w.name + " (checked build)")
    t.close()


for cfg in range(1, 11):
    w = configs.make(cfg, "mini")
    if w.expr in ("spmm_gemm", "spttm_spttm"):
        check(w, sa.SA_SCHED_ASSOC_LEFT)
        check(w, sa.SA_SCHED_ASSOC_RIGHT)
    elif w.expr in ("spttm_ttm4", "ttmc3"):
        check(w, sa.SA_SCHED_FUSED)
        check(w, sa.SA_SCHED_FISSIONED)
    else:
        check(w)
# edge tensors: large (i,j) subtrees and split slices of the order-4 chain, long fibers of the order-3 chain
for s4 in (sa.SA_SCHED_FUSED, sa.SA_SCHED_FISSIONED):
    check(configs.make_ttm4_zipf("edge4", 31, 90, 6, 130, 110, 150_000, 1.4, 5.0, 16, 16, 16), s4)
    check(configs.make_ttm4_zipf("edge4b", 32, 90, 700, 50, 45, 150_000, 1.4, 5.0, 16, 16, 16), s4)
check(configs.make_ttm3_zipf("edge3", 41, 50, 40, 3000, 120_000, 1.4, 300.0, 32, 16))
check(configs.make_ttm3_zipf("edge3b", 42, 700, 300, 40, 60_000, 1.0, 2.0, 16, 32))
print("CHECKED-OK")
"""


def test_checked_build_runs_clean_and_agrees_with_the_oracle():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_sa_build", os.path.join(ROOT, "paper_2311_09549_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    lib = mod.build_checked()
    env = dict(os.environ, SPARSEAUTO_LIB=lib,
               PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests"), os.environ.get("PYTHONPATH", "")]))
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "CHECKED-OK" in r.stdout, r.stdout[-2000:] + "\n" + r.stderr[-4000:]


def test_random_sweep_under_the_checked_build():
    """The randomised shapes of test_gpu_random.py once more with every device-side index check compiled in (its
    helper asserts that the status word stays SA_OK after each run)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("_sa_build", os.path.join(ROOT, "paper_2311_09549_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    lib = mod.build_checked()
    env = dict(os.environ, SPARSEAUTO_LIB=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_random.py"), "-x", "-q", "-m", "gpu",
                        "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and " passed" in r.stdout, r.stdout[-3000:] + "\n" + r.stderr[-2000:]
