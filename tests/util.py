"""Helpers shared by the GPU parity tests: run a workload through the C-ABI binding and compare
with the oracle element by element.  Tolerances (per output element, relative to the sum of the
absolute values of its terms, S): 1e-4 for stages computed in fp32 arithmetic, 1e-3 for stages
that go through TF32 tensor-core products."""
import numpy as np

TOL_FP32 = 1e-4
TOL_TF32 = 1e-3


def fmt_of(sa, w):
    return sa.SA_FMT_CSR if w.fmt == "csr" else sa.SA_FMT_CSF


def run_gpu(sa, w, sched=None, tensor=None):
    """Returns (A as float64 numpy, SparseTensor)."""
    import torch
    t = tensor or sa.SparseTensor(w.dims, w.coords, w.vals, fmt_of(sa, w), device=0)
    ops = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in w.dense]
    out, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_DEFAULT if sched is None else sched)
    torch.cuda.synchronize()
    assert sa.sa_last_device_status(t.handle, torch.cuda.current_stream().cuda_stream) == sa.SA_OK
    return out.cpu().numpy().astype(np.float64), t


def assert_close(A_gpu, A_ref, S_ref, tol, what=""):
    assert A_gpu.shape == A_ref.shape, (A_gpu.shape, A_ref.shape)
    if A_ref.size == 0:
        return 0.0                       # an output without elements (sparse output of an empty tensor)
    assert np.isfinite(A_gpu).all(), what + ": non-finite output"
    err = np.abs(A_gpu - A_ref)
    # an element without terms must be exactly zero
    none = S_ref == 0
    assert not A_gpu[none].any(), what + ": element without terms is not +0"
    bound = tol * S_ref
    bad = err > bound
    if bad.any():
        worst = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError("%s: %d elements above %.0e*S; worst at %s: gpu %.9g ref %.9g S %.9g"
                             % (what, int(bad.sum()), tol, worst, A_gpu[worst], A_ref[worst], S_ref[worst]))
    with np.errstate(divide="ignore", invalid="ignore"):
        return float(np.nanmax(np.where(S_ref > 0, err / S_ref, 0.0)))
