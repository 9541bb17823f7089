"""Python binding of the sparse-chain executor (``include/sparseauto.h``).

Argument marshalling only: every function forwards to the C-ABI entry point of the same
name in ``libsparseauto.so``; all arithmetic runs in the CUDA kernels.  PyTorch is used for
device memory and streams.  Importing this package fails loudly if the library has not been
built (``python paper_2311_09549_b200/build.py``); there is no CPU path.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPARSEAUTO_LIB selects another build of the same library (the self-checking one, libsparseauto_checked.so)
LIB_PATH = os.environ.get("SPARSEAUTO_LIB") or os.path.join(_HERE, "libsparseauto.so")

if not os.path.exists(LIB_PATH):
    raise ImportError("libsparseauto.so is missing: run `python paper_2311_09549_b200/build.py` "
                      "(needs nvcc; the library targets sm_100a and has no CPU fallback)")
_lib = ctypes.CDLL(LIB_PATH)

# ---- enums (values of include/sparseauto.h)
SA_OK = 0
(SA_E_ARG, SA_E_COORD_RANGE, SA_E_COORD_DUP, SA_E_FORMAT, SA_E_SHAPE, SA_E_UNSUPPORTED, SA_E_ALLOC,
 SA_E_WORKSPACE, SA_E_CUDA, SA_E_BOUNDS, SA_E_TIMEOUT) = range(1, 12)
SA_FMT_CSR, SA_FMT_CSF = 1, 2
SA_EXPR_SPTTM_TTM3, SA_EXPR_SPTTM_TTM4, SA_EXPR_SDDMM_SPMM, SA_EXPR_SPMM_GEMM, SA_EXPR_TTMC3, SA_EXPR_SDDMM_SPMM_GEMM = 1, 2, 3, 4, 5, 6
SA_EXPR_SPMMH_GEMM, SA_EXPR_MTTKRP_GEMM, SA_EXPR_SPTTM_SPTTM = 7, 8, 9
SA_SCHED_DEFAULT, SA_SCHED_FUSED, SA_SCHED_ASSOC_LEFT, SA_SCHED_ASSOC_RIGHT, SA_SCHED_FISSIONED = 0, 1, 2, 3, 4
SA_SCHED_DEBUG_MATERIALIZE = 9

EXPORTED_SYMBOLS = ["sa_tensor_create", "sa_tensor_info", "sa_tensor_export", "sa_tensor_worklist",
                    "sa_tensor_tasks", "sa_workspace_size", "sa_schedule_cost", "sa_tensor_set_aux_limit", "sa_run", "sa_last_launch_count", "sa_last_device_status", "sa_device_status_words",
                    "sa_destroy", "sa_status_string", "sa_run_ttm3_static_scratch"]


class SaDense(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("ld", ctypes.c_int64)]


_ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p)
_RELEASE_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class SaAllocator(ctypes.Structure):
    _fields_ = [("alloc", _ALLOC_FN), ("release", _RELEASE_FN), ("ctx", ctypes.c_void_p)]


_vp, _i64, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
_lib.sa_tensor_create.argtypes = [_int, _vp, _i64, _vp, _vp, _int, _int, ctypes.POINTER(SaAllocator), ctypes.POINTER(_vp)]
_lib.sa_tensor_info.argtypes = [_vp, ctypes.POINTER(_i64), _vp, ctypes.POINTER(_i64)]
_lib.sa_tensor_export.argtypes = [_vp, _int, _vp, _vp, _vp]
_lib.sa_tensor_worklist.argtypes = [_vp, _int, _vp, _vp, _vp]
_lib.sa_tensor_tasks.argtypes = [_vp, ctypes.POINTER(_i64), _vp, _vp]
_lib.sa_workspace_size.argtypes = [_vp, _int, _int, ctypes.POINTER(SaDense), _int, ctypes.POINTER(ctypes.c_size_t)]
class SaCost(ctypes.Structure):
    _fields_ = [("iterations", ctypes.c_double), ("moved_bytes", ctypes.c_double), ("temp_elements", ctypes.c_double),
                ("workspace_bytes", ctypes.c_size_t), ("resolved", ctypes.c_int)]


_lib.sa_schedule_cost.argtypes = [_vp, _int, _int, ctypes.POINTER(SaDense), _int, ctypes.POINTER(SaCost)]
_lib.sa_tensor_set_aux_limit.argtypes = [_vp, ctypes.c_size_t]
_lib.sa_run.argtypes = [_vp, _int, _int, ctypes.POINTER(SaDense), _int, _vp, _vp, ctypes.c_size_t, _vp]
_lib.sa_last_launch_count.argtypes = [_vp, ctypes.POINTER(_int)]
_lib.sa_last_device_status.argtypes = [_vp, _vp]
_lib.sa_device_status_words.argtypes = [_vp, _vp, _vp]
_lib.sa_destroy.argtypes = [_vp]
_lib.sa_destroy.restype = None
_lib.sa_status_string.argtypes = [_int]
_lib.sa_status_string.restype = ctypes.c_char_p
_lib.sa_run_ttm3_static_scratch.argtypes = [_vp, ctypes.POINTER(SaDense), _int, _vp, _vp]
for _n in EXPORTED_SYMBOLS:
    if _n not in ("sa_destroy", "sa_status_string"):
        getattr(_lib, _n).restype = _int


class SaError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, sa_status_string(status), status))


def _check(status, where):
    if status != SA_OK:
        raise SaError(status, where)


def sa_status_string(status):
    return _lib.sa_status_string(int(status)).decode()


class TorchAllocator:
    """sa_allocator backed by torch: device arrays of a tensor handle are torch allocations."""

    def __init__(self, device):
        import torch
        self._torch = torch
        self.device = torch.device("cuda", device)
        self.live = {}
        self._alloc = _ALLOC_FN(self._do_alloc)
        self._release = _RELEASE_FN(self._do_release)
        self.struct = SaAllocator(self._alloc, self._release, None)

    def _do_alloc(self, nbytes, _ctx):
        try:
            buf = self._torch.empty(max(int(nbytes), 1), dtype=self._torch.uint8, device=self.device)
        except Exception:
            return None
        self.live[buf.data_ptr()] = buf
        return buf.data_ptr()

    def _do_release(self, ptr, _ctx):
        self.live.pop(ptr, None)


def sa_tensor_create(order, dims, nnz, coords, vals, fmt, device, dev_alloc=None):
    """coords: int32 host array [nnz, order]; vals: float32 host array [nnz].  Returns the handle (int)."""
    dims_a = np.ascontiguousarray(dims, dtype=np.int64)
    coords_a = np.ascontiguousarray(coords, dtype=np.int32)
    vals_a = np.ascontiguousarray(vals, dtype=np.float32)
    handle = _vp()
    st = _lib.sa_tensor_create(int(order), dims_a.ctypes.data, int(nnz), coords_a.ctypes.data, vals_a.ctypes.data,
                               int(fmt), int(device), ctypes.byref(dev_alloc) if dev_alloc is not None else None,
                               ctypes.byref(handle))
    _check(st, "sa_tensor_create")
    return handle.value


def sa_tensor_info(handle, order):
    nnz, chunks = _i64(), _i64()
    counts = np.zeros(order, dtype=np.int64)
    _check(_lib.sa_tensor_info(handle, ctypes.byref(nnz), counts.ctypes.data, ctypes.byref(chunks)), "sa_tensor_info")
    return nnz.value, counts, chunks.value


def sa_tensor_export(handle, level, n_pos=0, n_crd=0, n_vals=0):
    """Returns (pos int64 | None, crd int32 | None, vals float32 | None) for the sizes given (0 = skip)."""
    pos = np.empty(n_pos, dtype=np.int64) if n_pos else None
    crd = np.empty(n_crd, dtype=np.int32) if n_crd else None
    vals = np.empty(n_vals, dtype=np.float32) if n_vals else None
    st = _lib.sa_tensor_export(handle, int(level), pos.ctypes.data if n_pos else None,
                               crd.ctypes.data if n_crd else None, vals.ctypes.data if n_vals else None)
    _check(st, "sa_tensor_export")
    return pos, crd, vals


def sa_tensor_worklist(handle, which=0):
    counts = np.zeros(4, dtype=np.int64)
    _check(_lib.sa_tensor_worklist(handle, int(which), counts.ctypes.data, None, None), "sa_tensor_worklist")
    items = np.zeros((int(counts[0]), 8), dtype=np.int32)
    fix = np.zeros((int(counts[2]), 4), dtype=np.int32)
    _check(_lib.sa_tensor_worklist(handle, int(which), None, items.ctypes.data, fix.ctypes.data), "sa_tensor_worklist")
    return counts, items, fix


def sa_tensor_tasks(handle):
    """Order-3 CSF: (task_start int32 [n_tasks + 1], stream_f0 int32 [n_items, 4])."""
    n = _i64()
    _check(_lib.sa_tensor_tasks(handle, ctypes.byref(n), None, None), "sa_tensor_tasks")
    counts = np.zeros(4, dtype=np.int64)
    _check(_lib.sa_tensor_worklist(handle, 0, counts.ctypes.data, None, None), "sa_tensor_worklist")
    task_start = np.zeros(n.value + 1, dtype=np.int32)
    stream_f0 = np.zeros((int(counts[0]), 4), dtype=np.int32)
    _check(_lib.sa_tensor_tasks(handle, None, task_start.ctypes.data, stream_f0.ctypes.data), "sa_tensor_tasks")
    return task_start, stream_f0


def _dense_array(ops):
    arr = (SaDense * len(ops))()
    for i, (ptr, rows, cols, ld) in enumerate(ops):
        arr[i] = SaDense(ptr, rows, cols, ld)
    return arr


def sa_workspace_size(handle, expr, sched, ops):
    """ops: list of (ptr, rows, cols, ld); only the shapes are read."""
    n = ctypes.c_size_t()
    _check(_lib.sa_workspace_size(handle, int(expr), int(sched), _dense_array(ops), len(ops), ctypes.byref(n)),
           "sa_workspace_size")
    return n.value


def sa_schedule_cost(handle, expr, sched, ops):
    """ops: list of (ptr, rows, cols, ld); only the shapes are read.  Returns a dict of the sa_cost fields."""
    c = SaCost()
    _check(_lib.sa_schedule_cost(handle, int(expr), int(sched), _dense_array(ops), len(ops), ctypes.byref(c)), "sa_schedule_cost")
    return {"iterations": c.iterations, "moved_bytes": c.moved_bytes, "temp_elements": c.temp_elements,
            "workspace_bytes": int(c.workspace_bytes), "resolved": int(c.resolved)}


def sa_tensor_set_aux_limit(handle, nbytes):
    _check(_lib.sa_tensor_set_aux_limit(handle, int(nbytes)), "sa_tensor_set_aux_limit")


def sa_run(handle, expr, sched, ops, out_ptr, workspace_ptr, workspace_bytes, stream):
    st = _lib.sa_run(handle, int(expr), int(sched), _dense_array(ops), len(ops), out_ptr, workspace_ptr,
                     int(workspace_bytes), stream)
    _check(st, "sa_run")


def sa_run_ttm3_static_scratch(handle, ops, out_ptr, stream):
    """The order-3 <SpTTM,TTM> chain with the library's built-in 4 MiB scratch instead of a workspace:
    for callers that cannot allocate device memory.  Raises SaError(SA_E_WORKSPACE) if the tensor
    needs more scratch than that."""
    st = _lib.sa_run_ttm3_static_scratch(handle, _dense_array(ops), len(ops), out_ptr, stream)
    _check(st, "sa_run_ttm3_static_scratch")


def sa_last_launch_count(handle):
    n = _int()
    _check(_lib.sa_last_launch_count(handle, ctypes.byref(n)), "sa_last_launch_count")
    return n.value


def sa_last_device_status(handle, stream):
    return int(_lib.sa_last_device_status(handle, stream))


def sa_device_status_words(handle, stream):
    words = np.zeros(4, dtype=np.int32)
    _check(_lib.sa_device_status_words(handle, stream, words.ctypes.data), "sa_device_status_words")
    return words


def sa_destroy(handle):
    _lib.sa_destroy(handle)


# ------------------------------------------------------------------ convenience wrapper

_EXPR_OF = {"spttm_ttm3": SA_EXPR_SPTTM_TTM3, "spttm_ttm4": SA_EXPR_SPTTM_TTM4,
            "sddmm_spmm": SA_EXPR_SDDMM_SPMM, "spmm_gemm": SA_EXPR_SPMM_GEMM, "ttmc3": SA_EXPR_TTMC3, "sddmm_spmm_gemm": SA_EXPR_SDDMM_SPMM_GEMM,
            "spmmh_gemm": SA_EXPR_SPMMH_GEMM, "mttkrp_gemm": SA_EXPR_MTTKRP_GEMM,
            "spttm_spttm": SA_EXPR_SPTTM_SPTTM}


class SparseTensor:
    """Owns a handle; device arrays come from torch through :class:`TorchAllocator`."""

    def __init__(self, dims, coords, vals, fmt, device=0):
        self.dims = tuple(int(d) for d in dims)
        self.order = len(self.dims)
        self.device = device
        self._allocator = TorchAllocator(device) if device >= 0 else None
        self.handle = sa_tensor_create(self.order, self.dims, len(vals), coords, vals, fmt, device,
                                       self._allocator.struct if self._allocator else None)
        self._ws = None

    def close(self):
        if self.handle:
            sa_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def info(self):
        return sa_tensor_info(self.handle, self.order)

    def run(self, expr, operands, out=None, sched=SA_SCHED_DEFAULT, stream=None, workspace=None):
        """operands: torch float32 CUDA matrices (row-major).  Returns (out, workspace)."""
        import torch
        expr = _EXPR_OF.get(expr, expr)
        ops = [(t.data_ptr(), t.shape[0], t.shape[1], t.stride(0)) for t in operands]
        need = sa_workspace_size(self.handle, expr, sched, ops)
        dev = torch.device("cuda", self.device)
        if workspace is None:
            if self._ws is None or self._ws.numel() < need:
                self._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
            workspace = self._ws
        if out is None:
            out = torch.empty(self.out_shape(expr, operands), dtype=torch.float32, device=dev)
        s = torch.cuda.current_stream(dev) if stream is None else stream
        sa_run(self.handle, expr, sched, ops, out.data_ptr(), workspace.data_ptr(), workspace.numel(), s.cuda_stream)
        return out, workspace

    def out_shape(self, expr, operands):
        expr = _EXPR_OF.get(expr, expr)
        cols = [int(t.shape[1]) for t in operands]
        if expr == SA_EXPR_SPTTM_TTM3:
            return (self.dims[0], cols[0], cols[1])
        if expr == SA_EXPR_SPTTM_TTM4:
            return (self.dims[0], cols[0], cols[1], cols[2])
        if expr == SA_EXPR_SDDMM_SPMM:
            return (self.dims[0], cols[2])
        if expr == SA_EXPR_SDDMM_SPMM_GEMM:
            return (self.dims[0], cols[3])
        if expr == SA_EXPR_TTMC3:
            return (cols[0], cols[1], cols[2])
        if expr in (SA_EXPR_SPMMH_GEMM, SA_EXPR_MTTKRP_GEMM):
            return (self.dims[0], cols[2])
        if expr == SA_EXPR_SPTTM_SPTTM:
            return (int(self.info()[1][1]), cols[1])      # one row per (i,j) fiber, in CSF order
        return (self.dims[0], cols[1])
