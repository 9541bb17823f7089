#!/usr/bin/env python
"""Throughput benchmark of the sparse contraction-chain executor.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--sched left|right]
    python bench.py --impl reference ...        # the CPU oracle on a bounded sample

One "step" is one pass of the whole hot path (sa_run: main kernel(s) + fix-up) over the
synthetic workload.  Default workload: config 2, the order-3 <SpTTM,TTM> chain at scale.
Prints ONE JSON line (rank 0).  With N > 1 (torchrun, one rank per GPU) every rank runs an
independent replica of the same workload -- the path has no exchange step -- and `value`
is the aggregate over ranks, timed as the max over ranks.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import configs  # noqa: E402

METRIC = "GNNZ/s and achieved HBM GB/s (% of ~8 TB/s) per sparse contraction chain"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# DRAM bytes (read + write) of one launch of the dominant kernel, from the ncu captures summarised under
# profiles/ (keyed by workload, or by (workload, schedule that ran)).  A figure is reported only while the kernel's
# source file still has the hash it had when the counters were taken; otherwise `traffic` is null.  Workloads 4 and 5
# are captured at a quarter of their size (--scale mid) and scaled by the nonzeros, see the profiles.
NCU_TRAFFIC = {
    2: {"kernel": "ttm3_kernel<32,32> (98.4 % of the step)", "source": "paper_2311_09549_b200/csrc/sa_ttm3.cu",
        "sha256": "16c36b6ee33b033d0b7e55b20c3ade065a6d5b28ef4f8267395b734b4ada9f3f",
        "dram_bytes": 853618688, "profile": "profiles/ttm3_kernel_cfg2.md"},
    3: {"kernel": "sddmm_spmm_kernel<64,64> (99.6 % of the step)", "source": "paper_2311_09549_b200/csrc/sa_sddmm_spmm.cu",
        "sha256": "7c9971e0e72e49dfbb4404b68def327568372ea956767048b5d3d830810b8ead",
        "dram_bytes": 13186066944, "profile": "profiles/sddmm_spmm_kernel_cfg3.md"},
    (4, "left"): {"kernel": "spmm_gemm_left_kernel<256,64> (the whole step; counters of the quarter-size case x 4)",
                  "source": "paper_2311_09549_b200/csrc/sa_spmm_gemm.cu", "sha256": "4cbda937e034c9869d74f7b8d341eab99531152e31ca898c803c7cd6cecf2622",
                  "dram_bytes": 4 * 24086787584, "profile": "profiles/spmm_gemm_kernels_cfg4.md"},
    (4, "right"): {"kernel": "spmm_kernel<2> (85 % of the step; counters of the quarter-size case x 4)",
                   "source": "paper_2311_09549_b200/csrc/sa_spmm_gemm.cu", "sha256": "4cbda937e034c9869d74f7b8d341eab99531152e31ca898c803c7cd6cecf2622",
                   "dram_bytes": 4 * 4974276864, "profile": "profiles/spmm_gemm_kernels_cfg4.md"},
    (5, "fused"): {"kernel": "ttm4_fused_kernel (94 % of the step; counters of the quarter-size case x 4)",
                   "source": "paper_2311_09549_b200/csrc/sa_ttm4.cu", "sha256": "77b9b58137c8e565f84a5ffd8762e5448c910f5befc50c3838442ae6007d0823",
                   "dram_bytes": 4 * 424084480, "profile": "profiles/ttm4_kernels_cfg5.md"},
    (5, "fissioned"): {"kernel": "ttm4_subtree_kernel (pass 1 on the small subtrees, 51 % of the step; counters of the "
                                 "quarter-size case x 4)",
                       "source": "paper_2311_09549_b200/csrc/sa_ttm4_fis.cu", "sha256": "be9575594a14a3633f6a12fba75381f08305534e694d350516c738ba12c2d61b",
                       "dram_bytes": 4 * 663252480, "profile": "profiles/ttm4_kernels_cfg5.md"},
    10: {"kernel": "fiber_spmm_kernel<32> (98 % of the step)", "source": "paper_2311_09549_b200/csrc/sa_spmm_gemm.cu",
         "sha256": "4cbda937e034c9869d74f7b8d341eab99531152e31ca898c803c7cd6cecf2622",
         "dram_bytes": 960941824, "profile": "profiles/fiber_spmm_kernel_w10.md"},
}


def ncu_traffic(workload, sched=None):
    import hashlib
    e = NCU_TRAFFIC.get((workload, sched)) or NCU_TRAFFIC.get(workload)
    if e is None:
        return None, None
    try:
        with open(os.path.join(ROOT, e["source"]), "rb") as f:
            same = hashlib.sha256(f.read()).hexdigest() == e["sha256"]
    except OSError:
        same = False
    return (e["dram_bytes"] if same else None), e["kernel"]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


def algorithmic_work(w, counts, sched):
    """(bytes, flops) one step must move / compute under the schedule that runs: streams of
    B's index and value arrays once, dense operands once (or one row per nonzero where the
    table exceeds L2), the output once."""
    nnz = w.nnz
    sz = lambda a: a.size * 4  # noqa: E731
    out_bytes = int(np.prod(w.out_shape)) * 4
    if w.expr == "spttm_ttm3":
        S, F2 = int(counts[0]), int(counts[1])
        L, M = w.dense[0].shape[1], w.dense[1].shape[1]
        return 8 * nnz + 8 * F2 + 8 * S + sz(w.dense[0]) + sz(w.dense[1]) + out_bytes, 2 * nnz * M + 2 * F2 * L * M
    if w.expr == "ttmc3":
        # the streams, the factors and the output (the slice temporaries T(i,m,n) of the fissioned schedule are
        # traffic, not algorithmic bytes: 8 I M N more)
        S, F2 = int(counts[0]), int(counts[1])
        L, M, N = (d.shape[1] for d in w.dense)
        return (8 * nnz + 8 * F2 + 8 * S + sum(sz(d) for d in w.dense) + out_bytes,
                2 * nnz * N + 2 * F2 * M * N + 2 * w.dims[0] * L * M * N)
    if w.expr == "spttm_ttm4":
        # what the method must move: the same for both schedules (the temporaries that the fissioned schedule sends
        # through the workspace are traffic, not algorithmic bytes)
        S, F2, F3 = int(counts[0]), int(counts[1]), int(counts[2])
        L, M, N = (d.shape[1] for d in w.dense)
        b = 8 * nnz + 8 * F3 + 8 * F2 + 8 * S + sum(sz(d) for d in w.dense) + out_bytes
        return b, 2 * (nnz * N + F3 * M * N + F2 * L * M * N)
    if w.expr == "sddmm_spmm_gemm":
        # the row temporaries T(i,:) that pass through the workspace are not counted
        I = w.dims[0]
        K, L, M = w.dense[0].shape[1], w.dense[2].shape[1], w.dense[3].shape[1]
        return (8 * nnz + 4 * (I + 1) + 4 * (K + L) * nnz + sz(w.dense[0]) + sz(w.dense[3]) + out_bytes,
                nnz * (2 * K + 1 + 2 * L) + 2 * I * L * M)
    if w.expr == "sddmm_spmm":
        I = w.dims[0]
        K, L = w.dense[0].shape[1], w.dense[2].shape[1]
        return 8 * nnz + 4 * (I + 1) + 4 * (K + L) * nnz + sz(w.dense[0]) + out_bytes, nnz * (2 * K + 1 + 2 * L)
    if w.expr == "mttkrp_gemm":
        # the rows T(i,:) that pass through the workspace are not counted
        S, F2 = int(counts[0]), int(counts[1])
        R, M = w.dense[0].shape[1], w.dense[2].shape[1]
        return (8 * nnz + 8 * F2 + 8 * S + sum(sz(d) for d in w.dense) + out_bytes,
                2 * nnz * R + 2 * F2 * R + 2 * w.dims[0] * R * M)
    if w.expr == "spttm_spttm":
        # fibers as rows: index/value streams, one pos entry per fiber, the output (one row per fiber) once;
        # (B'.C).D gathers a row of C per nonzero (C once: it fits L2), B'.(C.D) reads C and D once
        F2, K = int(counts[1]), w.dims[2]
        L, M = w.dense[0].shape[1], w.dense[1].shape[1]
        base = 8 * nnz + 4 * (F2 + 1) + sz(w.dense[0]) + sz(w.dense[1]) + out_bytes
        if sched == "left":
            return base, 2 * nnz * L + 2 * F2 * L * M
        return base, 2 * K * L * M + 2 * nnz * M
    if w.expr == "spmmh_gemm":
        # two gathered rows of L floats per nonzero (C and its Hadamard partner), E once, the output once
        I, J = w.dims
        L, M = w.dense[0].shape[1], w.dense[2].shape[1]
        return 8 * nnz + 4 * (I + 1) + 8 * L * nnz + sz(w.dense[2]) + out_bytes, 3 * nnz * L + 2 * I * L * M
    if w.expr == "spmm_gemm":
        I, J = w.dims
        L, M = w.dense[0].shape[1], w.dense[1].shape[1]
        if sched == "left":
            return 8 * nnz + 4 * (I + 1) + 4 * L * nnz + sz(w.dense[1]) + out_bytes, 2 * nnz * L + 2 * I * L * M
        e_bytes = J * M * 4
        return (sz(w.dense[0]) + e_bytes) + (8 * nnz + 4 * (I + 1) + 4 * M * nnz + out_bytes), 2 * J * L * M + 2 * nnz * M
    raise ValueError(w.expr)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def _oracle_run(w, counts, order, target_nnz, cores):
    """Evaluate the oracle on seeded random slices / rows holding about target_nnz nonzeros."""
    import oracle
    # the oracle gives one slice to one thread: leave out slices that alone would occupy a thread for
    # a large part of the run, so that the sample stays bounded
    cap = max(1, target_nnz // (2 * cores))
    order = order[counts[order] <= cap]
    csum = np.cumsum(counts[order])
    n_take = int(np.searchsorted(csum, min(target_nnz, int(csum[-1])), side="left")) + 1
    sel = np.sort(order[:n_take])
    nnz_sel = int(counts[sel].sum())
    t0 = time.perf_counter()
    oracle.evaluate(w, sel=sel, with_abs=False)
    return nnz_sel, time.perf_counter() - t0, len(sel), cap


def oracle_sample(w, budget_s=15.0):
    """Time the oracle, as it stands, on a bounded sample of output slices / rows of ``w``: a short
    pilot run measures its speed on this host, the timed run is sized to take about budget_s."""
    import oracle
    I = w.dims[0]
    per_nnz = {"spttm_ttm3": lambda: w.dense[0].shape[1] * w.dense[1].shape[1],
               "spttm_ttm4": lambda: w.dense[0].shape[1] * w.dense[1].shape[1] * w.dense[2].shape[1],
               "sddmm_spmm": lambda: w.dense[0].shape[1] * w.dense[2].shape[1],
               "spmm_gemm": lambda: w.dense[0].shape[1] * w.dense[1].shape[1],
               "spmmh_gemm": lambda: w.dense[0].shape[1] * w.dense[2].shape[1],
               "mttkrp_gemm": lambda: w.dense[0].shape[1] * w.dense[2].shape[1],
               "spttm_spttm": lambda: w.dense[0].shape[1] * w.dense[1].shape[1],
               "sddmm_spmm_gemm": lambda: w.dense[0].shape[1] * w.dense[2].shape[1] * w.dense[3].shape[1],
               "ttmc3": lambda: w.dense[0].shape[1] * w.dense[1].shape[1] * w.dense[2].shape[1]}[w.expr]()
    cores = oracle.max_threads()
    if w.expr == "ttmc3":
        # every output element sums over all nonzeros: sample output elements instead of slices
        n_out = int(np.prod(w.out_shape))
        order = configs.rng.permutation(w.seed, 77, n_out)

        def run(n_el):
            sel = np.sort(order[:max(1, min(n_out, n_el))])
            t0 = time.perf_counter()
            oracle.evaluate(w, sel=sel, with_abs=False)
            return len(sel), time.perf_counter() - t0
        n0, t0 = run(cores)
        n1, dt = run(int(n0 / max(t0, 1e-3) * budget_s))
        sample = "%d of %d output elements (seeded random), each over all %d nonzeros" % (n1, n_out, w.nnz)
        return {"value": w.nnz * (n1 / n_out) / dt / 1e9, "unit": "GNNZ/s", "cores": cores, "kind": "oracle",
                "sample": sample, "seconds": dt}
    if w.expr == "spttm_spttm":
        # the output rows are B's (i,j) fibers: sample fibers instead of slices
        _, inv = oracle.fiber_keys(w.coords, w.dims)
        counts = np.bincount(inv)
        I = counts.shape[0]
    else:
        counts = np.bincount(w.coords[:, 0], minlength=I)
    order = configs.rng.permutation(w.seed, 77, I)
    pilot_nnz = max(1000, int(0.5 * 0.25e9 * cores / per_nnz))          # ~0.5 s at a guessed rate
    n0, t0, _, _ = _oracle_run(w, counts, order, pilot_nnz, cores)
    rate = n0 / max(t0, 1e-3)
    nnz_sel, dt, n_sel, cap = _oracle_run(w, counts, order, max(pilot_nnz, int(rate * budget_s)), cores)
    sample = ("%d of %d output slices/rows (seeded random among those with <= %d nonzeros), %d of %d nonzeros"
              % (n_sel, I, cap, nnz_sel, w.nnz))
    return {"value": nnz_sel / dt / 1e9, "unit": "GNNZ/s", "cores": cores, "kind": "oracle", "sample": sample,
            "seconds": dt}


def reduce_max_over_ranks(values, device, world):
    """Element-wise maximum of ``values`` over all ranks (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def l2_gather_ceiling(sa, torch, w, tensor, ops, dev, stream):
    """For the TTM chains: time bare gathers of one factor row per nonzero (the rows the fiber stage reads, from
    the same L2-resident table) with the probe kernels of paper_2311_09549_b200/probe, over lane-group widths,
    numbers of rows in flight and blocks per SM, for uniformly random row indices and for the tensor's own index
    stream.  Returns the sweep and its best entry, or None."""
    import ctypes
    which = {"spttm_ttm3": 1, "spttm_ttm4": 2, "ttmc3": 2, "mttkrp_gemm": 1}.get(w.expr)
    lib_path = os.path.join(ROOT, "paper_2311_09549_b200", "probe", "libsaprobe.so")
    if which is None or not os.path.exists(lib_path):
        return None
    table = ops[which]
    rows, cols = int(table.shape[0]), int(table.shape[1])
    if cols not in (16, 32):
        return None
    lib = ctypes.CDLL(lib_path)
    vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    lib.sa_probe_row_gather.argtypes = [vp, i64, i64, ci, vp, i64, vp, ci, ci, ci, vp]
    lib.sa_probe_row_gather.restype = ci
    n = int(w.nnz)
    g = torch.Generator(device=dev)
    g.manual_seed(12345)
    streams = {"uniform random rows": torch.randint(0, rows, (n,), dtype=torch.int32, device=dev, generator=g)}
    last = tensor.order - 1
    _, crd, _ = sa.sa_tensor_export(tensor.handle, last, n_crd=n)
    streams["the tensor's last-mode indices in storage order"] = torch.from_numpy(crd).to(dev)
    sink = torch.zeros(1, dtype=torch.float32, device=dev)
    nbytes = n * cols * 4
    sweep = []
    for name, idx in streams.items():
        for lanes in (4, 8):
            for inflight in (4, 8, 16):
                for bps in (4, 8, 16):
                    def run():
                        rc = lib.sa_probe_row_gather(table.data_ptr(), rows, table.stride(0), cols, idx.data_ptr(), n,
                                                     sink.data_ptr(), lanes, inflight, bps, stream.cuda_stream)
                        if rc != 0:
                            raise RuntimeError("probe launch failed (%d)" % rc)
                    for _ in range(2):
                        run()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize(dev)
                    e0.record(stream)
                    reps = 5
                    for _ in range(reps):
                        run()
                    e1.record(stream)
                    torch.cuda.synchronize(dev)
                    ms = e0.elapsed_time(e1) / reps
                    sweep.append({"indices": name, "lanes_per_row": lanes, "rows_in_flight": inflight, "blocks_per_sm": bps,
                                  "ms": round(ms, 4), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1)})
    best = min(sweep, key=lambda r: r["ms"])
    # the same rows through the copy engine (cp.async.bulk.tensor tile::gather4 into shared memory, read back from there)
    lib.sa_probe_tma_gather.argtypes = [vp, i64, i64, ci, vp, i64, vp, ci, ci, vp, vp]
    lib.sa_probe_tma_gather.restype = ci
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    sink2 = torch.zeros(2, dtype=torch.float32, device=dev)
    idx = streams["the tensor's last-mode indices in storage order"]
    tma = []
    for stages in (1, 2, 4):
        for bps in (2, 4, 8):
            def run():
                rc = lib.sa_probe_tma_gather(table.data_ptr(), rows, table.stride(0), cols, idx.data_ptr(), n, sink2.data_ptr(),
                                             stages, bps, status.data_ptr(), stream.cuda_stream)
                if rc != 0:
                    raise RuntimeError("copy-engine probe launch failed (%d)" % rc)
            run()
            torch.cuda.synchronize(dev)
            if int(status[0]) != 0:
                raise RuntimeError("copy-engine probe gave up waiting for its rows (status %d)" % int(status[0]))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            reps = 3
            for _ in range(reps):
                run()
            e1.record(stream)
            torch.cuda.synchronize(dev)
            ms = e0.elapsed_time(e1) / reps
            tma.append({"groups_of_16_rows_in_flight_per_warp": stages, "blocks_of_4_warps_per_sm": bps, "ms": round(ms, 4),
                        "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1)})
    return {"what": "bare gather of one %d-byte factor row per nonzero from the L2-resident %d x %d table "
                    "(plus 4 index bytes per row from HBM); best of %d shapes" % (cols * 4, rows, cols, len(sweep)),
            "ms": best["ms"], "gbs": best["gbs"], "best": best, "sweep": sweep,
            "copy_engine_gather4": {"what": "the same rows fetched four per instruction by the copy engine into shared memory and "
                                            "read back from there (the tensor's own indices)",
                                    "ms": min(r["ms"] for r in tma), "sweep": tma}}


def nest_sample(w, target_nnz=4_000_000, seed=7):
    """Time the paper's scheduled loop nest of the chain on the host cores (oracle/nests.c: fp64, OpenMP over i), on
    seeded random output slices / rows holding about target_nnz nonzeros.  The sort into compressed storage is not
    timed (the GPU figure excludes the build as well).  Returns None for chains without a nest there."""
    import collections
    from oracle import nests
    import oracle
    if w.expr not in ("spttm_ttm3", "spttm_ttm4", "ttmc3", "sddmm_spmm", "spmm_gemm"):
        return None
    I = int(w.dims[0])
    i = w.coords[:, 0]
    counts = np.bincount(i, minlength=I)
    rs = np.random.RandomState(seed)
    cand = rs.permutation(I)
    cand = cand[counts[cand] <= max(1, target_nnz // 4)]           # one slice must not dominate the sample
    csum = np.cumsum(counts[cand])
    n_sel = min(int(np.searchsorted(csum, target_nnz, side="left")) + 1, cand.shape[0])
    sel = np.sort(cand[:n_sel])
    remap = np.full(I, -1, dtype=np.int64)
    remap[sel] = np.arange(n_sel)
    keep = remap[i] >= 0
    coords = w.coords[keep].copy()
    coords[:, 0] = remap[coords[:, 0]]
    dense = list(w.dense)
    if w.expr in ("sddmm_spmm", "ttmc3"):
        dense[0] = np.ascontiguousarray(dense[0][sel])             # the operand indexed by i
    Sub = collections.namedtuple("Sub", "expr dims coords vals dense")
    sub = Sub(w.expr, (n_sel,) + tuple(int(d) for d in w.dims[1:]), coords, w.vals[keep], dense)
    run = nests.prepare(sub, order="left")      # (B.C).D: its cost follows the sampled rows (C.D would be formed for all J)
    run()
    t0 = time.perf_counter()
    run()
    dt = time.perf_counter() - t0
    nnz_sel = int(keep.sum())
    return {"value": nnz_sel / dt / 1e9, "unit": "GNNZ/s", "cores": oracle.max_threads(), "kind": "paper's scheduled nest (fp64)",
            "sample": "%d of %d output slices/rows (seeded random among those with <= %d nonzeros), %d of %d nonzeros"
                      % (n_sel, I, max(1, target_nnz // 4), nnz_sel, int(w.nnz))}


def aggregate_throughput(nnz_per_rank, world, ms_per_step):
    """Whole-job GNNZ/s of ``world`` independent replicas that all finish within ms_per_step."""
    return world * nnz_per_rank / (ms_per_step * 1e-3) / 1e9


def workload_label(cfg, sched):
    names = {1: "cfg1 <SpTTM,TTM> 200^3 20k nnz L=M=16", 2: "cfg2 <SpTTM,TTM> 100000x80000x80000 50M nnz Zipf(1.2) L=M=32",
             3: "cfg3 <SDDMM,SpMM> 1Mx1M 30M nnz K=L=64", 4: "cfg4 <SpMM,GEMM> 4Mx4M 100M nnz L=256 M=64",
             5: "cfg5 order-4 <SpTTM,TTM> 50000x20000^3 100M nnz ranks 16",
             7: "kernel 2 <SDDMM,SpMM,GEMM> on the config-3 tensor, K=L=M=64",
             6: "kernel 5 <3D TTMC> on a nell-2-shaped tensor 12000x9000x288000 76.88M nnz L=M=N=16",
             8: "kernel 3 <SpMMH,GEMM> on the config-4 tensor recipe 4Mx4M 100M nnz L=256 M=64",
             9: "kernel 8 <MTTKRP,GEMM> on the config-2 tensor, R=32 M=32",
             10: "kernel 7 <SpTTM,SpTTM> on the config-2 tensor, L=M=32, sparse output (one row per (i,j) fiber)",
             11: "kernel 5 <3D TTMC> on a flickr-3d-shaped tensor 320000x2820000x1600000 112.89M nnz L=M=N=16"}
    return names[cfg] + (" (%s)" % sched if cfg in (4, 5, 6, 10, 11) else "")


def label(args):
    cfg = args.workload or 2
    sched = args.sched or ("right" if cfg in (4, 10) else "default")
    return workload_label(cfg, sched) + ("" if args.scale == "full" else " [%s-scale stand-in]" % args.scale)


def run_reference(args, w, rank, world):
    if rank != 0:
        return
    vals = []
    last = None
    for step in range(args.warmup + args.steps):
        last = oracle_sample(w, budget_s=min(6.0, 150.0 / max(1, args.warmup + args.steps)))
        if step >= args.warmup:
            vals.append(last)
    v = statistics.median(x["value"] for x in vals)
    ms = statistics.median(x["seconds"] for x in vals) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "GNNZ/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": label(args)},
            "cpu_baseline": {"value": v, "unit": "GNNZ/s", "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": v, "unit": "GNNZ/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def measure(sa, torch, dist, w, sched_name, steps, warmup, e2e_steps, dev, rank, world, sample_clocks=True,
            gather_probe=False, scale="full", workload_id=None):
    """Time ``steps`` steps of workload ``w`` (after ``warmup`` untimed ones) with CUDA events on the launching
    stream, then the same call end to end from / to pinned host memory.  Returns the record of one
    (config, schedule) pair (rank 0; other ranks return None after taking part in the barriers)."""
    fmt = sa.SA_FMT_CSR if w.fmt == "csr" else sa.SA_FMT_CSF
    t0 = time.perf_counter()
    tensor = sa.SparseTensor(w.dims, w.coords, w.vals, fmt, device=dev.index)
    build_s = time.perf_counter() - t0
    nnz, counts, n_chunks = tensor.info()
    two_schedules = w.expr in ("spttm_ttm4", "ttmc3")          # fused / fissioned
    sched = {"left": sa.SA_SCHED_ASSOC_LEFT, "right": sa.SA_SCHED_ASSOC_RIGHT, "default": sa.SA_SCHED_DEFAULT,
             "fused": sa.SA_SCHED_FUSED if two_schedules else sa.SA_SCHED_DEFAULT, "fissioned": sa.SA_SCHED_FISSIONED}[sched_name]
    host_ops = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in w.dense]
    ops = [x.to(dev, non_blocking=False) for x in host_ops]
    out = torch.empty(w.out_shape, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step():
        tensor.run(w.expr, ops, out=out, sched=sched, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(warmup):
        step()
    launches_per_step = sa.sa_last_launch_count(tensor.handle)
    barrier()
    sampler = ClockSampler(dev.index)
    if rank == 0 and sample_clocks:
        sampler.start()
        time.sleep(0.3)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    evs[0].record(stream)
    for k in range(steps):
        step()
        evs[k + 1].record(stream)
    barrier()
    total_ms = evs[0].elapsed_time(evs[-1])
    per_step = [evs[k].elapsed_time(evs[k + 1]) for k in range(steps)]
    clocks = None
    if rank == 0 and sample_clocks:
        # keep the GPU busy a little longer so that the clock sampler sees the loaded state
        t_end = time.perf_counter() + 1.0
        while time.perf_counter() < t_end:
            for _ in range(20):
                step()
            torch.cuda.synchronize(dev)
        clocks = sampler.stop()

    # end to end: dense operands from pinned host memory, result back to pinned host memory
    host_out = torch.empty(w.out_shape, dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(e2e_steps, steps))

    def e2e_step():
        dops = [x.to(dev, non_blocking=True) for x in host_ops]
        tensor.run(w.expr, dops, out=out, sched=sched, stream=stream)
        host_out.copy_(out, non_blocking=True)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    total_ms, e2e_ms = reduce_max_over_ranks([total_ms, e2e_ms], dev, world)
    ms_per_step = total_ms / steps
    rec = None
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        # the schedule that ran: the library's choice when the default was asked for
        ran = sched_name
        if sched_name == "default":
            ops_desc = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in ops]
            resolved = sa.sa_schedule_cost(tensor.handle, sa._EXPR_OF[w.expr], sa.SA_SCHED_DEFAULT, ops_desc)["resolved"]
            ran = {sa.SA_SCHED_FUSED: "fused", sa.SA_SCHED_ASSOC_LEFT: "left", sa.SA_SCHED_ASSOC_RIGHT: "right",
                   sa.SA_SCHED_FISSIONED: "fissioned"}[resolved]
        abytes, aflops = algorithmic_work(w, counts, ran)
        achieved = abytes / (ms_per_step * 1e-3) / 1e9
        traffic, traffic_kernel = ncu_traffic(workload_id, ran) if scale == "full" else (None, None)
        rec = {
            "workload": workload_label(workload_id, sched_name) + ("" if scale == "full" else " [%s-scale stand-in]" % scale),
            "schedule": sched_name if sched_name == ran else "%s (ran %s)" % (sched_name, ran),
            "value": aggregate_throughput(nnz, world, ms_per_step), "unit": "GNNZ/s", "ms_per_step": ms_per_step,
            "steps": steps, "warmup": warmup, "step_ms_median": statistics.median(per_step),
            "step_ms_stdev": statistics.pstdev(per_step), "nnz": nnz, "level_counts": [int(c) for c in counts],
            "work_items": int(n_chunks), "build_s": round(build_s, 3),
            "l2": "inputs + output exceed L2 (126 MB); no flush" if abytes > 200e6 else "smaller than L2; launch-bound",
            "gflops": aflops / (ms_per_step * 1e-3) / 1e9,
            "hbm_gbs_algorithmic": achieved, "hbm_frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": traffic, "peak_kind": "of " + peak_kind,
                         "kernel": "whole step (main kernel(s) + fix-up, fix-up <= 4 % by the ncu launch lists)",
                         "traffic_kernel": traffic_kernel, "algorithmic_bytes_per_launch": abytes},
            "e2e": {"value": aggregate_throughput(nnz, world, e2e_ms), "unit": "GNNZ/s",
                    "h2d_bytes_per_step": sum(int(x.numel()) * 4 for x in host_ops),
                    "d2h_bytes_per_step": int(host_out.numel()) * 4, "ms_per_step": e2e_ms},
            "gpu_launches": launches_per_step * steps, "clocks": clocks,
        }
        if gather_probe and scale == "full":
            gather = l2_gather_ceiling(sa, torch, w, tensor, ops, dev, stream)
            if gather is not None:
                rec["l2_gather_ceiling"] = gather
    tensor.close()
    del ops, out, host_ops, host_out
    torch.cuda.empty_cache()
    return rec


# (config, schedule) pairs of the default run besides the headline config 2
PER_CONFIG = [(1, "fused"), (3, "fused"), (4, "left"), (4, "right"), (4, "default"), (5, "fused"), (5, "fissioned"), (5, "default")]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=31)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=None, choices=[1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11],
                    help="one workload only; without it: config 2 as the headline plus a per_config list of all five configs")
    ap.add_argument("--scale", default="full", choices=["full", "mid", "mini"])
    ap.add_argument("--sched", default=None, choices=["left", "right", "fused", "fissioned", "default"],
                    help="schedule: left / right (association order, workloads 4 and 10), fused / fissioned (workloads 5, 6, 11), "
                         "default (the library's choice; also the default here, except workloads 4 and 10: right)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=5)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    all_configs = args.workload is None and not args.no_per_config and args.scale == "full" and args.impl == "ours"
    if args.workload is None:
        args.workload = 2

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            w = configs.make(args.workload, args.scale)
            run_reference(args, w, rank, world)
        return 0

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the executor has no CPU path")
    import paper_2311_09549_b200 as sa

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    all_configs = all_configs and world == 1

    # the other configs' inputs are generated on host threads while the GPU runs (numpy releases the GIL)
    pending = {}
    pool = None
    if all_configs:
        from concurrent.futures import ThreadPoolExecutor
        pool = ThreadPoolExecutor(max_workers=2)
        for cfg in sorted({c for c, _ in PER_CONFIG}, key=lambda c: (c != 5, c != 4, c)):
            pending[cfg] = pool.submit(configs.make, cfg, "full")

    w = configs.make(args.workload, args.scale)
    if w.expr in ("spmm_gemm", "spttm_spttm"):
        sched_name = args.sched if args.sched in ("left", "right", "default") else "right"
    elif w.expr in ("spttm_ttm4", "ttmc3"):
        sched_name = args.sched if args.sched in ("fused", "fissioned", "default") else "default"
    else:
        sched_name = "fused"
    rec = measure(sa, torch, dist, w, sched_name, args.steps, args.warmup, args.e2e_steps, dev, rank, world,
                  gather_probe=True, scale=args.scale, workload_id=args.workload)
    if rank == 0:
        line = {
            "metric": METRIC, "value": rec["value"], "unit": "GNNZ/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": rec["workload"], "scale": args.scale, "nnz": rec["nnz"],
                       "level_counts": rec["level_counts"], "work_items": rec["work_items"], "l2": rec["l2"],
                       "parallelism": "replicas x%d" % world, "build_s": rec["build_s"],
                       "step_ms_median": rec["step_ms_median"], "step_ms_stdev": rec["step_ms_stdev"]},
            "gflops": rec["gflops"], "hbm_gbs_algorithmic": rec["hbm_gbs_algorithmic"],
            "hbm_frac_of_nominal_8000": rec["hbm_frac_of_nominal_8000"], "roofline": rec["roofline"],
            "e2e": rec["e2e"], "gpu_launches": rec["gpu_launches"], "clocks": rec["clocks"],
        }
        if "l2_gather_ceiling" in rec:
            line["l2_gather_ceiling"] = rec["l2_gather_ceiling"]
        kept = {args.workload: w}
        records = [dict(rec, config=args.workload)]
        if all_configs:
            steps_pc = min(args.steps, 10)
            for cfg, sname in PER_CONFIG:
                if cfg not in kept:
                    kept[cfg] = pending[cfg].result()
                r = measure(sa, torch, dist, kept[cfg], sname, steps_pc, args.warmup, min(args.e2e_steps, 2), dev, rank, world,
                            scale="full", workload_id=cfg)
                records.append(dict(r, config=cfg))
            pool.shutdown()
        if not args.no_cpu_baseline and world == 1:
            budget = 15.0 if not all_configs else 6.0
            done = {}
            for r in records:
                cfg = r["config"]
                if cfg not in done:
                    cb = oracle_sample(kept[cfg], budget_s=budget)
                    cb.pop("seconds")
                    done[cfg] = cb
                r["cpu_baseline"] = done[cfg]
            line["cpu_baseline"] = done[args.workload]
            nest = nest_sample(kept[args.workload])
            if nest is not None:
                line["cpu_scheduled_nest"] = nest
        if all_configs:
            line["per_config"] = records
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
